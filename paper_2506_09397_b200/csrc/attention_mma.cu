// Ragged verification attention over the paged bf16 cache on tensor cores.
//
// A work item is (request, KV head, chunk of keys).  The q_len * (Hq/Hkv) query rows that share
// the KV head form the M side of warp-level bf16 MMAs (16 rows per warp, up to 64 per pass);
// keys stream through shared memory in tiles of 64 (four 16-token pages).  Every (page, KV head)
// block of the cache is a contiguous [16][h] array, fetched by TMA (boxes of 16 rows x 64
// columns, 128-byte swizzle, so ldmatrix reads are bank-conflict free) into a ring of stages
// guarded by full/empty mbarriers; a fifth warp issues all copies, so the four computing warps never
// meet at a block-wide barrier inside the key loop.  When a request has few query rows (<= 16 or
// <= 32) the warps split each key tile among themselves instead and merge at the end.  S = Q K^T and O += P V use
// mma.sync.m16n8k16 with fp32 accumulation; the softmax is the usual online form in fp32 with
// base-2 exponentials.  Each chunk either writes the normalised output (request not split) or
// its partial (max, normaliser, unnormalised output) for the merge kernel.  The cached prefix does not depend on
// the kernel that runs before this one (only the newest k+1 slots do): its first tiles are requested before the
// programmatic-launch dependency wait.
#include <cuda_bf16.h>

#include "common.cuh"
#include "kernels.h"

namespace sled {

namespace {

constexpr int kTile = 64;        // keys per tile
constexpr int kStages = 3;
constexpr long long kWaitCycles = 200000000LL;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}

// bounded wait; gives up at once when another warp of the block already has (*stop set)
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* stop) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*stop != 0 || clock64() - t0 > kWaitCycles) return false;
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y), "l"(policy)
      : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float c[4], const uint32_t a[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Shared-memory stage: K then V, each as H/64 sub-tiles of [64 keys][64 columns] (128-byte rows,
// chunk c of row r stored at chunk position c ^ (r & 7)); page p of the tile owns rows 16p..16p+15.
template <int H>
struct StageLayout {
  static constexpr int kHalves = H / 64;
  static constexpr int kSub = kTile * 128;             // 8 KB
  static constexpr int kKBytes = kHalves * kSub;
  static constexpr int kBytes = 2 * kKBytes;
  static constexpr int kTotal = kStages * kBytes + 1024 + 16 * kStages + 64;
};

struct ItemCtx {
  int req, kvh, key_start, key_count, key_end, n_tiles;
  int group, row0, n_rows, kv_base, chunk_idx;
  bool split;
  float scale;
};

// Consumer side of one work item for the case that MT warps cover the query rows (16 each) and the
// remaining 4/MT-fold parallelism goes over the keys: warp w handles m-tile w % MT and, of every 64-key
// tile, the 16*MT keys starting at (w / MT) * 16 * MT.  Warps that shared an m-tile merge their
// (max, normaliser, output) through shared memory at the end.
template <int H, int MT>
__device__ __forceinline__ void consume_item(const AttnArgs& a, const ItemCtx& c, int rbase, uint32_t base, uint32_t bar_full,
                                             uint32_t bar_empty, int& it, volatile int* s_abort, float* merge_buf) {
  using L = StageLayout<H>;
  constexpr int KS = H / 16;     // k-steps of Q K^T
  constexpr int DN = H / 8;      // n-tiles of the output
  constexpr int NT = 2 * MT;     // key n-tiles (8 keys) per warp and tile
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tq = lane & 3;
  const int mt = warp % MT, kq = warp / MT;
  const int key_off = kq * 16 * MT;
  const __nv_bfloat16* qbuf = static_cast<const __nv_bfloat16*>(a.q);

  const int r_lo = rbase + mt * 16 + g, r_hi = r_lo + 8;
  const bool active = rbase + mt * 16 < c.n_rows;
  const bool v_lo = r_lo < c.n_rows, v_hi = r_hi < c.n_rows;
  const int j_lo = v_lo ? r_lo / c.group : 0, j_hi = v_hi ? r_hi / c.group : 0;
  const int head_lo = c.kvh * c.group + (v_lo ? r_lo % c.group : 0), head_hi = c.kvh * c.group + (v_hi ? r_hi % c.group : 0);
  const int vis_lo = c.kv_base + j_lo, vis_hi = c.kv_base + j_hi;   // last key index each row may see

  // Q fragments (A operand, 16 x 16 per k-step), straight from global memory
  uint32_t qf[KS][4];
  {
    const uint32_t* q_lo = reinterpret_cast<const uint32_t*>(qbuf + (static_cast<int64_t>(c.row0 + j_lo) * a.Hq + head_lo) * H);
    const uint32_t* q_hi = reinterpret_cast<const uint32_t*>(qbuf + (static_cast<int64_t>(c.row0 + j_hi) * a.Hq + head_hi) * H);
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qf[ks][0] = (active && v_lo) ? q_lo[ks * 8 + tq] : 0u;
      qf[ks][1] = (active && v_hi) ? q_hi[ks * 8 + tq] : 0u;
      qf[ks][2] = (active && v_lo) ? q_lo[ks * 8 + 4 + tq] : 0u;
      qf[ks][3] = (active && v_hi) ? q_hi[ks * 8 + 4 + tq] : 0u;
    }
  }
  float o[DN][4];
#pragma unroll
  for (int i = 0; i < DN; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
  bool failed = false;

  for (int tile = 0; tile < c.n_tiles; ++tile, ++it) {
    const int s = it % kStages;
    if (*s_abort || !mbar_wait(bar_full + 8 * s, (it / kStages) & 1, s_abort)) { *s_abort = 1; failed = true; break; }
    if (active) {
      const uint32_t kb = base + s * L::kBytes, vb = kb + L::kKBytes;
      const int k0 = c.key_start + tile * kTile + key_off;    // first key of this warp's share
      // ---- S = Q K^T : 16 rows x 16*MT keys
      float sc[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) { sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f; }
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
        for (int np = 0; np < MT; ++np) {          // two key n-tiles per ldmatrix.x4
          const int key = key_off + (np * 2 + (lane >> 4)) * 8 + (lane & 7);
          const int chunk = 2 * ks + ((lane >> 3) & 1);
          const uint32_t addr = kb + (chunk >> 3) * L::kSub + key * 128 + (((chunk & 7) ^ (key & 7)) << 4);
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4(addr, b0, b1, b2, b3);
          mma_bf16(sc[np * 2], qf[ks], b0, b1);
          mma_bf16(sc[np * 2 + 1], qf[ks], b2, b3);
        }
      }
      // ---- scale, mask, online softmax
      const bool need_mask = (k0 + 16 * MT - 1 > c.kv_base) || (k0 + 16 * MT > c.key_end);
      float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float v = sc[nt][e] * c.scale;
          if (need_mask) {
            const int kk = k0 + nt * 8 + 2 * tq + (e & 1);
            const int vis = (e < 2) ? vis_lo : vis_hi;
            if (kk > vis || kk >= c.key_end) v = -INFINITY;
          }
          sc[nt][e] = v;
        }
        mx_lo = fmaxf(mx_lo, fmaxf(sc[nt][0], sc[nt][1]));
        mx_hi = fmaxf(mx_hi, fmaxf(sc[nt][2], sc[nt][3]));
      }
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
      const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
      const float ms_lo = mn_lo == -INFINITY ? 0.f : mn_lo, ms_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
      const float al_lo = exp2f(m_lo - ms_lo), al_hi = exp2f(m_hi - ms_hi);
      m_lo = mn_lo;
      m_hi = mn_hi;
      l_lo *= al_lo;
      l_hi *= al_hi;
#pragma unroll
      for (int i = 0; i < DN; ++i) { o[i][0] *= al_lo; o[i][1] *= al_lo; o[i][2] *= al_hi; o[i][3] *= al_hi; }
      uint32_t pf[MT][4];   // P as A operand: MT k-steps of 16 keys
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const float p0 = exp2f(sc[nt][0] - ms_lo), p1 = exp2f(sc[nt][1] - ms_lo);
        const float p2 = exp2f(sc[nt][2] - ms_hi), p3 = exp2f(sc[nt][3] - ms_hi);
        l_lo += p0 + p1;
        l_hi += p2 + p3;
        pf[nt >> 1][(nt & 1) * 2] = pack_bf16(p0, p1);
        pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
      }
      // ---- O += P V : 16 rows x H columns over this warp's keys
#pragma unroll
      for (int kt = 0; kt < MT; ++kt) {
#pragma unroll
        for (int dp = 0; dp < DN / 2; ++dp) {     // two output n-tiles per ldmatrix.x4.trans
          const int key = key_off + kt * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
          const int chunk = dp * 2 + (lane >> 4);
          const uint32_t addr = vb + (chunk >> 3) * L::kSub + key * 128 + (((chunk & 7) ^ (key & 7)) << 4);
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4_trans(addr, b0, b1, b2, b3);
          mma_bf16(o[dp * 2], pf[kt], b0, b1);
          mma_bf16(o[dp * 2 + 1], pf[kt], b2, b3);
        }
      }
    }
    __syncwarp();
    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_empty + 8 * s) : "memory");
  }

  // row sums over the four threads that share a row
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);

  if (MT < 4) {
    // merge the key shares of an m-tile: warps with kq > 0 publish, the kq == 0 warp combines.
    // Layout [share][value j][lane]: the same lane of every warp holds the same matrix positions.
    // (The stage memory is free: every tile of this pass has been consumed by all warps.)
    constexpr int kVals = DN * 4 + 4;
    asm volatile("bar.sync 2, 128;" ::: "memory");   // all consumer warps are past their last tile
    if (kq > 0) {
      float* dst = merge_buf + (static_cast<size_t>((kq - 1) * MT + mt) * kVals) * 32 + lane;
#pragma unroll
      for (int i = 0; i < DN; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) dst[(i * 4 + e) * 32] = o[i][e];
      dst[(DN * 4 + 0) * 32] = m_lo;
      dst[(DN * 4 + 1) * 32] = m_hi;
      dst[(DN * 4 + 2) * 32] = l_lo;
      dst[(DN * 4 + 3) * 32] = l_hi;
    }
    asm volatile("bar.sync 2, 128;" ::: "memory");
    if (kq == 0) {
      for (int sh = 1; sh < 4 / MT; ++sh) {
        const float* src = merge_buf + (static_cast<size_t>((sh - 1) * MT + mt) * kVals) * 32 + lane;
        const float om_lo = src[(DN * 4 + 0) * 32], om_hi = src[(DN * 4 + 1) * 32];
        const float ol_lo = src[(DN * 4 + 2) * 32], ol_hi = src[(DN * 4 + 3) * 32];
        const float nm_lo = fmaxf(m_lo, om_lo), nm_hi = fmaxf(m_hi, om_hi);
        const float s_lo = nm_lo == -INFINITY ? 0.f : nm_lo, s_hi = nm_hi == -INFINITY ? 0.f : nm_hi;
        const float a_lo = exp2f(m_lo - s_lo), a_hi = exp2f(m_hi - s_hi);
        const float b_lo = exp2f(om_lo - s_lo), b_hi = exp2f(om_hi - s_hi);
#pragma unroll
        for (int i = 0; i < DN; ++i) {
          o[i][0] = o[i][0] * a_lo + src[(i * 4 + 0) * 32] * b_lo;
          o[i][1] = o[i][1] * a_lo + src[(i * 4 + 1) * 32] * b_lo;
          o[i][2] = o[i][2] * a_hi + src[(i * 4 + 2) * 32] * b_hi;
          o[i][3] = o[i][3] * a_hi + src[(i * 4 + 3) * 32] * b_hi;
        }
        l_lo = l_lo * a_lo + ol_lo * b_lo;
        l_hi = l_hi * a_hi + ol_hi * b_hi;
        m_lo = nm_lo;
        m_hi = nm_hi;
      }
    }
    asm volatile("bar.sync 2, 128;" ::: "memory");   // merge_buf may be overwritten by the next pass's tiles
  }

  // ---- write this pass's rows
  if (active && kq == 0 && !failed && !*s_abort) {
    if (!c.split) {
      const float i_lo = 1.f / l_lo, i_hi = 1.f / l_hi;
      __nv_bfloat16* out = static_cast<__nv_bfloat16*>(a.out);
      uint32_t* o_lo = reinterpret_cast<uint32_t*>(out + (static_cast<int64_t>(c.row0 + j_lo) * a.Hq + head_lo) * H);
      uint32_t* o_hi = reinterpret_cast<uint32_t*>(out + (static_cast<int64_t>(c.row0 + j_hi) * a.Hq + head_hi) * H);
#pragma unroll
      for (int i = 0; i < DN; ++i) {
        if (v_lo) o_lo[i * 4 + tq] = pack_bf16(o[i][0] * i_lo, o[i][1] * i_lo);
        if (v_hi) o_hi[i * 4 + tq] = pack_bf16(o[i][2] * i_hi, o[i][3] * i_hi);
      }
    } else {
      const int64_t p_lo = static_cast<int64_t>(a.tok_part[c.row0 + j_lo] + c.chunk_idx) * a.Hq + head_lo;
      const int64_t p_hi = static_cast<int64_t>(a.tok_part[c.row0 + j_hi] + c.chunk_idx) * a.Hq + head_hi;
#pragma unroll
      for (int i = 0; i < DN; ++i) {
        if (v_lo) *reinterpret_cast<float2*>(a.part_acc + p_lo * H + i * 8 + 2 * tq) = make_float2(o[i][0], o[i][1]);
        if (v_hi) *reinterpret_cast<float2*>(a.part_acc + p_hi * H + i * 8 + 2 * tq) = make_float2(o[i][2], o[i][3]);
      }
      if (tq == 0) {
        if (v_lo) { a.part_ml[p_lo * 2] = m_lo; a.part_ml[p_lo * 2 + 1] = l_lo; }
        if (v_hi) { a.part_ml[p_hi * 2] = m_hi; a.part_ml[p_hi * 2 + 1] = l_hi; }
      }
    }
  }
}

// 160 threads: warps 0-3 compute, warp 4 issues the TMA copies (one thread).
template <int H>
__global__ void __launch_bounds__(160, 2) attn_mma_kernel(AttnArgs a, const __grid_constant__ CUtensorMap map_k,
                                                        const __grid_constant__ CUtensorMap map_v) {
  using L = StageLayout<H>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t bar_full = base + kStages * L::kBytes, bar_empty = bar_full + 8 * kStages;
  __shared__ int s_abort_mem;
  volatile int* s_abort = &s_abort_mem;

  const int warp = threadIdx.x >> 5;
  const LaunchStamp stamp{a.stamp.begin, a.stamp.end};
  stamp_begin(stamp);
  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    *s_abort = 0;
    for (int s = 0; s < kStages; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar_full + 8 * s), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar_empty + 8 * s), "r"(4));   // one arrival per computing warp
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_k)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_v)) : "memory");
  }
  __syncthreads();
  const int4 item = a.items[blockIdx.x];
  ItemCtx c;
  c.req = item.x; c.kvh = item.y; c.key_start = item.z; c.key_count = item.w;
  c.key_end = c.key_start + c.key_count;
  c.n_tiles = (c.key_count + kTile - 1) / kTile;
  c.group = a.Hq / a.Hkv;
  c.row0 = a.cu_q[c.req];
  c.n_rows = (a.cu_q[c.req + 1] - c.row0) * c.group;
  c.kv_base = a.kv_base[c.req];
  c.split = a.req_chunks[c.req] > 1;
  c.chunk_idx = c.key_start / a.req_chunk_keys[c.req];
  c.scale = rsqrtf(static_cast<float>(H)) * 1.4426950408889634f;
  const int n_pass = (c.n_rows + 63) / 64;
  // Everything above reads only what the host wrote before the step.  The queries and the cache slots of the step's
  // own tokens (key index >= kv_base) come from the preceding kernel; the cached prefix does not.

  if (warp == 4) {
    if ((threadIdx.x & 31) == 0) {
      const int32_t* pages = a.page_table + a.pt_off[c.req];
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      auto load_tile = [&](int tile, int s) {
        const uint32_t bar = bar_full + 8 * s;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(L::kBytes) : "memory");
        const uint32_t dst = base + s * L::kBytes;
#pragma unroll
        for (int p = 0; p < 4; ++p) {
          int kk = c.key_start + tile * kTile + p * 16;
          if (kk >= c.key_end) kk = c.key_end - 1;            // past the chunk: re-read a valid page (masked later)
          const int row = (pages[kk >> 4] * a.Hkv + c.kvh) * 16;
#pragma unroll
          for (int hh = 0; hh < L::kHalves; ++hh) {
            tma_load_2d(dst + hh * L::kSub + p * 2048, &map_k, hh * 64, row, bar, policy);
            tma_load_2d(dst + L::kKBytes + hh * L::kSub + p * 2048, &map_v, hh * 64, row, bar, policy);
          }
        }
      };
      // tiles that lie wholly inside the cached prefix are requested before the dependency wait (the ring is empty:
      // nothing to wait for), so the cache streams while the preceding kernel is still writing the new slots
      const int safe_tiles = c.key_end <= c.kv_base ? c.n_tiles : max(0, c.kv_base - c.key_start) / kTile;
      const int pre = min(min(kStages, c.n_tiles), safe_tiles);
      for (int tile = 0; tile < pre; ++tile) load_tile(tile, tile);
      pdl_wait();
      int it = pre;
      for (int pass = 0; pass < n_pass && !*s_abort; ++pass) {
        for (int tile = pass == 0 ? pre : 0; tile < c.n_tiles; ++tile, ++it) {
          const int s = it % kStages;
          if (*s_abort || !mbar_wait(bar_empty + 8 * s, ((it / kStages) & 1) ^ 1, s_abort)) { *s_abort = 1; break; }
          load_tile(tile, s);
        }
      }
    } else {
      pdl_wait();
      // an earlier kernel that gave up has left a code in *error: the copy-issuing warp's second lane (idle
      // otherwise) looks, so that nobody waits for this load; every loop below polls the flag
      if (threadIdx.x == 129 && *reinterpret_cast<volatile int32_t*>(a.error) != 0) *s_abort = 1;
    }
  } else {
    pdl_wait();
    int it = 0;
    float* merge_buf = reinterpret_cast<float*>(base_ptr);
    for (int pass = 0; pass < n_pass; ++pass) {   // no early exit: the warps meet at named barriers inside
      const int rows_here = min(64, c.n_rows - pass * 64);
      if (rows_here <= 16) consume_item<H, 1>(a, c, pass * 64, base, bar_full, bar_empty, it, s_abort, merge_buf);
      else if (rows_here <= 32) consume_item<H, 2>(a, c, pass * 64, base, bar_full, bar_empty, it, s_abort, merge_buf);
      else consume_item<H, 4>(a, c, pass * 64, base, bar_full, bar_empty, it, s_abort, merge_buf);
    }
  }
  __syncthreads();
  if (*s_abort) {
    if (threadIdx.x == 0) atomicCAS(a.error, 0, 4);
    // copies that were issued may still land: wait a little before the shared memory goes away
    const long long t1 = clock64();
    while (clock64() - t1 < 2000000LL) __nanosleep(1000);
  }
  stamp_end(stamp);
}

template <int H>
int launch_h(const AttnArgs& a, cudaStream_t s) {
  using L = StageLayout<H>;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(attn_mma_kernel<H>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal) != cudaSuccess)
      return -1;
    configured = true;
  }
  SLED_LAUNCH_PDL(attn_mma_kernel<H>, dim3(a.n_items), dim3(160), L::kTotal, s, a, *a.map_k, *a.map_v);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace

int launch_attention_mma(const AttnArgs& a, cudaStream_t s) {
  if (!a.map_k || !a.map_v || !a.error || a.page_size != 16) return -1;
  if (a.h == 128) return launch_h<128>(a, s);
  if (a.h == 64) return launch_h<64>(a, s);
  return -1;
}

}  // namespace sled
