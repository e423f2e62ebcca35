// Ragged verification attention on the 5th-generation tensor cores (tcgen05), for head_dim 128, bf16 cache,
// 16-token pages and up to 128 query rows per work item.
//
// A work item is (request, KV head, chunk of keys); its q_len * (Hq/Hkv) query rows are the M side (128 lanes of
// tensor memory, one row per lane) of two MMAs per 64-key tile:
//     S = Q K^T   (M 128 x N 64 keys,  K = 128 dims:  8 instructions of K 16)   -> tensor memory, fp32
//     O_t = P V   (M 128 x N 128 dims, K = 64 keys:   4 instructions of K 16)   -> tensor memory, fp32
// K and V pages arrive by TMA exactly as the cache stores them, [16 tokens][128 dims] per (page, KV head), as
// 128-byte swizzled rows of 64 dims; K is the K-major B operand of the first product, the same V tile is the
// MN-major B operand of the second (its rows are keys, i.e. the contraction runs down the rows), so nothing is
// transposed or copied.  The output accumulates in tensor memory over all tiles of the item.
// Eight softmax warps: a warp may only touch the 32 tensor-memory lanes of its quarter (warp index mod 4, which is
// also the SM's scheduler it runs on), so the query rows are dealt out over the four quarters (row r sits in lane
// 32 (r mod 4) + r / 4) and every quarter has two warps, one per half of a tile's 64 keys.  A thread reads its 32
// scores, the two halves of a row exchange their maxima through shared memory, P goes to shared memory as bf16 in
// the operand layout.  The row maximum used for the exponentials is only raised when a score exceeds it by more than
// 8 (a factor 256, harmless for bf16 probabilities and fp32 sums, and it cancels in the final division): raising it
// means rescaling the row of O in tensor memory, which is then rare (the first tiles of an item).  S and P are
// double-buffered: the scores of tile t+1 are computed under the softmax of tile t.
//   warps 0-7 : softmax + output (thread = query row x key half)
//   warp 8    : TMA producer (one thread), ring of 4 stages of 32 KB
//   warp 9    : tensor-memory allocation, MMA issue (one thread)
// Every wait on an mbarrier is bounded; when one runs out the block records a code in *error, lets copies in flight
// land, frees its tensor memory and returns.
#include <cuda_bf16.h>

#include "common.cuh"
#include "kernels.h"

namespace sled {

namespace {

constexpr int kTile = 64;            // keys per tile
constexpr int kStages = 4;
constexpr int kH = 128;              // head_dim
constexpr int kRows = 128;           // query rows per item (MMA M)
constexpr int kSub = kTile * 128;    // one [64 keys][64 dims] sub-tile of 128-byte rows: 8 KB
constexpr int kKBytes = 2 * kSub;    // K part of a stage (two halves of the head dimension)
constexpr int kStageBytes = 2 * kKBytes;
constexpr int kQBytes = 2 * kRows * 128;        // [2 halves][128 rows][64 dims]
constexpr int kPBytes = kRows * 128;            // [128 rows][64 keys] per buffer
constexpr int kOffQ = kStages * kStageBytes;
constexpr int kOffP = kOffQ + kQBytes;
constexpr int kOffX = kOffP + 2 * kPBytes;          // values exchanged between the two threads of a row: [3 slots][128 rows][2 halves] x (tag, value)
constexpr int kOffBar = kOffX + 3 * kRows * 2 * 8;
constexpr int kSmemBytes = kOffBar + 256 + 1024;   // barriers and the tensor-memory slot, plus alignment slack
constexpr long long kWaitCycles = 200000000LL;

// barrier indices (8 bytes each from kOffBar)
enum { B_FULL = 0, B_EMPTY = B_FULL + kStages, B_SFULL = B_EMPTY + kStages, B_SEMPTY = B_SFULL + 2, B_PFULL = B_SEMPTY + 2,
       B_ODONE = B_PFULL + 2, B_QFULL = B_ODONE + 1, B_COUNT = B_QFULL + 1 };
constexpr int kSoftmaxWarps = 8;
constexpr float kRaiseBy = 8.f;      // the reference maximum of a row is raised only by more than this (log2 units)

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
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// The two threads of a query row (different warps) hand each other one float: each writes (tag, value) as one
// 8-byte store into its own slot and polls the partner's slot until the tag shows up.  Bounded like every other
// wait here; no named barrier is involved, so a warp that has given up cannot leave its partner stuck.
__device__ __forceinline__ bool swap_with_partner(uint32_t mine, uint32_t theirs, uint32_t tag, float v, float* got,
                                                  volatile int* stop) {
  asm volatile("st.volatile.shared.v2.b32 [%0], {%1, %2};" ::"r"(mine), "r"(tag), "r"(__float_as_uint(v)) : "memory");
  const long long t0 = clock64();
  for (;;) {
    uint32_t tg, bits;
    asm volatile("ld.volatile.shared.v2.b32 {%0, %1}, [%2];" : "=r"(tg), "=r"(bits) : "r"(theirs) : "memory");
    if (tg == tag) {
      *got = __uint_as_float(bits);
      return true;
    }
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

// Shared-memory operand descriptors, 128-byte swizzle, rows of 128 bytes, 8-row groups 1024 bytes apart.
// K-major: the contraction runs along a row (Q, K and P tiles).
__device__ __forceinline__ uint64_t desc_k_major(uint32_t addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr & 0x3ffff) >> 4);
  d |= static_cast<uint64_t>(1) << 16;                   // leading byte offset: unused with a swizzled K-major tile
  d |= static_cast<uint64_t>(1024 >> 4) << 32;           // stride byte offset: next 8 rows
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
// MN-major: a row holds 64 consecutive columns of the N side (dims of V), the contraction runs down the rows
// (keys).  Leading byte offset = distance to the next 64 columns (the other half of the head dimension), stride byte
// offset = distance to the next 8 rows.
__device__ __forceinline__ uint64_t desc_mn_major(uint32_t addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr & 0x3ffff) >> 4);
  d |= static_cast<uint64_t>(kSub >> 4) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 consecutive fp32 columns of this warp's 32 tensor-memory lanes (thread = lane)
__device__ __forceinline__ void tmem_ld32(uint32_t addr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(addr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void tmem_st32(uint32_t addr, const float (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(addr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
        "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
        "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
        "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
        "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
        "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
        "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(320, 1) attn_tc_kernel(AttnArgs a, const __grid_constant__ CUtensorMap map_k,
                                                         const __grid_constant__ CUtensorMap map_v) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t bars = base + kOffBar;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kOffBar + 8 * B_COUNT);
  __shared__ int s_abort_mem;
  volatile int* s_abort = &s_abort_mem;
  auto bar = [&](int idx) { return bars + 8u * static_cast<uint32_t>(idx); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const LaunchStamp stamp{a.stamp.begin, a.stamp.end};
  stamp_begin(stamp);
  pdl_launch_dependents();

  const int4 item = a.items[blockIdx.x];
  const int req = item.x, kvh = item.y, key_start = item.z, key_count = item.w;
  const int key_end = key_start + key_count;
  const int n_tiles = (key_count + kTile - 1) / kTile;
  const int group = a.Hq / a.Hkv;
  const int row0 = a.cu_q[req];
  const int n_rows = (a.cu_q[req + 1] - row0) * group;      // <= 128 (the caller's condition for this kernel)
  const int kv_base = a.kv_base[req];
  const bool split = a.req_chunks[req] > 1;
  const int chunk_idx = key_start / a.req_chunk_keys[req];
  const float scale = rsqrtf(static_cast<float>(kH)) * 1.4426950408889634f;   // scores in log2 units

  for (int i = threadIdx.x; i < 3 * kRows * 2 * 2; i += blockDim.x)      // exchange slots: no tag set
    reinterpret_cast<uint32_t*>(base_ptr + kOffX)[i] = 0u;
  if (threadIdx.x == 0) {
    *s_abort = 0;
    for (int s = 0; s < kStages; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(B_FULL + s)), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(B_EMPTY + s)), "r"(1));
    }
    for (int b = 0; b < 2; ++b) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(B_SFULL + b)), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(B_SEMPTY + b)), "r"(kSoftmaxWarps));   // one arrival per softmax warp
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(B_PFULL + b)), "r"(kSoftmaxWarps));
    }
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(B_ODONE)), "r"(1));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(B_QFULL)), "r"(kSoftmaxWarps));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_k)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_v)) : "memory");
  }
  if (warp == 9) {   // tensor memory: S 2 x 64 columns, O 128 columns -> 256
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))),
                 "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + 128u;   // column offsets

  if (warp == 8) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      const int32_t* pages = a.page_table + a.pt_off[req];
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      auto load_tile = [&](int tile, int s) {
        const uint32_t full = bar(B_FULL + s);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full), "r"(kStageBytes) : "memory");
        const uint32_t dst = base + s * kStageBytes;
#pragma unroll
        for (int p = 0; p < 4; ++p) {
          int kk = key_start + tile * kTile + p * 16;
          if (kk >= key_end) kk = key_end - 1;              // past the chunk: re-read a valid page (masked later)
          const int row = (pages[kk >> 4] * a.Hkv + kvh) * 16;
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            tma_load_2d(dst + hh * kSub + p * 2048, &map_k, hh * 64, row, full, policy);
            tma_load_2d(dst + kKBytes + hh * kSub + p * 2048, &map_v, hh * 64, row, full, policy);
          }
        }
      };
      // tiles wholly inside the cached prefix do not depend on the preceding kernel: requested before the wait
      const int safe_tiles = key_end <= kv_base ? n_tiles : max(0, kv_base - key_start) / kTile;
      const int pre = min(min(kStages, n_tiles), safe_tiles);
      for (int tile = 0; tile < pre; ++tile) load_tile(tile, tile);
      pdl_wait();
      for (int tile = pre; tile < n_tiles; ++tile) {
        const int s = tile % kStages;
        if (*s_abort || !mbar_wait(bar(B_EMPTY + s), ((tile / kStages) & 1) ^ 1, s_abort)) { *s_abort = 1; break; }
        load_tile(tile, s);
      }
    } else {
      pdl_wait();
      if (lane == 1 && *reinterpret_cast<volatile int32_t*>(a.error) != 0) *s_abort = 1;   // an earlier kernel gave up
    }
  } else if (warp == 9) {
    // ---------------------------------------------------------------- MMA issue
    pdl_wait();
    if (lane == 0) {
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kTile >> 3) << 17) |
                               (static_cast<uint32_t>(kRows >> 4) << 24);                       // N = 64, both K-major
      const uint32_t idesc_pv = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (static_cast<uint32_t>(kH >> 3) << 17) |
                                (static_cast<uint32_t>(kRows >> 4) << 24);                      // N = 128, B MN-major
      bool ok = mbar_wait(bar(B_QFULL), 0, s_abort);
      auto issue_s = [&](int t) {
        const int s = t % kStages, b = t & 1;
        if (!mbar_wait(bar(B_FULL + s), (t / kStages) & 1, s_abort)) return false;
        if (!mbar_wait(bar(B_SEMPTY + b), ((t >> 1) & 1) ^ 1, s_abort)) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t kbase = base + s * kStageBytes;
#pragma unroll
        for (int ks = 0; ks < kH / 16; ++ks) {
          const uint64_t ad = desc_k_major(base + kOffQ + (ks >> 2) * (kRows * 128) + (ks & 3) * 32);
          const uint64_t bd = desc_k_major(kbase + (ks >> 2) * kSub + (ks & 3) * 32);
          umma(tmem_s + static_cast<uint32_t>(b * kTile), ad, bd, idesc_s, ks != 0 ? 1u : 0u);
        }
        umma_commit(bar(B_SFULL + b));
        return true;
      };
      auto issue_pv = [&](int t) {
        const int s = t % kStages, b = t & 1;
        if (!mbar_wait(bar(B_PFULL + b), (t >> 1) & 1, s_abort)) return false;   // P written, O rescaled if it had to be
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t vbase = base + s * kStageBytes + kKBytes;
#pragma unroll
        for (int kt = 0; kt < kTile / 16; ++kt) {
          const uint64_t ad = desc_k_major(base + kOffP + b * kPBytes + kt * 32);
          const uint64_t bd = desc_mn_major(vbase + kt * 2048);      // 16 keys further down: 16 rows of 128 bytes
          umma(tmem_o, ad, bd, idesc_pv, (t | kt) != 0 ? 1u : 0u);   // O accumulates over all tiles of the item
        }
        umma_commit(bar(B_ODONE));          // phase t: the products of tiles 0..t are in O
        umma_commit(bar(B_EMPTY + s));      // both products of this tile have read the stage
        return true;
      };
      if (ok) ok = issue_s(0);
      for (int t = 0; ok && t < n_tiles; ++t) {
        if (t + 1 < n_tiles) ok = issue_s(t + 1);    // the next tile's scores run under this tile's softmax
        if (ok) ok = issue_pv(t);
      }
      if (!ok) *s_abort = 1;
    }
  } else {
    // ---------------------------------------------------------------- softmax + output
    // quarter = warp % 4 owns tensor-memory lanes 32 quarter .. +31; lane i of it holds query row 4 i + quarter;
    // the two warps of a quarter take keys 0-31 / 32-63 of every tile and columns 0-63 / 64-127 of the output
    pdl_wait();
    const int quarter = warp & 3, half = warp >> 2;
    const int rho = quarter * 32 + lane;                       // row index in shared and tensor memory
    const int r = 4 * lane + quarter;                          // query row of the item
    const bool valid = r < n_rows;
    const int j = valid ? r / group : 0;
    const int head = kvh * group + (valid ? r % group : 0);
    const int vis = kv_base + j;                               // last key index this row may see
    const uint32_t tlane = static_cast<uint32_t>(quarter * 32) << 16;
    auto xslot = [&](int slot, int h) { return base + kOffX + static_cast<uint32_t>(((slot * kRows + rho) * 2 + h) * 8); };
    {
      // this row of Q into shared memory in the operand layout (zero for rows beyond the item's): each of the
      // row's two threads writes one half of the head dimension
      const uint4* src = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(a.q) +
                                                        (static_cast<int64_t>(row0 + j) * a.Hq + head) * kH + half * 64);
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint4 v = valid ? src[c] : make_uint4(0u, 0u, 0u, 0u);
        const uint32_t dst = base + kOffQ + half * (kRows * 128) + rho * 128 + ((c ^ (rho & 7)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_QFULL));
    }
    float m = -INFINITY, l = 0.f;     // reference maximum of the row (same in both of its threads), this half's share of the sum
    bool ok = true;

    for (int t = 0; t < n_tiles; ++t) {
      const int b = t & 1;
      // (every give-up decision below is taken by the whole warp: the warp-wide instructions that follow need all lanes)
      if (!__all_sync(0xffffffffu, *s_abort == 0 && mbar_wait(bar(B_SFULL + b), (t >> 1) & 1, s_abort))) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      float sc[32];
      tmem_ld32(tmem_s + tlane + static_cast<uint32_t>(b * kTile + half * 32), sc);
      // S has been read: the next-but-one tile's scores may overwrite it
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_SEMPTY + b));

      const int k0 = key_start + t * kTile + half * 32;
      const bool need_mask = (k0 + 31 > kv_base) || (k0 + 32 > key_end);
      float mx = -INFINITY;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        float v = sc[i] * scale;
        if (need_mask && (k0 + i > vis || k0 + i >= key_end)) v = -INFINITY;
        sc[i] = v;
        mx = fmaxf(mx, v);
      }
      // the row's maximum over both halves
      float other = -INFINITY;
      if (!__all_sync(0xffffffffu, swap_with_partner(xslot(b, half), xslot(b, half ^ 1), static_cast<uint32_t>(t + 1), mx, &other, s_abort))) {
        ok = false;
        break;
      }
      mx = fmaxf(mx, other);
      // raise the reference only when it is exceeded by a wide margin (or not set yet)
      float alpha = 1.f;
      const bool raise = mx > m + kRaiseBy || (m == -INFINITY && mx != -INFINITY);
      if (raise) {
        alpha = exp2f(m - mx);      // 0 when nothing had been seen before
        m = mx;
      }
      const float ms = m == -INFINITY ? 0.f : m;
      float sum = 0.f;
      uint32_t pk[16];
#pragma unroll
      for (int i = 0; i < 32; i += 2) {
        const float p0 = exp2f(sc[i] - ms), p1 = exp2f(sc[i + 1] - ms);
        sum += p0 + p1;
        pk[i >> 1] = pack_bf16(p0, p1);
      }
      l = fmaf(l, alpha, sum);
      // P buffer b is free: the product that read it (tile t-2) completed before the scores of tile t did
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const uint32_t dst = base + kOffP + b * kPBytes + rho * 128 + (((half * 4 + c) ^ (rho & 7)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pk[4 * c]), "r"(pk[4 * c + 1]),
                     "r"(pk[4 * c + 2]), "r"(pk[4 * c + 3]) : "memory");
      }
      // The previous tile's product must be in O before this tile's may be added; waiting for it in every tile
      // (it was issued a whole softmax ago: normally long complete) also keeps this warp within one phase of the
      // barrier, which a parity wait needs.  If some row of this warp raised its reference, its part of O (this
      // thread's 64 columns) is brought to the new scale first.
      if (t > 0 && !__all_sync(0xffffffffu, mbar_wait(bar(B_ODONE), (t - 1) & 1, s_abort))) { ok = false; break; }
      if (t > 0 && __any_sync(0xffffffffu, raise)) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          float v[32];
          const uint32_t addr = tmem_o + tlane + static_cast<uint32_t>(half * 64 + c * 32);
          tmem_ld32(addr, v);
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] *= alpha;
          tmem_st32(addr, v);
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_PFULL + b));
    }
    // ---- the item's result: O is complete once the last product is
    if (ok && n_tiles > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar(B_ODONE), (n_tiles - 1) & 1, s_abort));
    if (!ok) *s_abort = 1;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // the row's sum = the two halves' shares
    if (ok) {
      float other = 0.f;
      ok = __all_sync(0xffffffffu, swap_with_partner(xslot(2, half), xslot(2, half ^ 1), 0x7fffffffu, l, &other, s_abort));
      l += other;
      if (!ok) *s_abort = 1;
    }
    if (ok) {
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        float v[32];
        tmem_ld32(tmem_o + tlane + static_cast<uint32_t>(half * 64 + c * 32), v);
        if (!valid) continue;
        const int col = half * 64 + c * 32;
        if (!split) {
          const float inv = 1.f / l;
          uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(a.out) + (static_cast<int64_t>(row0 + j) * a.Hq + head) * kH + col);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4)
            dst[q4] = make_uint4(pack_bf16(v[8 * q4] * inv, v[8 * q4 + 1] * inv), pack_bf16(v[8 * q4 + 2] * inv, v[8 * q4 + 3] * inv),
                                 pack_bf16(v[8 * q4 + 4] * inv, v[8 * q4 + 5] * inv), pack_bf16(v[8 * q4 + 6] * inv, v[8 * q4 + 7] * inv));
        } else {
          const int64_t prow = static_cast<int64_t>(a.tok_part[row0 + j] + chunk_idx) * a.Hq + head;
          float4* dst = reinterpret_cast<float4*>(a.part_acc + prow * kH + col);
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4) dst[q4] = make_float4(v[4 * q4], v[4 * q4 + 1], v[4 * q4 + 2], v[4 * q4 + 3]);
          if (c == 0 && half == 0) {
            a.part_ml[prow * 2] = m;
            a.part_ml[prow * 2 + 1] = l;
          }
        }
      }
    }
  }

  // teardown
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (*s_abort) {
    if (threadIdx.x == 0) atomicCAS(a.error, 0, 8);
    // copies and products that were issued may still land: wait a little before the memory goes away
    const long long t1 = clock64();
    while (clock64() - t1 < 2000000LL) __nanosleep(1000);
  }
  if (warp == 9)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
  stamp_end(stamp);
}

}  // namespace

int launch_attention_tc(const AttnArgs& a, cudaStream_t s) {
  if (!a.map_k || !a.map_v || !a.error || a.page_size != 16 || a.h != kH) return -1;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return -1;
    configured = true;
  }
  SLED_LAUNCH_PDL(attn_tc_kernel, dim3(a.n_items), dim3(320), kSmemBytes, s, a, *a.map_k, *a.map_v);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace sled
