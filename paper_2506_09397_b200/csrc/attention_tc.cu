// Ragged verification attention on the 5th-generation tensor cores (tcgen05), for head_dim 128, bf16 cache,
// 16-token pages and work items of at most 48 query rows (a verification request: (k+1) tokens x 4 heads per KV head).
// Selected by sled_config.attention_impl = 1; the warp-level kernel (attention_mma.cu) is the default because it is
// faster on the measured workloads (this kernel's per-tile chain is walked by one warp per SM sub-partition).
//
// A work item is (request, KV head, chunk of keys).  The few query rows sit on the N side of the MMAs and the KEYS on
// the M side (one key per tensor-memory lane), so that the softmax work is proportional to the number of query rows
// instead of to a 128-row tile that is mostly padding.  Per 128-key tile:
//     S^T = K Q^T   (M 128 keys x N 48 rows,  K = 128 dims:  8 instructions of K 16)   -> tensor memory, fp32
//     O^T += V^T P^T (M 128 dims x N 48 rows, K = 128 keys:  8 instructions of K 16)   -> tensor memory, fp32
// K and V pages arrive by TMA exactly as the cache stores them, [16 tokens][128 dims] per (page, KV head), as
// 128-byte swizzled rows of 64 dims.  K is the K-major A operand of the first product; the same kind of tile of V is
// the MN-major A operand of the second (its rows are keys: the contraction runs down the rows), so nothing is
// transposed or copied.  Four softmax warps own one key per thread: a thread reads its key's 48 scores from tensor
// memory, masks, exponentiates, adds to per-thread partial row sums (reduced over the keys only once, at the end of
// the item) and writes its row of P^T - 48 bf16 values - into shared memory as the MN-major B operand.  The
// reference maximum of a query row is shared by all keys; it is raised only when some score exceeds it by more than
// 8 (log2 units: harmless for bf16 probabilities and fp32 sums, and it cancels in the final division), which the
// warps find out by a vote per tile; raising means rescaling that row's column of O^T in tensor memory and happens
// in an item's first tiles only.  S^T is double-buffered: the scores of tile t+1 are computed under the softmax of
// tile t.
//   warps 0-3 : softmax + output (thread = key of the tile = tensor-memory lane; in the output, thread = dim)
//   warp 4    : TMA producer (one thread), 3 stages of 64 KB
//   warp 5    : tensor-memory allocation, MMA issue (one thread)
// Every wait is bounded; when one runs out the block records a code in *error, lets copies in flight land, frees its
// tensor memory and returns.  Warps hand values to each other through tagged slots in shared memory with bounded
// polling, never through named barriers, so a warp that has given up cannot strand the others.
#include <cuda_bf16.h>

#include "common.cuh"
#include "kernels.h"

namespace sled {

namespace {

constexpr int kTile = 128;                  // keys per tile
constexpr int kStages = 3;                  // 192 KB of cache in the ring: two tiles in flight while one is consumed
constexpr int kH = 128;                     // head_dim
constexpr int kNR = 48;                     // query rows of an item, padded (MMA N)
constexpr int kHalfBytes = kTile * 128;     // one [128 keys][64 dims] sub-tile of 128-byte rows: 16 KB
constexpr int kKBytes = 2 * kHalfBytes;     // K part of a stage (two halves of the head dimension)
constexpr int kStageBytes = 2 * kKBytes;    // K and V: 64 KB
constexpr int kQHalf = kNR * 128;           // Q: [2 halves][48 rows][64 dims]
constexpr int kPBytes = kTile * 128;        // P^T: [128 keys][64 rows (48 used)]
constexpr int kOffQ = kStages * kStageBytes;
constexpr int kOffP = kOffQ + 2 * kQHalf;
constexpr int kOffX = kOffP + kPBytes;      // exchange area: flags [2][4] x 8 B; row maxima [4 warps][48] + 4 tags; row sums likewise; factors [48]
constexpr int kXFlags = 0, kXMax = 64, kXMaxTags = kXMax + 4 * kNR * 4, kXSum = kXMaxTags + 32, kXSumTags = kXSum + 4 * kNR * 4,
              kXAlpha = kXSumTags + 32;
constexpr int kXBytes = 3072;
static_assert(kXAlpha + 4 * 4 * kNR <= kXBytes, "exchange area");
static_assert(kOffX + kXBytes + 256 + 1024 <= 227 * 1024, "shared memory of one block");
constexpr int kOffBar = kOffX + kXBytes;
constexpr int kSmemBytes = kOffBar + 256 + 1024;   // barriers and the tensor-memory slot, plus alignment slack
constexpr long long kWaitCycles = 200000000LL;
constexpr float kRaiseBy = 8.f;             // a row's reference maximum is raised only by more than this (log2 units)

// barrier indices (8 bytes each from kOffBar)
enum { B_FULL = 0, B_EMPTY = B_FULL + kStages, B_SFULL = B_EMPTY + kStages, B_SEMPTY = B_SFULL + 2, B_PFULL = B_SEMPTY + 2,
       B_ODONE = B_PFULL + 1, B_QFULL = B_ODONE + 1, B_COUNT = B_QFULL + 1 };

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
// the same for the two single-thread roles (copy issue, MMA issue): they share their schedulers with softmax warps,
// so they sleep between polls instead of competing for issue slots
__device__ __forceinline__ bool mbar_wait_idle(uint32_t bar, uint32_t parity, volatile int* stop) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    __nanosleep(40);
    if (mbar_try_wait(bar, parity)) return true;
    if (*stop != 0 || clock64() - t0 > kWaitCycles) return false;
  }
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y), "l"(policy)
      : "memory");
}

// Shared-memory operand descriptors, 128-byte swizzle, rows of 128 bytes, 8-row groups 1024 bytes apart.
// K-major: the contraction runs along a row (the K tile, Q).
__device__ __forceinline__ uint64_t desc_k_major(uint32_t addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr & 0x3ffff) >> 4);
  d |= static_cast<uint64_t>(1) << 16;                   // leading byte offset: unused with a swizzled K-major tile
  d |= static_cast<uint64_t>(1024 >> 4) << 32;           // stride byte offset: next 8 rows
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

// MN-major: a row holds 64 consecutive elements of the M or N side (dims of V, query rows of P^T), the contraction
// runs down the rows (keys).  Leading byte offset = distance to the next 64 elements of that side, stride byte offset
// = distance to the next 8 rows.
__device__ __forceinline__ uint64_t desc_mn_major(uint32_t addr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr & 0x3ffff) >> 4);
  d |= static_cast<uint64_t>(lbo_bytes >> 4) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

// 16 consecutive fp32 columns of this warp's 32 tensor-memory lanes (thread = lane); the values may be used after
// tmem_ld_wait()
__device__ __forceinline__ void tmem_ld16_nowait(uint32_t addr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(addr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16(uint32_t addr, float* v) {
  uint32_t r[16];
  tmem_ld16_nowait(addr, r);
  tmem_ld_wait();
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st16(uint32_t addr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(addr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
        "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
        "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15]))
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// The four softmax warps tell each other something once per tile: lane 0 of a warp stores (tag, word) into the
// warp's slot and polls the other slots until they carry the same tag.  Bounded like every other wait.
__device__ __forceinline__ bool post_and_collect(uint32_t slots, int warp, uint32_t tag, uint32_t word, uint32_t* any_of_four,
                                                 volatile int* stop) {
  asm volatile("st.volatile.shared.v2.b32 [%0], {%1, %2};" ::"r"(slots + 8u * warp), "r"(tag), "r"(word) : "memory");
  uint32_t acc = word;
  const long long t0 = clock64();
  for (int w = 0; w < 4; ++w) {
    if (w == warp) continue;
    for (;;) {
      uint32_t tg, val;
      asm volatile("ld.volatile.shared.v2.b32 {%0, %1}, [%2];" : "=r"(tg), "=r"(val) : "r"(slots + 8u * w) : "memory");
      if (tg == tag) { acc |= val; break; }
      if (*stop != 0 || clock64() - t0 > kWaitCycles) return false;
    }
  }
  *any_of_four = acc;
  return true;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(192, 1) attn_tc_kernel(AttnArgs a, const __grid_constant__ CUtensorMap map_k,
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
  const int n_rows = (a.cu_q[req + 1] - row0) * group;      // <= 48 (the caller's condition for this kernel)
  const int kv_base = a.kv_base[req];
  const bool split = a.req_chunks[req] > 1;
  const int chunk_idx = key_start / a.req_chunk_keys[req];
  const float scale = rsqrtf(static_cast<float>(kH)) * 1.4426950408889634f;   // scores in log2 units

  for (int i = threadIdx.x; i < kXBytes / 4; i += blockDim.x)      // exchange area: no tag set
    reinterpret_cast<uint32_t*>(base_ptr + kOffX)[i] = 0u;
  if (threadIdx.x == 0) {
    *s_abort = 0;
    for (int s = 0; s < kStages; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(B_FULL + s)), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(B_EMPTY + s)), "r"(1));
    }
    for (int b = 0; b < 2; ++b) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(B_SFULL + b)), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(B_SEMPTY + b)), "r"(4));   // one arrival per softmax warp
    }
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(B_PFULL)), "r"(4));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(B_ODONE)), "r"(1));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar(B_QFULL)), "r"(4));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_k)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_v)) : "memory");
  }
  if (warp == 5) {   // tensor memory: S^T 2 x 48 columns (at 0 and 64), O^T 48 columns (at 128) -> 256 (a power of two)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))),
                 "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + 128u;   // column offsets

  if (warp == 4) {
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
        for (int p = 0; p < kTile / 16; ++p) {
          int kk = key_start + tile * kTile + p * 16;
          if (kk >= key_end) kk = key_end - 1;              // past the chunk: re-read a valid page (masked later)
          const int row = (pages[kk >> 4] * a.Hkv + kvh) * 16;
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            tma_load_2d(dst + hh * kHalfBytes + p * 2048, &map_k, hh * 64, row, full, policy);
            tma_load_2d(dst + kKBytes + hh * kHalfBytes + p * 2048, &map_v, hh * 64, row, full, policy);
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
        if (*s_abort || !mbar_wait_idle(bar(B_EMPTY + s), ((tile / kStages) & 1) ^ 1, s_abort)) { *s_abort = 1; break; }
        load_tile(tile, s);
      }
    } else {
      pdl_wait();
      if (lane == 1 && *reinterpret_cast<volatile int32_t*>(a.error) != 0) *s_abort = 1;   // an earlier kernel gave up
    }
  } else if (warp == 5) {
    // ---------------------------------------------------------------- MMA issue
    pdl_wait();
    if (lane == 0) {
      // fp32 accumulate, bf16 x bf16, N = 48, M = 128; second product: both operands MN-major
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kNR >> 3) << 17) |
                               (static_cast<uint32_t>(128 >> 4) << 24);
      const uint32_t idesc_pv = idesc_s | (1u << 15) | (1u << 16);
      bool ok = mbar_wait_idle(bar(B_QFULL), 0, s_abort);
      auto issue_s = [&](int t) {
        const int s = t % kStages, b = t & 1;
        if (!mbar_wait_idle(bar(B_FULL + s), (t / kStages) & 1, s_abort)) return false;
        if (!mbar_wait_idle(bar(B_SEMPTY + b), ((t >> 1) & 1) ^ 1, s_abort)) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t kbase = base + s * kStageBytes;
#pragma unroll
        for (int ks = 0; ks < kH / 16; ++ks) {
          const uint64_t ad = desc_k_major(kbase + (ks >> 2) * kHalfBytes + (ks & 3) * 32);            // keys x dims
          const uint64_t bd = desc_k_major(base + kOffQ + (ks >> 2) * kQHalf + (ks & 3) * 32);         // query rows x dims
          umma(tmem_s + static_cast<uint32_t>(b * 64), ad, bd, idesc_s, ks != 0 ? 1u : 0u);
        }
        umma_commit(bar(B_SFULL + b));
        return true;
      };
      auto issue_pv = [&](int t) {
        const int s = t % kStages;
        if (!mbar_wait_idle(bar(B_PFULL), t & 1, s_abort)) return false;   // P^T written, O^T rescaled if it had to be
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t vbase = base + s * kStageBytes + kKBytes;
#pragma unroll
        for (int kt = 0; kt < kTile / 16; ++kt) {      // 16 keys further down per step: 16 rows of 128 bytes
          const uint64_t ad = desc_mn_major(vbase + kt * 2048, kHalfBytes);                    // V^T: dims x keys
          const uint64_t bd = desc_mn_major(base + kOffP + kt * 2048, 16);                     // P^T: keys x query rows
          umma(tmem_o, ad, bd, idesc_pv, (t | kt) != 0 ? 1u : 0u);   // O^T accumulates over all tiles of the item
        }
        umma_commit(bar(B_ODONE));          // phase t: the products of tiles 0..t are in O^T, P^T may be overwritten
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
    // ---------------------------------------------------------------- softmax + output: thread = key of the tile
    pdl_wait();
    const int lam = threadIdx.x;                               // 0..127: tensor-memory lane, row of P^T, later the dim
    const uint32_t tlane = static_cast<uint32_t>(warp * 32) << 16;
    const uint32_t xbase = base + kOffX;
    {
      // Q into shared memory in the operand layout: [2 halves][48 rows][64 dims], rows beyond the item's are zero
      const __nv_bfloat16* qbuf = static_cast<const __nv_bfloat16*>(a.q);
      for (int idx = lam; idx < kNR * 16; idx += 128) {
        const int n = idx >> 4, cc = idx & 15, hh = cc >> 3, c = cc & 7;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (n < n_rows) {
          const int jn = n / group, head = kvh * group + n % group;
          v = *reinterpret_cast<const uint4*>(qbuf + (static_cast<int64_t>(row0 + jn) * a.Hq + head) * kH + hh * 64 + c * 8);
        }
        const uint32_t dst = base + kOffQ + hh * kQHalf + n * 128 + ((c ^ (n & 7)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_QFULL));
    }
    float m[kNR], l[kNR];        // per query row: reference maximum (the same in all threads), this key slot's share of the sum
#pragma unroll
    for (int n = 0; n < kNR; ++n) { m[n] = -INFINITY; l[n] = 0.f; }
    bool ok = true;

    for (int t = 0; t < n_tiles; ++t) {
      const int b = t & 1;
      // (every give-up decision is taken by the whole warp: the warp-wide instructions that follow need all lanes)
      if (!__all_sync(0xffffffffu, *s_abort == 0 && mbar_wait(bar(B_SFULL + b), (t >> 1) & 1, s_abort))) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      float sc[kNR];
      {
        uint32_t raw[kNR];
#pragma unroll
        for (int c = 0; c < kNR / 16; ++c) tmem_ld16_nowait(tmem_s + tlane + static_cast<uint32_t>(b * 64 + c * 16), raw + 16 * c);
        tmem_ld_wait();
#pragma unroll
        for (int n = 0; n < kNR; ++n) sc[n] = __uint_as_float(raw[n]);
      }
      // S^T has been read: the next-but-one tile's scores may overwrite it
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_SEMPTY + b));

      // query row n (token n / group of the request) sees keys up to kv_base + n / group:
      //   kk <= kv_base + n / group   <=>   (kk - kv_base) * group <= n
      const int kk = key_start + t * kTile + lam;
      const bool key_ok = kk < key_end;
      const int thr = (kk - kv_base) * group;
      bool exceed = false;
#pragma unroll
      for (int n = 0; n < kNR; ++n) {
        float v = sc[n] * scale;
        if (!key_ok || thr > n) v = -INFINITY;
        sc[n] = v;
        exceed |= v > m[n] + kRaiseBy;      // also true for the first finite score of a row (m = -inf)
      }
      // does any key of the tile exceed a row's reference by the margin?  One word per warp, all four collected.
      uint32_t any4 = 0;
      {
        const uint32_t mine = __any_sync(0xffffffffu, exceed) ? 1u : 0u;
        bool got = true;
        if (lane == 0) got = post_and_collect(xbase + kXFlags + 32u * b, warp, static_cast<uint32_t>(t + 1), mine, &any4, s_abort);
        any4 = __shfl_sync(0xffffffffu, any4, 0);
        if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
      }
      if (any4) {
        // ---- rare: raise the references.  Row maxima over this warp's keys, then over the four warps.
        volatile float* xv = reinterpret_cast<volatile float*>(base_ptr + kOffX + kXMax);
        volatile float* xa = reinterpret_cast<volatile float*>(base_ptr + kOffX + kXAlpha) + warp * kNR;   // this warp's copy
#pragma unroll
        for (int n = 0; n < kNR; ++n) {
          float v = sc[n];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
          if (lane == 0) xv[warp * kNR + n] = v;
        }
        if (lane == 0) __threadfence_block();      // the values before the tag
        __syncwarp();
        uint32_t dummy = 0;
        bool got = true;
        if (lane == 0) got = post_and_collect(xbase + kXMaxTags, warp, 0x40000000u + static_cast<uint32_t>(t), 0u, &dummy, s_abort);
        if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
        __threadfence_block();
#pragma unroll
        for (int n = 0; n < kNR; ++n) {
          const float cm = fmaxf(fmaxf(xv[n], xv[kNR + n]), fmaxf(xv[2 * kNR + n], xv[3 * kNR + n]));
          const float m_new = cm > m[n] + kRaiseBy ? cm : m[n];
          const float al = m_new == m[n] ? 1.f : exp2f(m[n] - m_new);      // 0 when nothing had been seen before
          l[n] *= al;
          m[n] = m_new;
          if (lane == 0) xa[n] = al;
        }
        __syncwarp();
        if (t > 0) {
          // bring O^T (this warp's 32 dims, all query rows) to the new scale; the previous product is complete
          // (waited for below in every tile before P^T is overwritten - here it is needed a little earlier)
          if (!__all_sync(0xffffffffu, mbar_wait(bar(B_ODONE), (t - 1) & 1, s_abort))) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
          for (int c = 0; c < kNR / 16; ++c) {
            float v[16];
            const uint32_t addr = tmem_o + tlane + static_cast<uint32_t>(c * 16);
            tmem_ld16(addr, v);
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] *= xa[16 * c + i];
            tmem_st16(addr, v);
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        }
      }
      // ---- probabilities of this key for every query row
      uint32_t pk[kNR / 2];
#pragma unroll
      for (int n = 0; n < kNR; n += 2) {
        const float p0 = exp2f(sc[n] - (m[n] == -INFINITY ? 0.f : m[n]));
        const float p1 = exp2f(sc[n + 1] - (m[n + 1] == -INFINITY ? 0.f : m[n + 1]));
        l[n] += p0;
        l[n + 1] += p1;
        pk[n >> 1] = pack_bf16(p0, p1);
      }
      // P^T was read by the product of the previous tile: wait for it (waiting in every tile also keeps the warp
      // within one phase of the barrier, which a parity wait needs)
      if (t >= 1 && !__all_sync(0xffffffffu, mbar_wait(bar(B_ODONE), (t - 1) & 1, s_abort))) { ok = false; break; }
#pragma unroll
      for (int c = 0; c < kNR / 8; ++c) {
        const uint32_t dst = base + kOffP + lam * 128 + ((c ^ (lam & 7)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pk[4 * c]), "r"(pk[4 * c + 1]),
                     "r"(pk[4 * c + 2]), "r"(pk[4 * c + 3]) : "memory");
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_PFULL));
    }

    // ---- the item's result: O^T is complete once the last product is
    if (ok && n_tiles >= 1) ok = __all_sync(0xffffffffu, mbar_wait(bar(B_ODONE), (n_tiles - 1) & 1, s_abort));
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ok) {
      // row sums: over this warp's keys by shuffles, over the four warps through shared memory
#pragma unroll
      for (int n = 0; n < kNR; ++n) {
        float v = l[n];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        l[n] = v;
      }
      volatile float* xv = reinterpret_cast<volatile float*>(base_ptr + kOffX + kXSum);
      if (lane == 0) {
#pragma unroll
        for (int n = 0; n < kNR; ++n) xv[warp * kNR + n] = l[n];
        __threadfence_block();        // the values before the tag
      }
      __syncwarp();
      uint32_t dummy = 0;
      bool got = true;
      if (lane == 0) got = post_and_collect(xbase + kXSumTags, warp, 0x7fffffffu, 0u, &dummy, s_abort);
      ok = __all_sync(0xffffffffu, got);
      __threadfence_block();
      if (ok) {
#pragma unroll
        for (int n = 0; n < kNR; ++n) l[n] = (xv[n] + xv[kNR + n]) + (xv[2 * kNR + n] + xv[3 * kNR + n]);
      }
    }
    if (!ok) *s_abort = 1;
    if (ok) {
      // thread = dim now: this lane's element of every query row's output
      int jn = 0, g = 0;      // token and head-in-group of row n
#pragma unroll
      for (int c = 0; c < kNR / 16; ++c) {
        float v[16];
        tmem_ld16(tmem_o + tlane + static_cast<uint32_t>(c * 16), v);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int n = 16 * c + i;
          if (n < n_rows) {
            const int head = kvh * group + g;
            if (!split) {
              static_cast<__nv_bfloat16*>(a.out)[(static_cast<int64_t>(row0 + jn) * a.Hq + head) * kH + lam] =
                  __float2bfloat16_rn(v[i] / l[n]);
            } else {
              const int64_t prow = static_cast<int64_t>(a.tok_part[row0 + jn] + chunk_idx) * a.Hq + head;
              a.part_acc[prow * kH + lam] = v[i];
              if (lam == 0) {
                a.part_ml[prow * 2] = m[n];
                a.part_ml[prow * 2 + 1] = l[n];
              }
            }
          }
          if (++g == group) { g = 0; ++jn; }
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
  if (warp == 5)
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
  SLED_LAUNCH_PDL(attn_tc_kernel, dim3(a.n_items), dim3(192), kSmemBytes, s, a, *a.map_k, *a.map_v);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace sled
