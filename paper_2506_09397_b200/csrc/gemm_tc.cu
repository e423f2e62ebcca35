// bf16 linear layers on the 5th-generation tensor cores (sm_100a).
//
// One CTA computes a 128 (weight rows, the MMA M side) x TN (tokens, the N side) tile over one K slice;
// the real token extent round_up(T,16) is a run-time field of the instruction descriptor, so nothing is
// padded to a fixed tile.  Two CTAs fit on an SM; the number of K slices is chosen so that all CTAs of a
// launch are resident at once with equal work (weight-streaming regime: they share HBM evenly and end
// together); with many tiles the hardware scheduler hands them out as CTAs retire.  Token tiles of one
// weight tile are neighbours in the grid, so the second reader of a weight slab finds it in L2.
//   warp 0   : TMA producer - 64-wide K slabs of W (evict-first: read once per step) and of the activations
//              (evict-last: re-read by every tile) into a ring of 128-byte-swizzled stages.  Weights do not
//              depend on the previous kernel: the ring is filled with weight slabs before the
//              programmatic-launch dependency wait, the activation slabs follow after it
//   warp 1   : allocates tensor memory, issues tcgen05.mma (M=128, N=tn, K=16) four per slab and commits
//              each stage back to the producer, the finished accumulator to the epilogue
//   warps 2-5: epilogue - tcgen05.ld the fp32 accumulator (lane = weight row, column = token) and either
//              store it transposed (32 consecutive outputs of one token per warp store) or apply SwiGLU
// K slices leave partial sums [slice][T][N]; the kernel that consumes the layer's output adds them up in
// slice order while doing its own work (no atomics, no extra pass).
// Every mbarrier wait is bounded: when one runs out the CTA records a code in *error, lets copies in
// flight land, frees its tensor memory and returns.
#include <cuda_bf16.h>

#include <algorithm>
#include <cstdio>

#include "fp8_split.cuh"
#include "gemm_tc.h"

namespace sled {

namespace {

constexpr int kBlockM = 128;          // weight rows per tile (UMMA M)
constexpr int kBlockK = 64;           // bf16 elements per K slab = one 128-byte swizzle row
constexpr int kWStageBytes = kBlockM * kBlockK * 2;
constexpr long long kWaitCycles = 2000000000LL;  // ~1 s at 2 GHz

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// bounded wait: false (and *error = code) when the phase did not complete in time
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int32_t* error, int code, volatile int* stop,
                                          long long limit = kWaitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*stop != 0) return false;            // another warp of this block gave up, or an earlier kernel did
    if (clock64() - t0 > limit) {
      atomicCAS(error, 0, code);
      return false;
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y), "l"(policy)
      : "memory");
}

// shared-memory operand descriptor: K-major tile of 128-byte rows, 128-byte swizzle,
// 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3ffff) >> 4);   // start address / 16
  d |= static_cast<uint64_t>(1) << 16;                      // leading byte offset (unused with swizzle)
  d |= static_cast<uint64_t>(1024 >> 4) << 32;              // stride byte offset between 8-row groups
  d |= static_cast<uint64_t>(1) << 46;                      // descriptor version of this architecture
  d |= static_cast<uint64_t>(2) << 61;                      // 128-byte swizzle
  return d;
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}

__device__ __forceinline__ void pdl_wait_here() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// benchmark mode: earliest block start / latest block end of the launch, in ns of the GPU's global timer
__device__ __forceinline__ void stamp_time(unsigned long long* slot, bool is_end) {
  if (slot == nullptr || threadIdx.x != 0) return;
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  if (is_end) atomicMax(slot, t); else atomicMin(slot, t);
}

__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}


// What the epilogue does with a finished 16-token run of one output row n:
//   kEpiStore : out[t][n] = value
//   kEpiSwiglu: rows come in (gate, up) pairs (2f, 2f+1); act[t][f] = silu(gate) * up as bf16
__device__ __forceinline__ void emit16(const TcEpilogue& e, float* out, int N, int T, int n, int t_first, const float (&val)[16]) {
  if (e.mode == kEpiSwiglu) {
    // lane pairs (gate, up) -> one value per even lane; two neighbouring results are packed so that
    // every fourth lane writes one 4-byte bf16 pair
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float other = __shfl_xor_sync(0xffffffffu, val[i], 1);   // the up value sits in the next lane
      const float gate = val[i];
      const float r = __fdividef(gate, 1.f + __expf(-gate)) * other;
      const float r2 = __shfl_down_sync(0xffffffffu, r, 2);          // result of the next (gate, up) pair
      const int t = t_first + i;
      if ((n & 3) == 0 && n + 3 < N && t < T) {
        __nv_bfloat162 pr = __floats2bfloat162_rn(r, r2);
        *reinterpret_cast<__nv_bfloat162*>(e.act_out + static_cast<long long>(t) * e.act_ld + (n >> 1)) = pr;
      } else if ((n & 3) == 0 && n < N && t < T) {
        e.act_out[static_cast<long long>(t) * e.act_ld + (n >> 1)] = __float2bfloat16_rn(r);
      }
    }
  } else if (n < N) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int t = t_first + i;
      if (t < T) out[static_cast<long long>(t) * N + n] = val[i];
    }
  }
}

template <int TN_MAX, int STAGES>
struct SplitSmemLayout {
  static constexpr int kAStageBytes = TN_MAX * kBlockK * 2;
  static constexpr int kStageBytes = kWStageBytes + kAStageBytes;
  static constexpr int kTiles = STAGES * kStageBytes;
  static constexpr int kTotal = kTiles + 256 /*barriers*/;   // two CTAs per SM: 2 * (kTotal + 1 KB) <= 228 KB
};

template <int TN_MAX, int STAGES>
__global__ void __launch_bounds__(192) tc_gemm_split_kernel(const __grid_constant__ CUtensorMap map_w,
                                                       const __grid_constant__ CUtensorMap map_a, int T, int N,
                                                       int kb_total, int kb_per_split, float* __restrict__ out,
                                                       long long split_stride, int32_t* error, TcEpilogue epi) {
  using L = SplitSmemLayout<TN_MAX, STAGES>;
  constexpr int kTmemCols = TN_MAX <= 32 ? 32 : TN_MAX <= 64 ? 64 : TN_MAX <= 128 ? 128 : 256;   // a power of two
  extern __shared__ __align__(1024) uint8_t smem_raw[];    // swizzled tiles need 1024-byte alignment
  const uint32_t base = smem_u32(smem_raw);
  uint8_t* base_ptr = smem_raw;
  const uint32_t bars = base + L::kTiles;                 // full[STAGES], empty[STAGES], tmem_full, then the tmem address
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + L::kTiles + 8 * (2 * STAGES + 1));
  volatile int* abort_slot = reinterpret_cast<volatile int*>(base_ptr + L::kTiles + 8 * (2 * STAGES + 1) + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  stamp_time(epi.stamp_begin, false);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may start its own prologue
  const int t_tile = blockIdx.x, m_tile = blockIdx.y, split = blockIdx.z;
  const int kb0 = split * kb_per_split;
  const int nkb = min(kb_per_split, kb_total - kb0);
  const int t0 = t_tile * TN_MAX;
  const int tn = min(TN_MAX, ((T - t0) + 15) & ~15);     // token columns of this tile, multiple of 16

  if (threadIdx.x == 0) {
    if (base & 1023u) atomicCAS(error, 0, 5);              // the stage layout below would be wrong: refuse to run
    *abort_slot = (base & 1023u) ? 1 : 0;
  }

  if (warp == 0 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
    for (int s = 0; s < 2 * STAGES + 1; ++s) mbar_init(bars + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // tensor memory for the accumulator tile: TN_MAX fp32 columns x 128 lanes
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))),
                 "r"(static_cast<uint32_t>(kTmemCols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  bool ok = true;
  // An earlier kernel or CTA that gave up has left a code in *error: stop early then.  The word is read by a
  // thread that has nothing to do until the accumulator is complete, so the load's latency delays nobody.
  if (threadIdx.x == 64 && *reinterpret_cast<volatile int32_t*>(error) != 0) *abort_slot = 1;

  if (warp == 0) {
    if (lane == 0 && *abort_slot == 0) {
      uint64_t pol_first, pol_last;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_first));
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_last));
      // The weights do not depend on the previous kernel: fill the ring with weight slabs first, then wait
      // for the predecessor (its output is this kernel's activation operand), then add the activation slabs.
      const int pre = min(STAGES, nkb);
      for (int kb = 0; kb < pre; ++kb) {
        const uint32_t full = bars + 8 * kb;
        mbar_expect_tx(full, L::kStageBytes);
        tma_load_2d(base + kb * L::kStageBytes, &map_w, 0, (m_tile * kb_total + kb0 + kb) * kBlockM, full, pol_first);
      }
      pdl_wait_here();
      for (int kb = 0; kb < pre; ++kb)
        tma_load_2d(base + kb * L::kStageBytes + kWStageBytes, &map_a, (kb0 + kb) * kBlockK, t0, bars + 8 * kb, pol_last);
      for (int kb = pre; kb < nkb; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        if (!mbar_wait(bars + 8 * (STAGES + s), ph ^ 1, error, 1, abort_slot)) { ok = false; break; }
        const uint32_t full = bars + 8 * s;
        mbar_expect_tx(full, L::kStageBytes);
        const uint32_t wdst = base + s * L::kStageBytes;
        tma_load_2d(wdst, &map_w, 0, (m_tile * kb_total + kb0 + kb) * kBlockM, full, pol_first);
        tma_load_2d(wdst + kWStageBytes, &map_a, (kb0 + kb) * kBlockK, t0, full, pol_last);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // instruction descriptor: fp32 accumulate, bf16 x bf16, both operands K-major, N = tn, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(tn >> 3) << 17) |
                             (static_cast<uint32_t>(kBlockM >> 4) << 24);
      for (int kb = 0; kb < nkb; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        if (!mbar_wait(bars + 8 * s, ph, error, 2, abort_slot)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t wsrc = base + s * L::kStageBytes;
        const uint64_t adesc = umma_desc(wsrc), bdesc = umma_desc(wsrc + kWStageBytes);
#pragma unroll
        for (int kk = 0; kk < kBlockK / 16; ++kk)   // 16 bf16 = 32 bytes further along K inside the swizzled row
          umma_bf16(tmem_base, adesc + 2 * kk, bdesc + 2 * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
        umma_commit(bars + 8 * (STAGES + s));       // stage free once these MMAs have read it
      }
      if (ok) umma_commit(bars + 8 * (2 * STAGES)); // accumulator complete
    }
  } else {
    const int quad = warp & 3;                      // a warp may only touch tensor-memory lanes 32*(warp%4)..+31
    if (nkb > 0) ok = mbar_wait(bars + 8 * (2 * STAGES), 0, error, 3, abort_slot);
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (ok) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int n = m_tile * kBlockM + quad * 32 + lane;
      float* dst = out + static_cast<long long>(split) * split_stride;
      for (int c0 = 0; c0 < tn; c0 += 16) {
        uint32_t v[16];
        if (nkb > 0) {
          asm volatile(
              "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
              : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
              : "r"(tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(c0)));
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] = 0u;
        }
        float val[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) val[i] = __uint_as_float(v[i]);
        emit16(epi, dst, N, T, n, t0 + c0, val);
      }
    }
  }

  // teardown
  if (!ok) *abort_slot = 1;
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    if (*abort_slot != 0) {
      // something timed out: give copies and MMAs still in flight time to land before the memory goes away
      const long long t1 = clock64();
      while (clock64() - t1 < 2000000LL) __nanosleep(1000);
    }
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(static_cast<uint32_t>(kTmemCols)) : "memory");
  }
  stamp_time(epi.stamp_end, true);   // thread 0 is past the block-wide barrier: every warp's work is done
}

// ------------------------------------------------------------------------------------------------
// Linear layer with 8-bit weights, fp8 MMAs (tcgen05 kind::f8f6f4): nothing is converted on the way to the tensor
// cores.  The instruction wants both operands in 8 (or fewer) bits, so the bf16 activations are handed over as TWO
// e4m3 numbers each, a = s_t * (hi + lo) with hi = e4m3(a / s_t), lo = e4m3(a / s_t - hi) and one scale s_t per
// token (written by the kernel that produces the activation, or by split_rows_f8_kernel): every product of two
// e4m3 numbers is exact and is added in fp32, so the sum carries eight significant bits of every activation, as
// with a bf16 operand.  Per k-slab
// (128 k = one 128-byte swizzle row) a CTA streams a 16 KB weight tile - the same bytes per slab as the bf16 kernel,
// twice the reduction length - and fetches the token tile's hi rows and lo rows into one stage; one MMA per 32-k
// step takes the whole stage as its N side (N = 2 x token tile), so W * hi and W * lo land side by side in tensor
// memory, and the epilogue adds them and applies both scales.  (Two MMAs per step into separate or into the same
// columns measured slower: at these widths an instruction costs about the same whether N is 96 or 192.)
// Structure, roles and waits as in tc_gemm_split_kernel; the weight ring and the activation ring are separate
// (4 + 2 stages at 96 tokens) so that two CTAs still fit an SM.  Wider steps run as 128-token tiles.
constexpr int kBlockK8 = 128;

__device__ __forceinline__ void umma_f8(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}

template <int TN_MAX>
struct F8SmemLayout {
  static constexpr int kWStages = TN_MAX <= 64 ? 5 : TN_MAX <= 96 ? 4 : 3;
  static constexpr int kAStages = TN_MAX <= 32 ? 3 : 2;
  static constexpr int kAStageBytes = 2 * TN_MAX * kBlockK8;               // hi rows, then lo rows
  static constexpr int kAOff = kWStages * kWStageBytes;
  static constexpr int kTiles = kAOff + kAStages * kAStageBytes;
  static constexpr int kTotal = kTiles + 256;
  static_assert(2 * (kTotal + 1024) <= 228 * 1024, "two CTAs per SM");
};

template <int TN_MAX>
__global__ void __launch_bounds__(192) tc_gemm_f8_kernel(const __grid_constant__ CUtensorMap map_w,
                                                         const __grid_constant__ CUtensorMap map_a, int T, int N,
                                                         int kb_total, int kb_per_split, int lo_row0,
                                                         const float* __restrict__ wscale, const float* __restrict__ ascale,
                                                         float* __restrict__ out, long long split_stride, int32_t* error,
                                                         TcEpilogue epi, int w4) {
  using L = F8SmemLayout<TN_MAX>;
  constexpr int SW = L::kWStages, SA = L::kAStages;
  constexpr int kTmemCols = TN_MAX <= 32 ? 64 : TN_MAX <= 64 ? 128 : 256;   // W * hi | W * lo, TN_MAX columns each
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  uint8_t* base_ptr = smem_raw;
  const uint32_t bars = base + L::kTiles;
  const uint32_t bar_w_full = bars, bar_w_empty = bars + 8 * SW, bar_a_full = bars + 16 * SW, bar_a_empty = bar_a_full + 8 * SA,
                 bar_acc = bar_a_empty + 8 * SA;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + L::kTiles + 8 * (2 * SW + 2 * SA + 1));
  volatile int* abort_slot = reinterpret_cast<volatile int*>(base_ptr + L::kTiles + 8 * (2 * SW + 2 * SA + 1) + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  stamp_time(epi.stamp_begin, false);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int t_tile = blockIdx.x, m_tile = blockIdx.y, split = blockIdx.z;
  const int kb0 = split * kb_per_split;
  const int nkb = min(kb_per_split, kb_total - kb0);
  const int t0 = t_tile * TN_MAX;
  const int tn = min(TN_MAX, ((T - t0) + 15) & ~15);

  if (threadIdx.x == 0) {
    if (base & 1023u) atomicCAS(error, 0, 5);
    *abort_slot = (base & 1023u) ? 1 : 0;
  }
  if (warp == 0 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
    for (int i = 0; i < 2 * SW + 2 * SA + 1; ++i) mbar_init(bars + 8 * i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))),
                 "r"(static_cast<uint32_t>(kTmemCols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  bool ok = true;
  if (threadIdx.x == 64 && *reinterpret_cast<volatile int32_t*>(error) != 0) *abort_slot = 1;

  if (warp == 0) {
    if (lane == 0 && *abort_slot == 0) {
      uint64_t pol_first, pol_last;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_first));
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_last));
      auto load_w = [&](int kb, int st) {
        // 4-bit weights: the copy reads 8 KB of nibbles and spreads them over the 16 KB stage (every 16 bytes of
        // shared memory hold 16 nibbles and 8 unused bytes); the bytes counted are the ones read
        mbar_expect_tx(bar_w_full + 8 * st, w4 ? kWStageBytes / 2 : kWStageBytes);
        tma_load_2d(base + st * kWStageBytes, &map_w, 0, (m_tile * kb_total + kb0 + kb) * kBlockM, bar_w_full + 8 * st, pol_first);
      };
      auto load_a = [&](int kb, int st) {
        mbar_expect_tx(bar_a_full + 8 * st, L::kAStageBytes);
        const uint32_t dst = base + L::kAOff + st * L::kAStageBytes;
        tma_load_2d(dst, &map_a, (kb0 + kb) * kBlockK8, t0, bar_a_full + 8 * st, pol_last);
        tma_load_2d(dst + TN_MAX * kBlockK8, &map_a, (kb0 + kb) * kBlockK8, lo_row0 + t0, bar_a_full + 8 * st, pol_last);
      };
      for (int kb = 0; kb < min(SW, nkb); ++kb) load_w(kb, kb);   // weights do not depend on the previous kernel
      pdl_wait_here();
      for (int kb = 0; kb < min(SA, nkb); ++kb) load_a(kb, kb);
      for (int kb = 0; ok && kb < nkb; ++kb) {
        const int kw = kb + SW, ka = kb + SA;
        if (ka < nkb) {
          if (!mbar_wait(bar_a_empty + 8 * (ka % SA), ((ka / SA) & 1) ^ 1, error, 6, abort_slot)) { ok = false; break; }
          load_a(ka, ka % SA);
        }
        if (kw < nkb) {
          if (!mbar_wait(bar_w_empty + 8 * (kw % SW), ((kw / SW) & 1) ^ 1, error, 1, abort_slot)) { ok = false; break; }
          load_w(kw, kw % SW);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // instruction descriptor: fp32 accumulate, e4m3 x e4m3 (format code 0 for both), K-major, M = 128, and
      // N = the whole activation stage - hi rows and lo rows in one instruction, their sums side by side
      // (4-bit weights: format code 5, e2m1, for the weight operand; a k-step is still 32 bytes of the swizzled row)
      const uint32_t idesc = (1u << 4) | (w4 ? (5u << 7) : 0u) | (static_cast<uint32_t>((2 * TN_MAX) >> 3) << 17) |
                             (static_cast<uint32_t>(kBlockM >> 4) << 24);
      for (int kb = 0; kb < nkb; ++kb) {
        const int ws = kb % SW, as = kb % SA;
        if (!mbar_wait(bar_w_full + 8 * ws, (kb / SW) & 1, error, 2, abort_slot)) { ok = false; break; }
        if (!mbar_wait(bar_a_full + 8 * as, (kb / SA) & 1, error, 7, abort_slot)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint64_t adesc = umma_desc(base + ws * kWStageBytes);
        const uint64_t bdesc = umma_desc(base + L::kAOff + as * L::kAStageBytes);
#pragma unroll
        for (int kk = 0; kk < kBlockK8 / 32; ++kk)   // 32 fp8 = 32 bytes further along K inside the swizzled row
          umma_f8(tmem_base, adesc + 2 * kk, bdesc + 2 * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
        umma_commit(bar_w_empty + 8 * ws);
        umma_commit(bar_a_empty + 8 * as);
      }
      if (ok) umma_commit(bar_acc);
    }
  } else {
    const int quad = warp & 3;                      // tensor-memory lanes 32 * (warp % 4) .. + 31
    if (nkb > 0) ok = mbar_wait(bar_acc, 0, error, 3, abort_slot);
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (ok) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int n = m_tile * kBlockM + quad * 32 + lane;
      const float ws = n < N ? __ldg(wscale + n) : 0.f;
      float* dst = out + static_cast<long long>(split) * split_stride;
      for (int c0 = 0; c0 < tn; c0 += 16) {
        uint32_t vh[16], vl[16];
        if (nkb > 0) {
          const uint32_t addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(c0);
          asm volatile(
              "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
              : "=r"(vh[0]), "=r"(vh[1]), "=r"(vh[2]), "=r"(vh[3]), "=r"(vh[4]), "=r"(vh[5]), "=r"(vh[6]), "=r"(vh[7]),
                "=r"(vh[8]), "=r"(vh[9]), "=r"(vh[10]), "=r"(vh[11]), "=r"(vh[12]), "=r"(vh[13]), "=r"(vh[14]), "=r"(vh[15])
              : "r"(addr));
          asm volatile(
              "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
              : "=r"(vl[0]), "=r"(vl[1]), "=r"(vl[2]), "=r"(vl[3]), "=r"(vl[4]), "=r"(vl[5]), "=r"(vl[6]), "=r"(vl[7]),
                "=r"(vl[8]), "=r"(vl[9]), "=r"(vl[10]), "=r"(vl[11]), "=r"(vl[12]), "=r"(vl[13]), "=r"(vl[14]), "=r"(vl[15])
              : "r"(addr + static_cast<uint32_t>(TN_MAX)));
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) vh[i] = vl[i] = 0u;
        }
        float val[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int t = t0 + c0 + i;
          const float as = t < T ? __ldg(ascale + t) : 0.f;
          val[i] = (__uint_as_float(vh[i]) + __uint_as_float(vl[i])) * (ws * as);
        }
        emit16(epi, dst, N, T, n, t0 + c0, val);
      }
    }
  }

  if (!ok) *abort_slot = 1;
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    if (*abort_slot != 0) {
      const long long t1 = clock64();
      while (clock64() - t1 < 2000000LL) __nanosleep(1000);
    }
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"(static_cast<uint32_t>(kTmemCols)) : "memory");
  }
  stamp_time(epi.stamp_end, true);
}

// One block per token: a[t][k] (bf16) -> s_t = max|a[t]| / 448, hi = e4m3(a / s_t), lo = e4m3(a / s_t - hi);
// hi rows at out[t], lo rows at out[lo_row0 + t], s_t at scale[t].
__global__ void __launch_bounds__(256) split_rows_f8_kernel(const __nv_bfloat16* __restrict__ a, int K, uint8_t* __restrict__ out,
                                                            int lo_row0, float* __restrict__ scale,
                                                            unsigned long long* stamp_begin, unsigned long long* stamp_end) {
  __shared__ float red[8];
  stamp_time(stamp_begin, false);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  pdl_wait_here();
  const int t = blockIdx.x;
  const uint4* row = reinterpret_cast<const uint4*>(a + static_cast<long long>(t) * K);
  float amax = 0.f;
  for (int i = threadIdx.x; i < K / 8; i += blockDim.x) {
    const uint4 v = row[i];
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      amax = fmaxf(amax, fabsf(__uint_as_float(w[j] << 16)));
      amax = fmaxf(amax, fabsf(__uint_as_float(w[j] & 0xffff0000u)));
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = red[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) amax = fmaxf(amax, red[i]);
  const float s = token_scale_e4m3(amax);
  const float inv = 1.f / s;
  if (threadIdx.x == 0) scale[t] = s;
  uint2* hi = reinterpret_cast<uint2*>(out + static_cast<long long>(t) * K);
  uint2* lo = reinterpret_cast<uint2*>(out + static_cast<long long>(lo_row0 + t) * K);
  for (int i = threadIdx.x; i < K / 8; i += blockDim.x) {
    const uint4 v = row[i];
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t h[2] = {0, 0}, l[2] = {0, 0};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t hq, lq;
      split_pair_e4m3(__uint_as_float(w[j] << 16) * inv, __uint_as_float(w[j] & 0xffff0000u) * inv, hq, lq);
      h[j >> 1] |= hq << (16 * (j & 1));
      l[j >> 1] |= lq << (16 * (j & 1));
    }
    hi[i] = make_uint2(h[0], h[1]);
    lo[i] = make_uint2(l[0], l[1]);
  }
  __syncthreads();
  stamp_time(stamp_end, true);
}

// row-major e4m3 bytes [N][K] -> tiles of 128 rows x 128 bytes (k), zero where the matrix ends
__global__ void __launch_bounds__(256) retile_f8_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, int N, int K,
                                                        int n_kslabs) {
  const int kb = blockIdx.x, mt = blockIdx.y;
  uint8_t* out = dst + (static_cast<long long>(mt) * n_kslabs + kb) * (kBlockM * kBlockK8);
  for (int i = threadIdx.x; i < kBlockM * kBlockK8; i += blockDim.x) {
    const int r = i / kBlockK8, b = i % kBlockK8;
    const int n = mt * kBlockM + r, k = kb * kBlockK8 + b;
    out[i] = (n < N && k < K) ? src[static_cast<long long>(n) * K + k] : static_cast<uint8_t>(0);
  }
}

// row-major e2m1 nibbles [N][K / 2] bytes -> tiles of 128 rows x 64 bytes (128 k), zero where the matrix ends
__global__ void __launch_bounds__(256) retile_f4_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, int N, int K,
                                                        int n_kslabs) {
  constexpr int kRowBytes = kBlockK8 / 2;
  const int kb = blockIdx.x, mt = blockIdx.y;
  uint8_t* out = dst + (static_cast<long long>(mt) * n_kslabs + kb) * (kBlockM * kRowBytes);
  for (int i = threadIdx.x; i < kBlockM * kRowBytes; i += blockDim.x) {
    const int r = i / kRowBytes, b = i % kRowBytes;
    const int n = mt * kBlockM + r, k = kb * kBlockK8 + 2 * b;   // K is even: a byte's two entries end together
    out[i] = (n < N && k < K) ? src[static_cast<long long>(n) * (K / 2) + k / 2] : static_cast<uint8_t>(0);
  }
}

// ------------------------------------------------------------------------------------------------
// CTA-pair kernel for steps of more than 128 tokens (the tensor-bound regime).
//
// Two CTAs of a cluster own two neighbouring 128-row weight tiles and the same token tile; one
// tcgen05.mma.cta_group::2 (M = 256) drives both SMs' tensor cores.  Each CTA loads its own weight slab and only
// HALF of the token tile's activations (its tn/2 rows of the N side; the instruction reads the two halves from the
// two CTAs' shared memory): a stage is 32 KB instead of 48 KB, the activations cross L2 -> SM once per 256 weight
// rows instead of once per 128, and shared memory is read at about half the rate per flop.
// The kernel is persistent: one pair per two SMs walks over its units (weight-tile pair, K slice, token tile) - token
// tile fastest, so the pairs that share a weight slab run at the same time and the second reader finds it in
// L2 - with the accumulator double-buffered in tensor memory (2 x 256 columns): the epilogue of one unit runs
// under the main loop of the next.  One CTA per SM by construction (192 KB ring, all 512 tensor-memory columns).
//   both CTAs : warp 0 loads (plain TMA loads; the bytes are counted on the leader's "full" barrier),
//               warps 2-5 read their own 128 accumulator rows from tensor memory, store them and hand the
//               accumulator buffer back to the leader
//   leader    : warp 1 issues the MMAs and commits every stage to BOTH CTAs' "empty" barriers
// All waits on mbarriers are bounded as in the kernel above; the two cluster-wide barriers (after set-up, before
// the tensor memory is freed) are reached by every thread of both CTAs on every path.
constexpr int kPairTN = 256;
constexpr int kPairStages = 6;
constexpr int kPairAStageBytes = 128 * kBlockK * 2;
constexpr int kPairStageBytes = kWStageBytes + kPairAStageBytes;
constexpr int kPairTiles = kPairStages * kPairStageBytes;
constexpr int kPairSmem = kPairTiles + 256;
constexpr int kPairBars = 2 * kPairStages + 4;   // full[S], empty[S], acc_full[2], acc_empty[2]

__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t leader_bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(leader_bar), "r"(x), "r"(y), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
// arrives (once the MMAs issued so far have completed) on the barrier at this shared-memory offset in both CTAs:
// one commit per CTA, each naming that CTA's barrier by its cluster address
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  uint32_t peer_bar;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(peer_bar) : "r"(bar), "r"(1));
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(peer_bar) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t leader_address(uint32_t local) {   // the same offset in the leader CTA's shared memory
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(0));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

// Unit u = ((weight-tile pair * K slices) + slice) * token tiles + token tile.  In round r the pair with index q
// takes unit r * n_pairs + (q + r) % n_pairs: neighbouring pairs work on the token tiles of one weight slab at
// the same time, and the rotation by r gives every pair a mix of wide and narrow token tiles.
struct PairUnit { int m_pair, t_tile, split; };
__device__ __forceinline__ PairUnit pair_unit(int u, int n_t, int n_split) {
  PairUnit r;
  r.t_tile = u % n_t;
  const int q = u / n_t;
  r.split = q % n_split;
  r.m_pair = q / n_split;
  return r;
}

__global__ void __launch_bounds__(192) tc_gemm_pair_kernel(const __grid_constant__ CUtensorMap map_w,
                                                      const __grid_constant__ CUtensorMap map_a, int T, int N,
                                                      int kb_total, int kb_per_split, int n_split, int n_units,
                                                      float* __restrict__ out, long long split_stride, int32_t* error,
                                                      TcEpilogue epi) {
  constexpr int S = kPairStages;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  uint8_t* base_ptr = smem_raw;
  const uint32_t bars = base + kPairTiles;
  const uint32_t bar_full = bars, bar_empty = bars + 8 * S, bar_acc_full = bars + 16 * S, bar_acc_empty = bars + 16 * S + 16;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kPairTiles + 8 * kPairBars);
  volatile int* abort_slot = reinterpret_cast<volatile int*>(base_ptr + kPairTiles + 8 * kPairBars + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  stamp_time(epi.stamp_begin, false);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int n_t = (T + kPairTN - 1) / kPairTN;

  if (threadIdx.x == 0) {
    if (base & 1023u) atomicCAS(error, 0, 5);
    *abort_slot = (base & 1023u) ? 1 : 0;
  }
  if (warp == 0 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
    for (int s = 0; s < 2 * S + 2; ++s) mbar_init(bars + 8 * s, 1);
    mbar_init(bar_acc_empty, 8);        // the four epilogue warps of both CTAs
    mbar_init(bar_acc_empty + 8, 8);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // the pair's two accumulator buffers: 2 x 256 fp32 columns x 128 lanes in each CTA
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))),
                 "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();                                      // both CTAs' barriers exist before anything arrives on them
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  bool ok = true;
  if (threadIdx.x == 64 && *reinterpret_cast<volatile int32_t*>(error) != 0) *abort_slot = 1;

  if (warp == 0) {
    if (lane == 0 && *abort_slot == 0) {
      uint64_t pol_w, pol_last;
      // a weight slab is read by the pairs of all token tiles at about the same time: no "evict first" here
      asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol_w));
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_last));
      const uint32_t leader_full = leader_address(bar_full);
      int it = 0;                                          // slabs loaded so far, over all units
      bool waited = false;                                 // griddepcontrol.wait done (before the first activation load)
      for (int r = 0; ok && r * n_pairs < n_units; ++r) {
        const int u = r * n_pairs + (pair_id + r) % n_pairs;   // round r, rotated: see pair_unit
        if (u >= n_units) break;                               // only the last round is incomplete
        const PairUnit pu = pair_unit(u, n_t, n_split);
        const int m_tile = 2 * pu.m_pair + static_cast<int>(rank);
        const int kb0 = pu.split * kb_per_split;
        const int nkb = min(kb_per_split, kb_total - kb0);
        const int t0 = pu.t_tile * kPairTN;
        const int tn = min(kPairTN, ((T - t0) + 31) & ~31);
        const int a_row = t0 + static_cast<int>(rank) * (tn >> 1);
        int kb = 0;
        if (!waited) {
          // weights do not depend on the previous kernel: fill the ring with weight slabs, then wait, then the activations
          const int pre = min(S, nkb);
          for (int k2 = 0; k2 < pre; ++k2) {
            if (rank == 0) mbar_expect_tx(bar_full + 8 * k2, 2 * kPairStageBytes);   // this CTA's and the peer's bytes
            tma_load_2d_pair(base + k2 * kPairStageBytes, &map_w, 0, (m_tile * kb_total + kb0 + k2) * kBlockM, leader_full + 8 * k2, pol_w);
          }
          pdl_wait_here();
          waited = true;
          for (int k2 = 0; k2 < pre; ++k2)
            tma_load_2d_pair(base + k2 * kPairStageBytes + kWStageBytes, &map_a, (kb0 + k2) * kBlockK, a_row, leader_full + 8 * k2, pol_last);
          kb = pre;
          it = pre;
        }
        for (; kb < nkb; ++kb, ++it) {
          const int s = it % S;
          const uint32_t ph = (it / S) & 1;
          if (!mbar_wait(bar_empty + 8 * s, ph ^ 1, error, 1, abort_slot)) { ok = false; break; }
          if (rank == 0) mbar_expect_tx(bar_full + 8 * s, 2 * kPairStageBytes);
          const uint32_t wdst = base + s * kPairStageBytes;
          tma_load_2d_pair(wdst, &map_w, 0, (m_tile * kb_total + kb0 + kb) * kBlockM, leader_full + 8 * s, pol_w);
          tma_load_2d_pair(wdst + kWStageBytes, &map_a, (kb0 + kb) * kBlockK, a_row, leader_full + 8 * s, pol_last);
        }
      }
      if (!waited) pdl_wait_here();
      // every stage handed back: no arrival from the leader's commits is still on its way to this CTA's barriers
      for (int j = max(it - S, 0); ok && j < it; ++j)
        if (!mbar_wait(bar_empty + 8 * (j % S), (j / S) & 1, error, 6, abort_slot)) ok = false;
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      int it = 0, iter = 0;
      for (int r = 0; ok && r * n_pairs < n_units; ++r, ++iter) {
        const int u = r * n_pairs + (pair_id + r) % n_pairs;
        if (u >= n_units) break;
        const PairUnit pu = pair_unit(u, n_t, n_split);
        const int kb0 = pu.split * kb_per_split;
        const int nkb = min(kb_per_split, kb_total - kb0);
        const int t0 = pu.t_tile * kPairTN;
        const int tn = min(kPairTN, ((T - t0) + 31) & ~31);
        // instruction descriptor: fp32 accumulate, bf16 x bf16, both operands K-major, N = tn, M = 256 over the pair
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(tn >> 3) << 17) |
                               (static_cast<uint32_t>(256 >> 4) << 24);
        const int b = iter & 1;
        // the epilogue warps of both CTAs have read what the unit before last left in this buffer
        if (!mbar_wait(bar_acc_empty + 8 * b, ((iter >> 1) & 1) ^ 1, error, 7, abort_slot)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t acc = tmem_base + static_cast<uint32_t>(b * kPairTN);
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % S;
          const uint32_t ph = (it / S) & 1;
          if (!mbar_wait(bar_full + 8 * s, ph, error, 2, abort_slot)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t wsrc = base + s * kPairStageBytes;
          const uint64_t adesc = umma_desc(wsrc), bdesc = umma_desc(wsrc + kWStageBytes);
#pragma unroll
          for (int kk = 0; kk < kBlockK / 16; ++kk)
            umma_bf16_pair(acc, adesc + 2 * kk, bdesc + 2 * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
          umma_commit_pair(bar_empty + 8 * s);          // the stage is free in both CTAs once these MMAs have read it
        }
        if (ok) umma_commit_pair(bar_acc_full + 8 * b);  // this unit's accumulators are complete, in both CTAs
      }
    }
  } else {
    const int quad = warp & 3;
    const uint32_t leader_acc_empty = leader_address(bar_acc_empty);
    int iter = 0;
    for (int r = 0; r * n_pairs < n_units; ++r, ++iter) {
      const int u = r * n_pairs + (pair_id + r) % n_pairs;
      if (u >= n_units) break;
      const PairUnit pu = pair_unit(u, n_t, n_split);
      const int m_tile = 2 * pu.m_pair + static_cast<int>(rank);
      const int t0 = pu.t_tile * kPairTN;
      const int tn = min(kPairTN, ((T - t0) + 31) & ~31);
      const int b = iter & 1;
      if (ok) ok = mbar_wait(bar_acc_full + 8 * b, (iter >> 1) & 1, error, 3, abort_slot);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int n = m_tile * kBlockM + quad * 32 + lane;
      float* dst = out + static_cast<long long>(pu.split) * split_stride;
      for (int c0 = 0; c0 < tn; c0 += 16) {
        uint32_t v[16];
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
              "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
            : "r"(tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(b * kPairTN + c0)));
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        float val[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) val[i] = __uint_as_float(v[i]);
        emit16(epi, dst, N, T, n, t0 + c0, val);
      }
      // this warp is done with the buffer: tell the leader's MMA warp (eight such arrivals free it)
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(leader_acc_empty + 8 * b);
    }
  }

  // teardown
  if (!ok) *abort_slot = 1;
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1 && *abort_slot != 0) {
    // something timed out: give copies and MMAs still in flight time to land before the memory goes away
    const long long t1 = clock64();
    while (clock64() - t1 < 2000000LL) __nanosleep(1000);
  }
  cluster_sync_all();                                      // neither CTA leaves while the other may still use its memory
  if (warp == 1)
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  stamp_time(epi.stamp_end, true);
}

// Self-test of the give-up path: one thread waits, with the same bounded wait as the kernels above but a short
// limit, on a barrier that nobody will ever signal.  The wait runs out, the code lands in *error and the kernel
// returns normally; kernels launched afterwards find the word set and return early, and the host reports the step
// as failed.  Nothing traps, spins without bound or touches memory it does not own.
__global__ void wait_probe_kernel(int32_t* error, long long limit_cycles) {
  __shared__ __align__(8) unsigned long long bar_mem;
  __shared__ int stop_mem;
  if (threadIdx.x == 0) {
    stop_mem = 0;
    mbar_init(smem_u32(&bar_mem), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_wait(smem_u32(&bar_mem), 0, error, 9, &stop_mem, limit_cycles);
  }
}

// Weights are kept tile by tile: block (m, kb) of the tiled array is the 128 x 64 piece W[128m .. +127][64kb .. +63]
// as 128 rows of 128 bytes, zero where the matrix ends.  One pipeline stage is then one contiguous 16 KB read, and
// the stages of a CTA follow each other in memory (DRAM pages are read whole instead of 128 bytes at a time).
__global__ void __launch_bounds__(256) retile_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst,
                                                     int N, int K, int n_kslabs) {
  const int kb = blockIdx.x, mt = blockIdx.y;
  uint4* out = reinterpret_cast<uint4*>(dst + (static_cast<long long>(mt) * n_kslabs + kb) * (kBlockM * kBlockK));
  for (int i = threadIdx.x; i < kBlockM * (kBlockK / 8); i += blockDim.x) {
    const int r = i / (kBlockK / 8), c = i % (kBlockK / 8);
    const int n = mt * kBlockM + r, k = kb * kBlockK + c * 8;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (n < N && k < K) v = *reinterpret_cast<const uint4*>(src + static_cast<long long>(n) * K + k);   // K is a multiple of 8
    out[i] = v;
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

int make_map(CUtensorMap* map, const void* ptr, long long rows, int K, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return -1;
  if (K % 8 || (reinterpret_cast<uintptr_t>(ptr) & 15)) return -1;   // rows must stay 16-byte aligned; a K tail is zero-filled by TMA
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(rows)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(K) * 2};
  cuuint32_t box[2] = {kBlockK, static_cast<cuuint32_t>(box_rows)};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    std::fprintf(stderr, "sled: cuTensorMapEncodeTiled failed (%d) rows=%lld K=%d box=%d\n", static_cast<int>(r), rows, K, box_rows);
    return -1;
  }
  return 0;
}

// the same for an array of bytes: boxes of 128 bytes x box_rows rows
int make_map_u8(CUtensorMap* map, const void* ptr, long long rows, int K, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return -1;
  if (K % 16 || (reinterpret_cast<uintptr_t>(ptr) & 15)) return -1;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(rows)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(K)};
  cuuint32_t box[2] = {kBlockK8, static_cast<cuuint32_t>(box_rows)};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    std::fprintf(stderr, "sled: cuTensorMapEncodeTiled (bytes) failed (%d) rows=%lld K=%d box=%d\n", static_cast<int>(r), rows, K, box_rows);
    return -1;
  }
  return 0;
}

// tiles of 128 rows x 128 nibbles (64 bytes a row in global memory): the element type "16 x 4 bits, 16-byte aligned"
// lets the copy write each 8 bytes of nibbles into the first half of a 16-byte piece of shared memory
int make_map_u4(CUtensorMap* map, const void* ptr, long long rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return -1;
  if (reinterpret_cast<uintptr_t>(ptr) & 31) return -1;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(kBlockK8), static_cast<cuuint64_t>(rows)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(kBlockK8 / 2)};
  cuuint32_t box[2] = {kBlockK8, kBlockM};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    std::fprintf(stderr, "sled: cuTensorMapEncodeTiled (nibbles) failed (%d) rows=%lld\n", static_cast<int>(r), rows);
    return -1;
  }
  return 0;
}

}  // namespace

int tc_wait_probe_launch(int32_t* error, long long limit_cycles, cudaStream_t s) {
  if (!error || limit_cycles <= 0 || limit_cycles > kWaitCycles) return -1;
  wait_probe_kernel<<<1, 32, 0, s>>>(error, limit_cycles);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int tma_map_bf16_rows(CUtensorMap* map, const void* dev_ptr, long long rows, int cols, int box_rows) {
  return make_map(map, dev_ptr, rows, cols, box_rows);
}

size_t tc_weight_tiled_bytes(int N, int K) {
  return static_cast<size_t>((N + kBlockM - 1) / kBlockM) * ((K + kBlockK - 1) / kBlockK) * kWStageBytes;
}

int tc_weight_init(TcWeight* w, const void* rowmajor, void* tiled, int N, int K) {
  if (K % 8 || (reinterpret_cast<uintptr_t>(rowmajor) & 15) || (reinterpret_cast<uintptr_t>(tiled) & 15)) return -1;
  const int n_mtiles = (N + kBlockM - 1) / kBlockM, n_kslabs = (K + kBlockK - 1) / kBlockK;
  retile_kernel<<<dim3(n_kslabs, n_mtiles), 256>>>(static_cast<const __nv_bfloat16*>(rowmajor), static_cast<__nv_bfloat16*>(tiled), N, K, n_kslabs);
  if (cudaDeviceSynchronize() != cudaSuccess) return -1;
  if (make_map(&w->map, tiled, static_cast<long long>(n_mtiles) * n_kslabs * kBlockM, kBlockK, kBlockM)) return -1;
  w->N = N;
  w->K = K;
  w->ready = true;
  return 0;
}

size_t tc_weight_f8_tiled_bytes(int N, int K) {
  return static_cast<size_t>((N + kBlockM - 1) / kBlockM) * ((K + kBlockK8 - 1) / kBlockK8) * kWStageBytes;
}

int tc_weight_init_f8(TcWeight* w, const void* rowmajor_bytes, void* tiled, const float* scale, int N, int K) {
  if (K % 16 || !scale || (reinterpret_cast<uintptr_t>(tiled) & 15)) return -1;
  const int n_mtiles = (N + kBlockM - 1) / kBlockM, n_kslabs = (K + kBlockK8 - 1) / kBlockK8;
  retile_f8_kernel<<<dim3(n_kslabs, n_mtiles), 256>>>(static_cast<const uint8_t*>(rowmajor_bytes), static_cast<uint8_t*>(tiled), N, K, n_kslabs);
  if (cudaDeviceSynchronize() != cudaSuccess) return -1;
  if (make_map_u8(&w->map8, tiled, static_cast<long long>(n_mtiles) * n_kslabs * kBlockM, kBlockK8, kBlockM)) return -1;
  w->scale = scale;
  w->N = N;
  w->K = K;
  w->f8 = true;
  w->ready = true;
  return 0;
}

size_t tc_weight_f4_tiled_bytes(int N, int K) {
  return static_cast<size_t>((N + kBlockM - 1) / kBlockM) * ((K + kBlockK8 - 1) / kBlockK8) * (kWStageBytes / 2);
}

int tc_weight_init_f4(TcWeight* w, const void* rowmajor_nibbles, void* tiled, const float* scale, int N, int K) {
  if (K % 16 || !scale || (reinterpret_cast<uintptr_t>(tiled) & 31)) return -1;
  const int n_mtiles = (N + kBlockM - 1) / kBlockM, n_kslabs = (K + kBlockK8 - 1) / kBlockK8;
  retile_f4_kernel<<<dim3(n_kslabs, n_mtiles), 256>>>(static_cast<const uint8_t*>(rowmajor_nibbles), static_cast<uint8_t*>(tiled), N, K, n_kslabs);
  if (cudaDeviceSynchronize() != cudaSuccess) return -1;
  if (make_map_u4(&w->map8, tiled, static_cast<long long>(n_mtiles) * n_kslabs * kBlockM)) return -1;
  w->scale = scale;
  w->N = N;
  w->K = K;
  w->f8 = true;
  w->f4 = true;
  w->ready = true;
  return 0;
}

int tc_activation8_init(TcActivation8* a, void* data, float* scale, int rows, int K) {
  if (rows % 128 || K % 16 || !data || !scale) return -1;
  const int boxes[4] = {32, 64, 96, 128};
  for (int i = 0; i < 4; ++i)
    if (make_map_u8(&a->map[i], data, 2LL * rows, K, boxes[i])) return -1;
  a->data = static_cast<uint8_t*>(data);
  a->scale = scale;
  a->rows = rows;
  a->K = K;
  return 0;
}

int tc_split_rows_launch(const void* a_bf16, int T, const TcActivation8& dst, cudaStream_t s,
                         unsigned long long* stamp_begin, unsigned long long* stamp_end) {
  if (T <= 0) return 0;
  if (T > dst.rows || (reinterpret_cast<uintptr_t>(a_bf16) & 15)) return -1;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(T, 1, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t err = cudaLaunchKernelEx(&cfg, split_rows_f8_kernel, static_cast<const __nv_bfloat16*>(a_bf16), dst.K, dst.data, dst.rows,
                                       dst.scale, stamp_begin, stamp_end);
  return err == cudaSuccess ? 1 : -1;
}

void tc_weight_free(TcWeight* w) { w->ready = false; }

int tc_activation_init(TcActivation* a, const void* dev_ptr, int rows, int K) {
  if (rows % 256) return -1;
  const int boxes[kTokenTiles] = {32, 64, 96, 128, 160, 256};
  for (int i = 0; i < kTokenTiles; ++i)
    if (make_map(&a->map[i], dev_ptr, rows, K, boxes[i])) return -1;
  a->rows = rows;
  a->K = K;
  return 0;
}

// K slices: as many as keep every CTA of the launch resident at once (two per SM), each with at least 4 slabs;
// the returned count is the number of slices that actually get work.
// Above 160 tokens, when the weight tiles pair up, the CTA-pair kernel runs (see tc_gemm_launch): its n_sm / 2 pairs
// work round by round over (weight-tile pairs x token tiles x slices) units, so the slice count is chosen to
// minimise rounds x (k-slabs per unit + a unit's fixed cost) + what the consumer pays for adding up the slices
// (both in units of one k-slab's main-loop time).
constexpr int kSingleTileMax = 160;   // widest step that one token tile of the single-CTA kernel (two CTAs per SM) holds
static bool pair_kernel_applies(int T, int N) { return T > kSingleTileMax && ((N + kBlockM - 1) / kBlockM) % 2 == 0; }

int tc_gemm_split(int T, int N, int K, int n_sm) {
  const int tiles = ((N + kBlockM - 1) / kBlockM) * (T > kSingleTileMax ? (T + 255) / 256 : 1);
  const int kb_total = (K + kBlockK - 1) / kBlockK;
  if (pair_kernel_applies(T, N) && n_sm >= 2) {
    const int n_pairs = n_sm / 2, base = tiles / 2;
    int best = 1;
    double best_cost = 0.0;
    for (int cand = 1; cand <= 8 && cand <= std::max(1, kb_total / 8); ++cand) {
      const int kb_per = (kb_total + cand - 1) / cand;
      if ((kb_total + kb_per - 1) / kb_per != cand) continue;          // this count leaves a slice without work
      const int rounds = (base * cand + n_pairs - 1) / n_pairs;
      const double cost = rounds * (kb_per + 8.0) + cand * 3e-6 * static_cast<double>(T) * N;
      if (cand == 1 || cost < best_cost) { best = cand; best_cost = cost; }
    }
    return best;
  }
  int s = std::max(1, (2 * n_sm) / tiles);
  s = std::min(s, std::max(1, kb_total / 4));
  s = std::min(s, 16);
  const int kb_per = (kb_total + s - 1) / s;
  return (kb_total + kb_per - 1) / kb_per;
}

// fp8 MMAs, 128-wide k-slabs: one weight tile per CTA and two CTAs per SM, as in the bf16 kernel
int tc_gemm_split_f8(int T, int N, int K, int n_sm) {
  const int tn = T <= 128 ? T : 128;
  const int m_tiles = (N + kBlockM - 1) / kBlockM;
  const int tiles = m_tiles * ((T + tn - 1) / tn);
  const int kb_total = (K + kBlockK8 - 1) / kBlockK8;
  int s = std::max(1, (2 * n_sm) / tiles);
  s = std::min(s, std::max(1, kb_total / 2));
  s = std::min(s, 16);
  const int kb_per = (kb_total + s - 1) / s;
  return (kb_total + kb_per - 1) / kb_per;
}

template <int TN_MAX>
static int launch_f8(const TcWeight& w, const TcActivation8& a, int box, int T, int n_split, float* out, int64_t split_stride,
                     int32_t* error, const TcEpilogue& epi, cudaStream_t s) {
  using L = F8SmemLayout<TN_MAX>;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(tc_gemm_f8_kernel<TN_MAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal) != cudaSuccess) return -1;
    configured = true;
  }
  const int kb_total = (w.K + kBlockK8 - 1) / kBlockK8;
  const int kb_per = (kb_total + n_split - 1) / n_split;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((T + TN_MAX - 1) / TN_MAX, (w.N + kBlockM - 1) / kBlockM, n_split);
  cfg.blockDim = dim3(192, 1, 1);
  cfg.dynamicSmemBytes = L::kTotal;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const long long stride = split_stride;
  cudaError_t err = cudaLaunchKernelEx(&cfg, tc_gemm_f8_kernel<TN_MAX>, w.map8, a.map[box], T, w.N, kb_total, kb_per, a.rows, w.scale,
                                       static_cast<const float*>(a.scale), out, stride, error, epi, w.f4 ? 1 : 0);
  return err == cudaSuccess ? 1 : -1;
}

int tc_gemm_f8_launch(const TcActivation8& a, const TcWeight& w, int T, int n_split, float* out, int64_t split_stride,
                      int32_t* error, const TcEpilogue& epi, cudaStream_t s) {
  if (!w.ready || !w.f8 || a.K != w.K || T <= 0 || T > a.rows || n_split < 1) return -1;
  if (epi.mode != kEpiStore && n_split != 1) return -1;
  if (T <= 32) return launch_f8<32>(w, a, 0, T, n_split, out, split_stride, error, epi, s);
  if (T <= 64) return launch_f8<64>(w, a, 1, T, n_split, out, split_stride, error, epi, s);
  if (T <= 96) return launch_f8<96>(w, a, 2, T, n_split, out, split_stride, error, epi, s);
  return launch_f8<128>(w, a, 3, T, n_split, out, split_stride, error, epi, s);   // wider steps: 128-token tiles
}

template <int TN_MAX, int STAGES>
static int launch_split(const CUtensorMap& mw, const CUtensorMap& ma, int T, int N, int K, int n_split, float* out,
                        int64_t split_stride, int32_t* error, const TcEpilogue& epi, cudaStream_t s) {
  using L = SplitSmemLayout<TN_MAX, STAGES>;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(tc_gemm_split_kernel<TN_MAX, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal) != cudaSuccess)
      return -1;
    configured = true;
  }
  const int kb_total = (K + kBlockK - 1) / kBlockK;
  const int kb_per = (kb_total + n_split - 1) / n_split;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((T + TN_MAX - 1) / TN_MAX, (N + kBlockM - 1) / kBlockM, n_split);   // token tiles of one weight tile are neighbours
  cfg.blockDim = dim3(192, 1, 1);
  cfg.dynamicSmemBytes = L::kTotal;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may start while the previous kernel drains
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const long long stride = split_stride;
  cudaError_t err = cudaLaunchKernelEx(&cfg, tc_gemm_split_kernel<TN_MAX, STAGES>, mw, ma, T, N, kb_total, kb_per, out, stride, error, epi);
  return err == cudaSuccess ? 1 : -1;
}

static int launch_pair(const CUtensorMap& mw, const CUtensorMap& ma, int T, int N, int K, int n_split, float* out,
                       int64_t split_stride, int32_t* error, const TcEpilogue& epi, int n_sm, cudaStream_t s) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e0 = cudaFuncSetAttribute(tc_gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmem);
    if (e0 != cudaSuccess) {
      std::fprintf(stderr, "sled: shared-memory size of the CTA-pair kernel refused: %s\n", cudaGetErrorString(e0));
      return -1;
    }
    configured = true;
  }
  const int kb_total = (K + kBlockK - 1) / kBlockK;
  const int kb_per = (kb_total + n_split - 1) / n_split;
  const int n_t = (T + kPairTN - 1) / kPairTN;
  const int n_units = ((N + kBlockM - 1) / kBlockM / 2) * n_split * n_t;
  const int n_pairs = std::min(std::max(1, n_sm / 2), n_units);   // one pair per two SMs
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(2 * n_pairs, 1, 1);
  cfg.blockDim = dim3(192, 1, 1);
  cfg.dynamicSmemBytes = kPairSmem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;   // a pair = two consecutive blocks
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const long long stride = split_stride;
  cudaError_t err = cudaLaunchKernelEx(&cfg, tc_gemm_pair_kernel, mw, ma, T, N, kb_total, kb_per, n_split, n_units, out, stride, error, epi);
  if (err != cudaSuccess)
    std::fprintf(stderr, "sled: launch of the CTA-pair linear-layer kernel failed: %s\n", cudaGetErrorString(err));
  return err == cudaSuccess ? 1 : -1;
}

int tc_gemm_launch(const TcActivation& a, const TcWeight& w, int T, int n_split, float* out, int64_t split_stride,
                   int32_t* error, const TcEpilogue& epi, cudaStream_t s) {
  if (!w.ready || a.K != w.K || T <= 0 || T > a.rows || n_split < 1) return -1;
  if (epi.mode != kEpiStore && n_split != 1) return -1;   // a fused epilogue needs the complete sum
  if (w.f8) return -1;   // 8-bit weights go through tc_gemm_f8_launch
  // token tile = the smallest box that holds the step; what the narrower activation stage saves goes into ring depth
  if (T <= 32) return launch_split<32, 5>(w.map, a.map[0], T, w.N, w.K, n_split, out, split_stride, error, epi, s);
  if (T <= 64) return launch_split<64, 4>(w.map, a.map[1], T, w.N, w.K, n_split, out, split_stride, error, epi, s);
  if (T <= 96) return launch_split<96, 4>(w.map, a.map[2], T, w.N, w.K, n_split, out, split_stride, error, epi, s);
  if (T <= 128) return launch_split<128, 3>(w.map, a.map[3], T, w.N, w.K, n_split, out, split_stride, error, epi, s);
  if (T <= kSingleTileMax) return launch_split<160, 3>(w.map, a.map[4], T, w.N, w.K, n_split, out, split_stride, error, epi, s);
  if (pair_kernel_applies(T, w.N)) {
    static int n_sm = 0;
    if (n_sm == 0) {
      int dev = 0;
      cudaDeviceProp prop;
      if (cudaGetDevice(&dev) == cudaSuccess && cudaGetDeviceProperties(&prop, dev) == cudaSuccess) n_sm = prop.multiProcessorCount;
    }
    if (n_sm >= 2)   // weight tiles pair up: persistent CTA pairs, half of the token tile staged by each CTA
      return launch_pair(w.map, a.map[3], T, w.N, w.K, n_split, out, split_stride, error, epi, n_sm, s);
  }
  return launch_split<256, 2>(w.map, a.map[5], T, w.N, w.K, n_split, out, split_stride, error, epi, s);
}

}  // namespace sled
