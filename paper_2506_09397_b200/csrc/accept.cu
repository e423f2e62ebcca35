// Fused vocabulary softmax + speculative acceptance + corrective / bonus draw.
//
// One thread-block cluster per request walks its rows in
// order and stops at the deciding row: rows behind the first rejection are never read.  All quantities that decide anything are
// order-independent: the row maximum, integer softmax numerators E_v (a fixed sequence
// of correctly rounded fp32 operations followed by an exact scaling to 2^40), their
// exact 64-bit sum Z, and integer prefix sums for the inverse-CDF draw.  The accept test
// u < p/q is evaluated as U * q_d * Z < E_d * 2^24 in fp64 with U the 24-bit uniform.
#include "common.cuh"
#include "kernels.h"

namespace sled {

namespace {

constexpr int kVec = 4;                       // consecutive vocabulary entries per lane and step

enum { ST_OK = 0, ST_NONFINITE = -8 };

__device__ __forceinline__ void philox4x32_10(uint32_t k0, uint32_t k1, uint32_t c0, uint32_t c1, uint32_t c2,
                                              uint32_t c3, uint32_t out[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    c0 = hi1 ^ c1 ^ k0;
    c1 = lo1;
    c2 = hi0 ^ c3 ^ k1;
    c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// trunc(exp(x) * 2^40), x <= 0, by explicit round-to-nearest operations only
__device__ __forceinline__ unsigned long long fixed_exp(float x) {
  if (!(x >= -30.0f)) return 0ull;
  const float shift = 12582912.0f;
  const float t = __fmaf_rn(x, 0x1.715476p+0f, shift);   // log2(e)
  const float nf = __fsub_rn(t, shift);
  float r = __fmaf_rn(nf, -0x1.62e4p-1f, x);              // ln 2, high part
  r = __fmaf_rn(nf, -0x1.7f7d1cp-20f, r);                 // ln 2, low part
  float p = 0x1.6c16c2p-10f;                              // 1/720
  p = __fmaf_rn(p, r, 0x1.111112p-7f);                    // 1/120
  p = __fmaf_rn(p, r, 0x1.555556p-5f);                    // 1/24
  p = __fmaf_rn(p, r, 0x1.555556p-3f);                    // 1/6
  p = __fmaf_rn(p, r, 0.5f);
  p = __fmaf_rn(p, r, 1.0f);
  p = __fmaf_rn(p, r, 1.0f);
  const int n = static_cast<int>(nf);
  // p * 2^(n+40): p is in [0.7, 1.42], n + 40 >= -3, so the exponent add cannot leave the normal range;
  // the product is exact and one truncating conversion gives the integer
  const float scaled = __uint_as_float(__float_as_uint(p) + (static_cast<uint32_t>(n + 40) << 23));
  return __float2ull_rz(scaled);
}

// Two fp32 lanes per instruction (add / mul / fma .f32x2): each lane is rounded to nearest exactly like the scalar
// operation, so the packed form of fixed_exp below returns the same integers with about half the instructions.
__device__ __forceinline__ unsigned long long pack2(float a, float b) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ unsigned long long mul2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}

// fixed_exp(z0 * inv_tau - m) and fixed_exp(z1 * inv_tau - m): the same operations in the same order, two lanes at
// a time.  The integer part n of x * log2(e) is read off the low mantissa bits of t = x * log2(e) + 1.5 * 2^23
// (t keeps the exponent of the shift constant, so its bit pattern minus the constant's is n).
struct Exp2Consts {
  unsigned long long inv_tau, neg_m, log2e, shift, neg_shift, ln2_hi, ln2_lo, c6, c5, c4, c3, half, one;
};
__device__ __forceinline__ Exp2Consts exp2_consts(float inv_tau, float m) {
  Exp2Consts c;
  c.inv_tau = pack2(inv_tau, inv_tau);
  c.neg_m = pack2(-m, -m);
  c.log2e = pack2(0x1.715476p+0f, 0x1.715476p+0f);
  c.shift = pack2(12582912.0f, 12582912.0f);
  c.neg_shift = pack2(-12582912.0f, -12582912.0f);
  c.ln2_hi = pack2(-0x1.62e4p-1f, -0x1.62e4p-1f);
  c.ln2_lo = pack2(-0x1.7f7d1cp-20f, -0x1.7f7d1cp-20f);
  c.c6 = pack2(0x1.6c16c2p-10f, 0x1.6c16c2p-10f);
  c.c5 = pack2(0x1.111112p-7f, 0x1.111112p-7f);
  c.c4 = pack2(0x1.555556p-5f, 0x1.555556p-5f);
  c.c3 = pack2(0x1.555556p-3f, 0x1.555556p-3f);
  c.half = pack2(0.5f, 0.5f);
  c.one = pack2(1.0f, 1.0f);
  return c;
}
// the two scaled numerators as floats (zero below the cut-off); their truncation is the integer numerator
__device__ __forceinline__ void fixed_exp_pair_f(float z0, float z1, const Exp2Consts& c, float& s0, float& s1) {
  const unsigned long long x = add2(mul2(pack2(z0, z1), c.inv_tau), c.neg_m);   // a - m == a + (-m), rounded once
  const unsigned long long t = fma2(x, c.log2e, c.shift);
  const unsigned long long nf = add2(t, c.neg_shift);
  unsigned long long r = fma2(nf, c.ln2_hi, x);
  r = fma2(nf, c.ln2_lo, r);
  unsigned long long p = fma2(c.c6, r, c.c5);
  p = fma2(p, r, c.c4);
  p = fma2(p, r, c.c3);
  p = fma2(p, r, c.half);
  p = fma2(p, r, c.one);
  p = fma2(p, r, c.one);
  float x0, x1, t0, t1, p0, p1;
  unpack2(x, x0, x1);
  unpack2(t, t0, t1);
  unpack2(p, p0, p1);
  // bits(t) - bits(1.5 * 2^23) = n; scaled = p * 2^(n + 40) by adding (n + 40) to p's exponent field
  const uint32_t base = 0x4B400000u - 40u;
  const float f0 = __uint_as_float(__float_as_uint(p0) + ((__float_as_uint(t0) - base) << 23));
  const float f1 = __uint_as_float(__float_as_uint(p1) + ((__float_as_uint(t1) - base) << 23));
  s0 = x0 >= -30.0f ? f0 : 0.0f;
  s1 = x1 >= -30.0f ? f1 : 0.0f;
}
__device__ __forceinline__ void fixed_exp_pair(float z0, float z1, const Exp2Consts& c, unsigned long long& e0,
                                               unsigned long long& e1) {
  float s0, s1;
  fixed_exp_pair_f(z0, z1, c, s0, s1);
  e0 = __float2ull_rz(s0);
  e1 = __float2ull_rz(s1);
}

// 16-byte load with an L2 eviction policy (createpolicy): rows that will be read again are kept, rows and draft
// rows on their last reading make room first
__device__ __forceinline__ float4 ld4_policy(const float* p, uint64_t policy) {
  float4 v;
  asm volatile("ld.global.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p), "l"(policy));
  return v;
}

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// block-wide sum, result to every thread; scratch holds 32 values
template <int kThreads>
__device__ __forceinline__ unsigned long long block_sum_u64(unsigned long long v, unsigned long long* scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = warp_sum_u64(v);
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  unsigned long long t = lane < (kThreads / 32) ? scratch[lane] : 0ull;
  return warp_sum_u64(t);
}

constexpr int kMaxCluster = 8;
constexpr int kCacheBytes = 64 * 1024;        // a block's share of a row kept in shared memory (cached form)
constexpr int kStep = 32 * kVec;              // entries a warp covers per step (512 contiguous bytes of fp32)

struct Shared {
  unsigned long long sum_scratch[32];
  unsigned long long warp_tot[32];            // deciding row: sum of the weights in each warp's range
  // exchange slots, one per CTA of the cluster (written by every CTA into every CTA's copy)
  unsigned long long x_sum[2][kMaxCluster];   // Z, then W of the deciding row (double-buffered)
  float x_max[2][kMaxCluster];                // row maximum (double-buffered over rows)
  int x_idx[2][kMaxCluster];
  int x_bad[2][kMaxCluster];
  float max_scratch[32];
  int idx_scratch[32];
  int flag;
  int decision;      // 1 accepted, 0 decide here
  // what the accept test of the row in work needs besides Z, fetched while the row is being read
  float dec_z, dec_q;
  uint32_t dec_u[2];
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, int rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Entries of the vocabulary that one warp owns: the row is cut into C * kWarps contiguous ranges of `per_warp`
// entries (a multiple of kStep), block after block and warp after warp in vocabulary order.
__host__ __device__ inline int entries_per_warp(int V, int C, int warps) {
  const int64_t cut = static_cast<int64_t>(C) * warps * kStep;
  return static_cast<int>((V + cut - 1) / cut) * kStep;
}

// One cluster of C blocks per request.  Every warp owns one contiguous range of the vocabulary, so that the sum a
// warp forms over its range is one entry of a prefix structure in vocabulary order: block totals (exchanged through
// each other's shared memory), warp totals, and - for the one warp in whose range the draw falls - a scan over its
// steps.  Per examined row the blocks exchange (maximum, argmax, finiteness), then the integer sums; every block
// then takes the same decision from the same numbers.
//
// kCache (sampling, 16-byte aligned rows whose share per block fits kCacheBytes): a row is read from global memory
// once.  The first pass leaves the block's share of the logits in shared memory, the second replaces each by its
// scaled numerator (the float whose truncation is E_v), the third - on the deciding row - converts those instead of
// evaluating the exponential again.  A lane meets the same entries in every pass.
template <int kThreads, bool kCache>
__global__ void __launch_bounds__(kThreads, kThreads == 512 ? 3 : 1) accept_kernel(AcceptArgs a, int C) {
  constexpr int kWarps = kThreads / 32;
  __shared__ Shared sh;
  extern __shared__ __align__(16) float zc[];   // kCache: entries b_lo.. of the row in work
  StampScope scope(LaunchStamp{a.stamp.begin, a.stamp.end});
  pdl_enter();
  const int req = blockIdx.x / C, rank = blockIdx.x % C;
  const int row0 = a.cu_q[req];
  const int k = a.cu_q[req + 1] - row0 - 1;
  const int V = a.V;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const void* qbase = a.q_rows ? a.q_rows[req] : nullptr;   // the request's [k][V] draft rows, fp32 or bf16
  const bool q16 = a.q_bf16 != 0;
  auto q_at = [&](int64_t idx) -> float {                     // a bf16 entry widens exactly
    return q16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(qbase)[idx]) : static_cast<const float*>(qbase)[idx];
  };
  int32_t* res = a.results + 3 * req;
  const int per_warp = entries_per_warp(V, C, kWarps);
  const int64_t b_first = static_cast<int64_t>(rank) * kWarps * per_warp;
  const int b_lo = static_cast<int>(b_first < V ? b_first : V);                       // this block's range
  const int b_hi = static_cast<int>(b_first + kWarps * per_warp < V ? b_first + kWarps * per_warp : V);
  const int w_lo = min(b_hi, b_lo + warp * per_warp), w_hi = min(b_hi, w_lo + per_warp);   // this warp's range
  const bool vec = ((V & 3) == 0) && ((reinterpret_cast<uintptr_t>(a.logits) & 15) == 0);
  // the draft rows are the caller's memory: any 4-byte aligned address is legal, 16-byte loads need more
  const bool q_vec = vec && ((reinterpret_cast<uintptr_t>(qbase) & (q16 ? 7 : 15)) == 0);   // four entries per load
  int xphase = 0;   // parity of the sum exchange slots
  uint64_t pol_keep, pol_last;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_last));
  if (kCache) pol_keep = pol_last;   // a row is read from memory once

  for (int j = 0; j <= k; ++j) {
    const float* z = a.logits + static_cast<int64_t>(row0 + j) * V;
    // ---- pass 1: maximum of the scaled logits (argmax of the raw ones when greedy), finiteness
    float best = -INFINITY;
    int best_i = 0x7fffffff;
    int bad = 0;
    if (!a.greedy && threadIdx.x == 32) {          // the two uniforms of this position
      uint32_t w[4];
      philox4x32_10(static_cast<uint32_t>(a.seed), static_cast<uint32_t>(a.seed >> 32), a.ctx_lo[req], a.ctx_hi[req],
                    static_cast<uint32_t>(a.pos0[req] + j + 1), 0u, w);
      sh.dec_u[0] = w[0];
      sh.dec_u[1] = w[1];
    }
    if (!a.greedy && threadIdx.x == 64 && j < k) {   // the draft's logit and its draft probability
      const int d = a.ids[row0 + 1 + j];
      sh.dec_z = z[d];
      sh.dec_q = q_at(static_cast<int64_t>(j) * V + d);
    }
    if (vec && !a.greedy) {
      // sampling needs the maximum only, and rounding is monotone: max(z * inv_tau) = max(z) * inv_tau.  A NaN or an
      // infinity anywhere turns the running sum of z * 0 into a NaN.
      float mx = -INFINITY;
      unsigned long long nan2 = pack2(0.f, 0.f);
      const unsigned long long zero2 = pack2(0.f, 0.f);
      auto look = [&](const float4& x4) {
        mx = fmaxf(fmaxf(mx, fmaxf(x4.x, x4.y)), fmaxf(x4.z, x4.w));
        nan2 = fma2(pack2(x4.x, x4.y), zero2, nan2);
        nan2 = fma2(pack2(x4.z, x4.w), zero2, nan2);
      };
      int v = w_lo + lane * kVec;
      for (; v + 3 * kStep < w_hi; v += 4 * kStep) {
        const float4 x0 = ld4_policy(z + v, pol_keep);
        const float4 x1 = ld4_policy(z + v + kStep, pol_keep);
        const float4 x2 = ld4_policy(z + v + 2 * kStep, pol_keep);
        const float4 x3 = ld4_policy(z + v + 3 * kStep, pol_keep);
        look(x0); look(x1); look(x2); look(x3);
        if constexpr (kCache) {
          *reinterpret_cast<float4*>(zc + (v - b_lo)) = x0;
          *reinterpret_cast<float4*>(zc + (v - b_lo) + kStep) = x1;
          *reinterpret_cast<float4*>(zc + (v - b_lo) + 2 * kStep) = x2;
          *reinterpret_cast<float4*>(zc + (v - b_lo) + 3 * kStep) = x3;
        }
      }
      for (; v < w_hi; v += kStep) {
        const float4 x0 = ld4_policy(z + v, pol_keep);
        look(x0);
        if constexpr (kCache) *reinterpret_cast<float4*>(zc + (v - b_lo)) = x0;
      }
      float n0, n1;
      unpack2(nan2, n0, n1);
      bad = !(n0 == 0.f) || !(n1 == 0.f);
      best = __fmul_rn(mx, a.inv_tau);   // -inf when this lane saw no entry
      best_i = 0;                        // not used when sampling
    } else if (vec) {   // four consecutive entries per lane and step (16-byte loads), four steps in flight
      auto look = [&](int v, const float4& x4) {
        const float xs[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          bad |= !(fabsf(xs[e]) < INFINITY);
          const float sv = a.greedy ? xs[e] : __fmul_rn(xs[e], a.inv_tau);
          if (sv > best) { best = sv; best_i = v + e; }   // ascending v per lane: first maximum kept
        }
      };
      int v = w_lo + lane * kVec;
      for (; v + 3 * kStep < w_hi; v += 4 * kStep) {
        const float4 x0 = *reinterpret_cast<const float4*>(z + v);
        const float4 x1 = *reinterpret_cast<const float4*>(z + v + kStep);
        const float4 x2 = *reinterpret_cast<const float4*>(z + v + 2 * kStep);
        const float4 x3 = *reinterpret_cast<const float4*>(z + v + 3 * kStep);
        look(v, x0); look(v + kStep, x1); look(v + 2 * kStep, x2); look(v + 3 * kStep, x3);
      }
      for (; v < w_hi; v += kStep) look(v, *reinterpret_cast<const float4*>(z + v));
    } else {
      for (int v = w_lo + lane; v < w_hi; v += 32) {
        const float x = z[v];
        bad |= !(fabsf(x) < INFINITY);
        const float sv = a.greedy ? x : __fmul_rn(x, a.inv_tau);
        if (sv > best) { best = sv; best_i = v; }   // ascending v per lane: first maximum kept
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
      if (ob > best || (ob == best && oi < best_i)) { best = ob; best_i = oi; }
    }
    bad = __syncthreads_or(bad);
    if (lane == 0) { sh.max_scratch[warp] = best; sh.idx_scratch[warp] = best_i; }
    __syncthreads();
    best = lane < kWarps ? sh.max_scratch[lane] : -INFINITY;
    best_i = lane < kWarps ? sh.idx_scratch[lane] : 0x7fffffff;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
      if (ob > best || (ob == best && oi < best_i)) { best = ob; best_i = oi; }
    }
    if (C > 1) {
      const int pb = j & 1;
      if (threadIdx.x < C) {   // thread r delivers this block's triple to block r
        const int r = threadIdx.x;
        asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(map_to_rank(smem_addr(&sh.x_max[pb][rank]), r)), "f"(best) : "memory");
        asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(map_to_rank(smem_addr(&sh.x_idx[pb][rank]), r)), "r"(best_i) : "memory");
        asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(map_to_rank(smem_addr(&sh.x_bad[pb][rank]), r)), "r"(bad) : "memory");
      }
      cluster_barrier();
      best = sh.x_max[pb][0];
      best_i = sh.x_idx[pb][0];
      bad = sh.x_bad[pb][0];
      for (int r = 1; r < C; ++r) {
        const float ob = sh.x_max[pb][r];
        const int oi = sh.x_idx[pb][r];
        bad |= sh.x_bad[pb][r];
        if (ob > best || (ob == best && oi < best_i)) { best = ob; best_i = oi; }
      }
    }
    if (bad) {
      if (threadIdx.x == 0 && rank == 0) { res[0] = 0; res[1] = -1; res[2] = ST_NONFINITE; }
      return;
    }
    if (a.greedy) {
      if (j < k && a.ids[row0 + 1 + j] == best_i) continue;
      if (threadIdx.x == 0 && rank == 0) { res[0] = j; res[1] = best_i; res[2] = ST_OK; }
      return;
    }
    const float m = best;
    // ---- pass 2: Z = sum of the integer numerators
    unsigned long long zsum = 0;
    const Exp2Consts ec = exp2_consts(a.inv_tau, m);
    if constexpr (kCache) {
      // numerators from the share in shared memory; each entry is replaced by its scaled numerator
      for (int o = w_lo - b_lo + lane * kVec; o < w_hi - b_lo; o += kStep) {
        const float4 x4 = *reinterpret_cast<const float4*>(zc + o);
        float4 s4;
        fixed_exp_pair_f(x4.x, x4.y, ec, s4.x, s4.y);
        fixed_exp_pair_f(x4.z, x4.w, ec, s4.z, s4.w);
        zsum += (__float2ull_rz(s4.x) + __float2ull_rz(s4.y)) + (__float2ull_rz(s4.z) + __float2ull_rz(s4.w));
        *reinterpret_cast<float4*>(zc + o) = s4;
      }
    } else if (vec) {
      auto add4 = [&](const float4& x4) {
        unsigned long long e0, e1, e2, e3;
        fixed_exp_pair(x4.x, x4.y, ec, e0, e1);
        fixed_exp_pair(x4.z, x4.w, ec, e2, e3);
        zsum += (e0 + e1) + (e2 + e3);
      };
      int v = w_lo + lane * kVec;
      for (; v + 3 * kStep < w_hi; v += 4 * kStep) {
        const float4 x0 = *reinterpret_cast<const float4*>(z + v);
        const float4 x1 = *reinterpret_cast<const float4*>(z + v + kStep);
        const float4 x2 = *reinterpret_cast<const float4*>(z + v + 2 * kStep);
        const float4 x3 = *reinterpret_cast<const float4*>(z + v + 3 * kStep);
        add4(x0); add4(x1); add4(x2); add4(x3);
      }
      for (; v < w_hi; v += kStep) add4(*reinterpret_cast<const float4*>(z + v));
    } else {
      for (int v = w_lo + lane; v < w_hi; v += 32) zsum += fixed_exp(__fsub_rn(__fmul_rn(z[v], a.inv_tau), m));
    }
    unsigned long long Z = block_sum_u64<kThreads>(zsum, sh.sum_scratch);
    if (C > 1) {
      if (threadIdx.x < C)
        asm volatile("st.shared::cluster.b64 [%0], %1;" ::"r"(map_to_rank(smem_addr(&sh.x_sum[xphase][rank]), threadIdx.x)), "l"(Z) : "memory");
      cluster_barrier();
      Z = 0;
      for (int r = 0; r < C; ++r) Z += sh.x_sum[xphase][r];
      xphase ^= 1;
    }
    // ---- the accept test of draft j+1, or fall through on the bonus row (same numbers in every block)
    int64_t q_off = -1;     // first entry of the deciding row's draft distribution, -1: none (bonus row)
    uint32_t u_smp = 0;
    if (threadIdx.x == 0) {
      int accepted = 0;
      if (j < k) {
        const unsigned long long Ed = fixed_exp(__fsub_rn(__fmul_rn(sh.dec_z, a.inv_tau), m));
        const double lhs = __dmul_rn(__dmul_rn(static_cast<double>(sh.dec_u[0] >> 8), static_cast<double>(sh.dec_q)),
                                     __ull2double_rn(Z));
        const double rhs = __dmul_rn(__ull2double_rn(Ed), 16777216.0);
        accepted = lhs < rhs;
      }
      sh.decision = accepted;
      sh.flag = static_cast<int>(sh.dec_u[1]);
    }
    __syncthreads();
    if (sh.decision) continue;
    u_smp = static_cast<uint32_t>(sh.flag);
    if (j < k) q_off = static_cast<int64_t>(j) * V;

    // ---- deciding row: weights R_v = max(E_v - trunc(q_v * Z), 0) (or E_v), summed per warp range
    const double Zd = __ull2double_rn(Z);
    bool use_q = q_off >= 0;
    if (use_q && b_lo < b_hi) {
      // this block's share of the draft row is wanted step by step: ask for all of its lines now
      const int es = q16 ? 2 : 4;
      const char* qb = static_cast<const char*>(qbase) + (q_off + b_lo) * es;
      const int bytes = (b_hi - b_lo) * es;
      for (int b = threadIdx.x * 128; b < bytes; b += kThreads * 128)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(qb + b));
    }
    // the four weights of a lane at entries v0..v0+3 (entries from w_hi on count zero)
    auto fetch = [&](int v0, float (&zs)[kVec], float (&qs)[kVec]) {
      if (vec) {   // V % 4 == 0: a lane's four entries are inside the row together
        if constexpr (!kCache) {
          const float4 z4 = ld4_policy(z + v0, pol_last);
          zs[0] = z4.x; zs[1] = z4.y; zs[2] = z4.z; zs[3] = z4.w;
        }
        if (use_q && q_vec && !q16) {
          const float4 q4 = ld4_policy(static_cast<const float*>(qbase) + q_off + v0, pol_last);
          qs[0] = q4.x; qs[1] = q4.y; qs[2] = q4.z; qs[3] = q4.w;
        } else if (use_q && q_vec) {
          const uint2 q4 = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(qbase) + q_off + v0);
          qs[0] = __uint_as_float(q4.x << 16); qs[1] = __uint_as_float(q4.x & 0xffff0000u);
          qs[2] = __uint_as_float(q4.y << 16); qs[3] = __uint_as_float(q4.y & 0xffff0000u);
        } else if (use_q) {
#pragma unroll
          for (int e = 0; e < kVec; ++e) qs[e] = q_at(q_off + v0 + e);
        }
      } else {
#pragma unroll
        for (int e = 0; e < kVec; ++e) {
          zs[e] = v0 + e < w_hi ? z[v0 + e] : 0.f;
          qs[e] = (use_q && v0 + e < w_hi) ? q_at(q_off + v0 + e) : 0.f;
        }
      }
    };
    auto weights = [&](int v0, const float (&zs)[kVec], const float (&qs)[kVec], unsigned long long (&r)[kVec]) {
      if constexpr (kCache) {   // the scaled numerators the second pass left behind
        const float4 s4 = *reinterpret_cast<const float4*>(zc + (v0 - b_lo));
        r[0] = __float2ull_rz(s4.x); r[1] = __float2ull_rz(s4.y);
        r[2] = __float2ull_rz(s4.z); r[3] = __float2ull_rz(s4.w);
      } else {
#pragma unroll
        for (int e = 0; e < kVec; e += 2) fixed_exp_pair(zs[e], zs[e + 1], ec, r[e], r[e + 1]);
      }
#pragma unroll
      for (int e = 0; e < kVec; ++e) {
        if (use_q) {
          const unsigned long long Q = __double2ull_rz(__dmul_rn(static_cast<double>(qs[e]), Zd));
          r[e] = r[e] > Q ? r[e] - Q : 0ull;
        }
        if (v0 + e >= w_hi) r[e] = 0ull;
      }
    };
    unsigned long long W = 0, before_me = 0, mine_w = 0;
    for (int attempt = 0; attempt < 2; ++attempt) {
      unsigned long long mine = 0;
      // the loads of the next step are in flight while this one is worked on
      float zn[kVec] = {0.f, 0.f, 0.f, 0.f}, qn[kVec] = {0.f, 0.f, 0.f, 0.f};
      int v0 = w_lo + lane * kVec;
      if (v0 < w_hi) fetch(v0, zn, qn);
      for (; v0 < w_hi; v0 += kStep) {
        float zs[kVec], qs[kVec];
#pragma unroll
        for (int e = 0; e < kVec; ++e) { zs[e] = zn[e]; qs[e] = qn[e]; }
        if (v0 + kStep < w_hi) fetch(v0 + kStep, zn, qn);
        unsigned long long r[kVec];
        weights(v0, zs, qs, r);
        mine += (r[0] + r[1]) + (r[2] + r[3]);
      }
      mine = warp_sum_u64(mine);   // integer adds: any order, same sum
      __syncthreads();
      if (lane == 0) sh.warp_tot[warp] = mine;
      __syncthreads();
      mine_w = warp_sum_u64(lane < kWarps ? sh.warp_tot[lane] : 0ull);
      W = mine_w;
      before_me = 0;
      if (C > 1) {
        if (threadIdx.x < C)
          asm volatile("st.shared::cluster.b64 [%0], %1;" ::"r"(map_to_rank(smem_addr(&sh.x_sum[xphase][rank]), threadIdx.x)), "l"(mine_w) : "memory");
        cluster_barrier();
        W = 0;
        for (int r = 0; r < C; ++r) {
          if (r < rank) before_me += sh.x_sum[xphase][r];
          W += sh.x_sum[xphase][r];
        }
        xphase ^= 1;
      }
      if (W != 0 || !use_q) break;
      use_q = false;   // residual mass zero (p <= q everywhere after rounding): draw from p itself
    }
    // ---- inverse CDF: tgt = (U' * W) >> 32, first v whose running sum exceeds tgt
    const unsigned long long tgt = __umul64hi(W, static_cast<unsigned long long>(u_smp) << 32);
    if (!(before_me <= tgt && tgt < before_me + mine_w)) return;   // the crossing lies in another block's range
    unsigned long long run = before_me;
    for (int w = 0; w < warp; ++w) run += sh.warp_tot[w];
    if (!(run <= tgt && tgt < run + sh.warp_tot[warp])) return;    // ... or in another warp's
    // this warp scans its range step by step (all lanes take the same path)
    for (int base = w_lo; base < w_hi; base += kStep) {
      const int v0 = base + lane * kVec;
      unsigned long long r[kVec] = {0ull, 0ull, 0ull, 0ull};
      if (v0 < w_hi) {
        float zs[kVec] = {0.f, 0.f, 0.f, 0.f}, qs[kVec] = {0.f, 0.f, 0.f, 0.f};
        fetch(v0, zs, qs);
        weights(v0, zs, qs, r);
      }
      const unsigned long long lane_sum = (r[0] + r[1]) + (r[2] + r[3]);
      unsigned long long incl = lane_sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
      }
      const unsigned long long step_sum = __shfl_sync(0xffffffffu, incl, 31);
      if (run + step_sum > tgt) {
        unsigned long long at = run + incl - lane_sum;   // weight in front of this lane's entries
        if (at <= tgt && tgt < at + lane_sum) {          // exactly one lane sees the crossing
          int pick = v0;
#pragma unroll
          for (int e = 0; e < kVec; ++e) {
            at += r[e];
            if (at > tgt) { pick = v0 + e; break; }
          }
          res[0] = j; res[1] = pick; res[2] = ST_OK;
        }
        return;
      }
      run += step_sum;
    }
    return;
  }
}

}  // namespace

template <int kThreads, bool kCache>
static int launch_accept_t(const AcceptArgs& a, int C, cudaStream_t s) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(a.B * C, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = 0;
  if (kCache) {
    // the cached form's dynamic shared memory is above the default limit (set per device; cheap enough per launch)
    if (cudaFuncSetAttribute(accept_kernel<kThreads, kCache>, cudaFuncAttributeMaxDynamicSharedMemorySize, kCacheBytes) != cudaSuccess)
      return -1;
    cfg.dynamicSmemBytes = static_cast<size_t>(kThreads / 32) * entries_per_warp(a.V, C, kThreads / 32) * sizeof(float);
  }
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, accept_kernel<kThreads, kCache>, a, C) == cudaSuccess ? 1 : -1;
}

// Whether the cached form applies with C blocks per request: sampling, 16-byte aligned rows, and a block's share of
// a row within kCacheBytes.  (More blocks per request than occupancy asks for, only to make a row fit, measured slower
// on 512 requests: a row then costs three exchanges between eight blocks, and those, not the arithmetic, set the pace.)
template <int kThreads>
static bool cached_form_fits(const AcceptArgs& a, int C) {
  if (a.greedy || (a.V & 3) || (reinterpret_cast<uintptr_t>(a.logits) & 15)) return false;
  return static_cast<size_t>(kThreads / 32) * entries_per_warp(a.V, C, kThreads / 32) * sizeof(float) <= kCacheBytes;
}

int launch_accept(const AcceptArgs& a, cudaStream_t s) {
  if (a.B <= 0) return 0;
  static int n_sm = 0;
  if (n_sm == 0) {
    int dev = 0;
    cudaDeviceProp prop;
    n_sm = (cudaGetDevice(&dev) == cudaSuccess && cudaGetDeviceProperties(&prop, dev) == cudaSuccess) ? prop.multiProcessorCount : 1;
  }
  // Small batches: blocks of 1024 threads, as many blocks per request (a cluster) as it takes to occupy the machine.
  // Large batches: blocks of 512 threads, compiled for three per SM (one 1024-thread block fits otherwise), so that
  // several requests hide each other's latencies - and two blocks per request (measured best among 1 / 2 / 4).  Either
  // way a row stays in shared memory between the passes (the cached form) where a block's share of it fits.
  if (a.V > (1 << 30)) return -1;
  if (a.B * kMaxCluster >= 2 * n_sm) {
    constexpr int kTile = 512 * kVec;
    int C = 1;
    while (C < kMaxCluster && a.B * C < 6 * n_sm && (a.V + kTile - 1) / kTile >= 2 * C) C *= 2;
    return cached_form_fits<512>(a, C) ? launch_accept_t<512, true>(a, C, s) : launch_accept_t<512, false>(a, C, s);
  }
  constexpr int kTile = 1024 * kVec;
  int C = 1;
  while (C < kMaxCluster && a.B * C < 128 && (a.V + kTile - 1) / kTile >= 2 * C) C *= 2;
  return cached_form_fits<1024>(a, C) ? launch_accept_t<1024, true>(a, C, s) : launch_accept_t<1024, false>(a, C, s);
}

}  // namespace sled
