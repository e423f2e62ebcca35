// Fused vocabulary softmax + speculative acceptance + corrective / bonus draw.
//
// One block (or, for small batches, one thread-block cluster) per request walks its rows in
// order and stops at the deciding row: rows behind the first rejection are never read.  All quantities that decide anything are
// order-independent: the row maximum, integer softmax numerators E_v (a fixed sequence
// of correctly rounded fp32 operations followed by an exact scaling to 2^40), their
// exact 64-bit sum Z, and integer prefix sums for the inverse-CDF draw.  The accept test
// u < p/q is evaluated as U * q_d * Z < E_d * 2^24 in fp64 with U the 24-bit uniform.
#include "common.cuh"
#include "kernels.h"

namespace sled {

namespace {

constexpr int kVec = 4;                       // consecutive vocabulary entries per thread per tile
constexpr int kMaxTiles = 1024;               // vocabularies up to 4M entries

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
__device__ __forceinline__ void fixed_exp_pair(float z0, float z1, const Exp2Consts& c, unsigned long long& e0,
                                               unsigned long long& e1) {
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
  const float s0 = __uint_as_float(__float_as_uint(p0) + ((__float_as_uint(t0) - base) << 23));
  const float s1 = __uint_as_float(__float_as_uint(p1) + ((__float_as_uint(t1) - base) << 23));
  e0 = __float2ull_rz(x0 >= -30.0f ? s0 : 0.0f);
  e1 = __float2ull_rz(x1 >= -30.0f ? s1 : 0.0f);
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

struct Shared {
  unsigned long long sum_scratch[32];
  unsigned long long tile_sum[kMaxTiles];
  unsigned long long warp_pref[32];
  // exchange slots, one per CTA of the cluster (written by every CTA into every CTA's copy)
  unsigned long long x_sum[2][kMaxCluster];   // Z, then W of the deciding row (double-buffered)
  float x_max[2][kMaxCluster];                // row maximum (double-buffered over rows)
  int x_idx[2][kMaxCluster];
  int x_bad[2][kMaxCluster];
  float max_scratch[32];
  int idx_scratch[32];
  int flag;
  int decision;      // 1 accepted, 0 decide here
  int pick;
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

// One cluster of C blocks per request; block `rank` owns a contiguous run of 4096-entry vocabulary tiles.
// Per examined row the blocks exchange (maximum, argmax, finiteness), then the integer sums, through
// each other's shared memory; every block then takes the same decision from the same numbers.
template <int kThreads>
__global__ void __launch_bounds__(kThreads, kThreads == 512 ? 3 : 1) accept_kernel(AcceptArgs a, int C) {
  constexpr int kTile = kThreads * kVec;        // entries per tile: 4096 with 1024 threads, 2048 with 512
  __shared__ Shared sh;
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
  const int n_tiles = (V + kTile - 1) / kTile;
  const int tiles_per_rank = (n_tiles + C - 1) / C;
  const int tl_lo = min(n_tiles, rank * tiles_per_rank), tl_hi = min(n_tiles, tl_lo + tiles_per_rank);
  const int v_lo = tl_lo * kTile, v_hi = min(V, tl_hi * kTile);   // this block's vocabulary range
  int xphase = 0;   // parity of the sum exchange slots

  for (int j = 0; j <= k; ++j) {
    const float* z = a.logits + static_cast<int64_t>(row0 + j) * V;
    // ---- pass 1: maximum of the scaled logits (argmax of the raw ones when greedy), finiteness
    float best = -INFINITY;
    int best_i = 0x7fffffff;
    int bad = 0;
    const bool vec = ((V & 3) == 0) && ((reinterpret_cast<uintptr_t>(a.logits) & 15) == 0);
    // the draft rows are the caller's memory: any 4-byte aligned address is legal, 16-byte loads need more
    const bool q_vec = vec && ((reinterpret_cast<uintptr_t>(qbase) & (q16 ? 7 : 15)) == 0);   // four entries per load
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
      constexpr int kStep = kThreads * 4;
      int v = v_lo + threadIdx.x * 4;
      for (; v + 3 * kStep < v_hi; v += 4 * kStep) {
        const float4 x0 = *reinterpret_cast<const float4*>(z + v);
        const float4 x1 = *reinterpret_cast<const float4*>(z + v + kStep);
        const float4 x2 = *reinterpret_cast<const float4*>(z + v + 2 * kStep);
        const float4 x3 = *reinterpret_cast<const float4*>(z + v + 3 * kStep);
        look(x0); look(x1); look(x2); look(x3);
      }
      for (; v < v_hi; v += kStep) look(*reinterpret_cast<const float4*>(z + v));
      float n0, n1;
      unpack2(nan2, n0, n1);
      bad = !(n0 == 0.f) || !(n1 == 0.f);
      best = __fmul_rn(mx, a.inv_tau);   // -inf when this thread saw no entry
      best_i = 0;                        // not used when sampling
    } else if (vec) {   // four consecutive entries per thread and step (16-byte loads), four steps in flight
      auto look = [&](int v, const float4& x4) {
        const float xs[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          bad |= !(fabsf(xs[e]) < INFINITY);
          const float sv = a.greedy ? xs[e] : __fmul_rn(xs[e], a.inv_tau);
          if (sv > best) { best = sv; best_i = v + e; }   // ascending v per thread: first maximum kept
        }
      };
      constexpr int kStep = kThreads * 4;
      int v = v_lo + threadIdx.x * 4;
      for (; v + 3 * kStep < v_hi; v += 4 * kStep) {
        const float4 x0 = *reinterpret_cast<const float4*>(z + v);
        const float4 x1 = *reinterpret_cast<const float4*>(z + v + kStep);
        const float4 x2 = *reinterpret_cast<const float4*>(z + v + 2 * kStep);
        const float4 x3 = *reinterpret_cast<const float4*>(z + v + 3 * kStep);
        look(v, x0); look(v + kStep, x1); look(v + 2 * kStep, x2); look(v + 3 * kStep, x3);
      }
      for (; v < v_hi; v += kStep) look(v, *reinterpret_cast<const float4*>(z + v));
    } else {
      for (int v = v_lo + threadIdx.x; v < v_hi; v += kThreads) {
        const float x = z[v];
        bad |= !(fabsf(x) < INFINITY);
        const float sv = a.greedy ? x : __fmul_rn(x, a.inv_tau);
        if (sv > best) { best = sv; best_i = v; }   // ascending v per thread: first maximum kept
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
    best = sh.max_scratch[0];
    best_i = sh.idx_scratch[0];
    for (int w = 1; w < kThreads / 32; ++w) {
      const float ob = sh.max_scratch[w];
      const int oi = sh.idx_scratch[w];
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
    if (vec) {
      auto add4 = [&](const float4& x4) {
        unsigned long long e0, e1, e2, e3;
        fixed_exp_pair(x4.x, x4.y, ec, e0, e1);
        fixed_exp_pair(x4.z, x4.w, ec, e2, e3);
        zsum += (e0 + e1) + (e2 + e3);
      };
      constexpr int kStep = kThreads * 4;
      int v = v_lo + threadIdx.x * 4;
      for (; v + 3 * kStep < v_hi; v += 4 * kStep) {
        const float4 x0 = *reinterpret_cast<const float4*>(z + v);
        const float4 x1 = *reinterpret_cast<const float4*>(z + v + kStep);
        const float4 x2 = *reinterpret_cast<const float4*>(z + v + 2 * kStep);
        const float4 x3 = *reinterpret_cast<const float4*>(z + v + 3 * kStep);
        add4(x0); add4(x1); add4(x2); add4(x3);
      }
      for (; v < v_hi; v += kStep) add4(*reinterpret_cast<const float4*>(z + v));
    } else {
      for (int v = v_lo + threadIdx.x; v < v_hi; v += kThreads) zsum += fixed_exp(__fsub_rn(__fmul_rn(z[v], a.inv_tau), m));
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
      uint32_t w[4];
      philox4x32_10(static_cast<uint32_t>(a.seed), static_cast<uint32_t>(a.seed >> 32), a.ctx_lo[req], a.ctx_hi[req],
                    static_cast<uint32_t>(a.pos0[req] + j + 1), 0u, w);
      int accepted = 0;
      if (j < k) {
        const int d = a.ids[row0 + 1 + j];
        const unsigned long long Ed = fixed_exp(__fsub_rn(__fmul_rn(z[d], a.inv_tau), m));
        const float qd = q_at(static_cast<int64_t>(j) * V + d);
        const double lhs = __dmul_rn(__dmul_rn(static_cast<double>(w[0] >> 8), static_cast<double>(qd)),
                                     __ull2double_rn(Z));
        const double rhs = __dmul_rn(__ull2double_rn(Ed), 16777216.0);
        accepted = lhs < rhs;
      }
      sh.decision = accepted;
      sh.flag = static_cast<int>(w[1]);
    }
    __syncthreads();
    if (sh.decision) continue;
    u_smp = static_cast<uint32_t>(sh.flag);
    if (j < k) q_off = static_cast<int64_t>(j) * V;

    // ---- deciding row: weights R_v = max(E_v - trunc(q_v * Z), 0) (or E_v), tile sums in vocabulary order
    const double Zd = __ull2double_rn(Z);
    bool use_q = q_off >= 0;
    unsigned long long W = 0, before_me = 0;
    for (int attempt = 0; attempt < 2; ++attempt) {
      for (int tl = threadIdx.x; tl < n_tiles; tl += kThreads) sh.tile_sum[tl] = 0ull;
      __syncthreads();
      for (int tl = tl_lo; tl < tl_hi; ++tl) {
        unsigned long long mine = 0;
        const int v0 = tl * kTile + threadIdx.x * kVec;
        float zs[kVec], qs[kVec];
        if (vec && v0 + kVec <= V) {
          const float4 z4 = *reinterpret_cast<const float4*>(z + v0);
          zs[0] = z4.x; zs[1] = z4.y; zs[2] = z4.z; zs[3] = z4.w;
          if (use_q && q_vec && !q16) {
            const float4 q4 = *reinterpret_cast<const float4*>(static_cast<const float*>(qbase) + q_off + v0);
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
            zs[e] = v0 + e < V ? z[v0 + e] : 0.f;
            qs[e] = (use_q && v0 + e < V) ? q_at(q_off + v0 + e) : 0.f;
          }
        }
        unsigned long long Es[kVec];
#pragma unroll
        for (int e = 0; e < kVec; e += 2) fixed_exp_pair(zs[e], zs[e + 1], ec, Es[e], Es[e + 1]);
#pragma unroll
        for (int e = 0; e < kVec; ++e) {
          if (v0 + e < V) {
            unsigned long long E = Es[e];
            if (use_q) {
              const unsigned long long Q = __double2ull_rz(__dmul_rn(static_cast<double>(qs[e]), Zd));
              E = E > Q ? E - Q : 0ull;
            }
            mine += E;
          }
        }
        mine = warp_sum_u64(mine);
        if (lane == 0 && mine) atomicAdd(&sh.tile_sum[tl], mine);  // integer adds: any order, same sum
      }
      __syncthreads();
      unsigned long long mine_w = 0;
      for (int tl = tl_lo; tl < tl_hi; ++tl) mine_w += sh.tile_sum[tl];
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
      __syncthreads();
    }
    // ---- inverse CDF: tgt = (U' * W) >> 32, first v whose running sum exceeds tgt
    const unsigned long long tgt = __umul64hi(W, static_cast<unsigned long long>(u_smp) << 32);
    unsigned long long my_w = 0;
    for (int tl = tl_lo; tl < tl_hi; ++tl) my_w += sh.tile_sum[tl];
    if (!(before_me <= tgt && tgt < before_me + my_w)) return;   // the crossing lies in another block's range
    int tl_hit = tl_lo;
    unsigned long long before = before_me;
    for (int tl = tl_lo; tl < tl_hi; ++tl) {
      const unsigned long long nx = before + sh.tile_sum[tl];
      if (nx > tgt) { tl_hit = tl; break; }
      before = nx;
      tl_hit = tl;
    }
    unsigned long long r[kVec];
    unsigned long long mine = 0;
    {
      const int v0 = tl_hit * kTile + threadIdx.x * kVec;
#pragma unroll
      for (int e = 0; e < kVec; ++e) {
        const int v = v0 + e;
        unsigned long long E = 0;
        if (v < V) {
          E = fixed_exp(__fsub_rn(__fmul_rn(z[v], a.inv_tau), m));
          if (use_q) {
            const unsigned long long Q = __double2ull_rz(__dmul_rn(static_cast<double>(q_at(q_off + v)), Zd));
            E = E > Q ? E - Q : 0ull;
          }
        }
        r[e] = E;
        mine += E;
      }
    }
    // exclusive prefix of `mine` over the block in thread order
    unsigned long long incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += up;
    }
    __syncthreads();
    if (lane == 31) sh.warp_pref[warp] = incl;
    if (threadIdx.x == 0) sh.pick = V - 1;
    __syncthreads();
    unsigned long long run = before + incl - mine;
    for (int w = 0; w < warp; ++w) run += sh.warp_pref[w];
    // exactly one thread sees the crossing
    if (run <= tgt && run + mine > tgt) {
      int pick = tl_hit * kTile + threadIdx.x * kVec;
#pragma unroll
      for (int e = 0; e < kVec; ++e) {
        run += r[e];
        if (run > tgt) { pick += e; break; }
      }
      sh.pick = pick;
    }
    __syncthreads();
    if (threadIdx.x == 0) { res[0] = j; res[1] = sh.pick; res[2] = ST_OK; }
    return;
  }
}

}  // namespace

template <int kThreads>
static int launch_accept_t(const AcceptArgs& a, int C, cudaStream_t s) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(a.B * C, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = 0;
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
  return cudaLaunchKernelEx(&cfg, accept_kernel<kThreads>, a, C) == cudaSuccess ? 1 : -1;
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
  // several requests hide each other's latencies - and two blocks per request (measured best among 1 / 2 / 4).
  if (a.B * kMaxCluster >= 2 * n_sm && a.V <= 512 * kVec * kMaxTiles) {
    constexpr int kTile = 512 * kVec;
    int C = 1;
    while (C < kMaxCluster && a.B * C < 6 * n_sm && (a.V + kTile - 1) / kTile >= 2 * C) C *= 2;
    return launch_accept_t<512>(a, C, s);
  }
  constexpr int kTile = 1024 * kVec;
  if (a.V > kTile * kMaxTiles) return -1;
  int C = 1;
  while (C < kMaxCluster && a.B * C < 128 && (a.V + kTile - 1) / kTile >= 2 * C) C *= 2;
  return launch_accept_t<1024>(a, C, s);
}

}  // namespace sled
