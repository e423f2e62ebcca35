// Small kernels of the verification step: token embedding, residual-add + RMSNorm,
// rotary embedding with the write of new keys/values into their cache pages, SwiGLU,
// cache scatter/gather, and the CUDA-core GEMM used by the fp32 configuration.
// The linear layers leave split-K partial sums behind; the kernel that consumes a
// linear layer's output adds them up, in a fixed order, while it does its own work.
#include "common.cuh"
#include "fp8_split.cuh"
#include "kernels.h"

namespace sled {

static inline LaunchStamp dev_stamp(const Stamp& st) { return LaunchStamp{st.begin, st.end}; }

// ------------------------------------------------------------------ embedding --
template <typename WT>
__global__ void embed_kernel(const WT* __restrict__ table, const int32_t* __restrict__ ids, int d, float* __restrict__ x,
                             LaunchStamp stamp) {
  StampScope scope(stamp);
  pdl_enter();
  const int t = blockIdx.x;
  const WT* row = table + static_cast<int64_t>(ids[t]) * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x) x[static_cast<int64_t>(t) * d + i] = to_f32(row[i]);
}

int launch_embed(const void* table, int wdtype, const int32_t* ids, int T, int d, float* x, cudaStream_t s, Stamp st) {
  if (T <= 0) return 0;
  if (wdtype == BF16)
    SLED_LAUNCH_PDL(embed_kernel<__nv_bfloat16>, dim3(T), dim3(256), 0, s, static_cast<const __nv_bfloat16*>(table), ids, d, x, dev_stamp(st));
  else
    SLED_LAUNCH_PDL(embed_kernel<float>, dim3(T), dim3(256), 0, s, static_cast<const float*>(table), ids, d, x, dev_stamp(st));
  return 1;
}

// ------------------------------------------------------- residual add + RMSNorm --
// One block per token.  x (fp32 residual stream) is updated in place with the split-K
// partial sums of the preceding linear layer, then normalised:
//   y_i = x_i * rsqrt(mean(x^2) + eps) * g_i
template <typename WT, typename AT>
__global__ void add_rmsnorm_kernel(float* __restrict__ x, const float* __restrict__ partial, int n_split,
                                   int64_t split_stride, const WT* __restrict__ gain, float eps, int d,
                                   AT* __restrict__ out, LaunchStamp stamp) {
  __shared__ float scratch[32];
  StampScope scope(stamp);
  pdl_enter();
  const int64_t base = static_cast<int64_t>(blockIdx.x) * d;
  float ss = 0.f;
  // four consecutive features per thread and pass; the slices of a feature are summed in slice order
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    float4 v = *reinterpret_cast<const float4*>(x + base + i);
#pragma unroll 8
    for (int sp = 0; sp < n_split; ++sp) {
      const float4 p = __ldcg(reinterpret_cast<const float4*>(partial + sp * split_stride + base + i));
      v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
    }
    if (n_split > 0) *reinterpret_cast<float4*>(x + base + i) = v;
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = block_sum(ss, scratch);
  const float scale = rsqrtf(ss / static_cast<float>(d) + eps);
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {  // each thread re-reads what it wrote itself
    const float4 v = *reinterpret_cast<const float4*>(x + base + i);
    out[base + i] = from_f32<AT>(v.x * scale * to_f32(gain[i]));
    out[base + i + 1] = from_f32<AT>(v.y * scale * to_f32(gain[i + 1]));
    out[base + i + 2] = from_f32<AT>(v.z * scale * to_f32(gain[i + 2]));
    out[base + i + 3] = from_f32<AT>(v.w * scale * to_f32(gain[i + 3]));
  }
}

// The same with bf16 gains and outputs for rows of at most four features per thread, which stay in registers, and
// the outputs written a second time as two e4m3 parts per element plus the token's scale (the operand format of the
// fp8 linear layers): hi rows at out8[t], lo rows at out8[lo_row0 + t].
__global__ void add_rmsnorm_split_kernel(float* __restrict__ x, const float* __restrict__ partial, int n_split,
                                         int64_t split_stride, const __nv_bfloat16* __restrict__ gain, float eps, int d,
                                         __nv_bfloat16* __restrict__ out, uint8_t* __restrict__ out8, int lo_row0,
                                         float* __restrict__ scale8, LaunchStamp stamp) {
  __shared__ float scratch[32];
  StampScope scope(stamp);
  pdl_enter();
  const int64_t base = static_cast<int64_t>(blockIdx.x) * d;
  const int i = threadIdx.x * 4;
  const bool mine = i < d;
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (mine) {
    v = *reinterpret_cast<const float4*>(x + base + i);
#pragma unroll 8
    for (int sp = 0; sp < n_split; ++sp) {
      const float4 p = __ldcg(reinterpret_cast<const float4*>(partial + sp * split_stride + base + i));
      v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
    }
    if (n_split > 0) *reinterpret_cast<float4*>(x + base + i) = v;
  }
  const float ss = block_sum(v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w, scratch);
  const float scale = rsqrtf(ss / static_cast<float>(d) + eps);
  float y[4] = {0.f, 0.f, 0.f, 0.f};
  if (mine) {
    const float vv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const __nv_bfloat16 r = __float2bfloat16_rn(vv[j] * scale * __bfloat162float(gain[i + j]));
      out[base + i + j] = r;
      y[j] = __bfloat162float(r);
    }
  }
  // the row's largest output: a maximum is a sum in the (max, +) sense, and exact in any order
  float amax = fmaxf(fmaxf(fabsf(y[0]), fabsf(y[1])), fmaxf(fabsf(y[2]), fabsf(y[3])));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = 0.f;
  for (int w = 0; w < (blockDim.x + 31) / 32; ++w) amax = fmaxf(amax, scratch[w]);
  const float s8 = token_scale_e4m3(amax);
  const float inv = 1.f / s8;
  if (threadIdx.x == 0) scale8[blockIdx.x] = s8;
  if (mine) {
    uint32_t h0, l0, h1, l1;
    split_pair_e4m3(y[0] * inv, y[1] * inv, h0, l0);
    split_pair_e4m3(y[2] * inv, y[3] * inv, h1, l1);
    *reinterpret_cast<uint32_t*>(out8 + static_cast<int64_t>(blockIdx.x) * d + i) = h0 | (h1 << 16);
    *reinterpret_cast<uint32_t*>(out8 + static_cast<int64_t>(lo_row0 + blockIdx.x) * d + i) = l0 | (l1 << 16);
  }
}

int launch_add_rmsnorm(float* x, const float* partial, int n_split, int64_t split_stride, const void* gain, int wdtype,
                       float eps, int T, int d, void* out, int adtype, cudaStream_t s, Stamp st, uint8_t* out8, int lo_row0,
                       float* scale8, bool* split_done) {
  if (split_done) *split_done = false;
  if (T <= 0) return 0;
  if (!partial) n_split = 0;
  int nt = d >= 4096 ? 1024 : (d >= 2048 ? 512 : 256);   // d is a multiple of 8 (checked at init)
  // many tokens: smaller blocks, so that all of them are resident at once (2048 threads per SM) instead of running
  // as a full wave followed by a short one
  static int n_sm = 0;
  if (n_sm == 0) {
    int dev = 0;
    cudaDeviceProp prop;
    n_sm = (cudaGetDevice(&dev) == cudaSuccess && cudaGetDeviceProperties(&prop, dev) == cudaSuccess) ? prop.multiProcessorCount : 1;
  }
  while (nt > 128 && static_cast<long long>(T) * nt > 2048LL * n_sm) nt /= 2;
  if (out8 && scale8 && wdtype == BF16 && adtype == BF16 && d <= 4 * nt && d % 4 == 0) {
    SLED_LAUNCH_PDL(add_rmsnorm_split_kernel, dim3(T), dim3(nt), 0, s, x, partial, n_split, split_stride,
                    static_cast<const __nv_bfloat16*>(gain), eps, d, static_cast<__nv_bfloat16*>(out), out8, lo_row0, scale8, dev_stamp(st));
    if (split_done) *split_done = true;
    return 1;
  }
  if (wdtype == BF16 && adtype == BF16)
    SLED_LAUNCH_PDL((add_rmsnorm_kernel<__nv_bfloat16, __nv_bfloat16>), dim3(T), dim3(nt), 0, s, x, partial, n_split,
                    split_stride, static_cast<const __nv_bfloat16*>(gain), eps, d, static_cast<__nv_bfloat16*>(out), dev_stamp(st));
  else if (wdtype == F32 && adtype == F32)
    SLED_LAUNCH_PDL((add_rmsnorm_kernel<float, float>), dim3(T), dim3(nt), 0, s, x, partial, n_split, split_stride,
                    static_cast<const float*>(gain), eps, d, static_cast<float*>(out), dev_stamp(st));
  else
    return -1;
  return 1;
}

// --------------------------------------------------------------- rotary table --
// cs[t][i] = (cos, sin)(pos_t * theta^(-2i/h)), angle and functions in fp64, stored fp32;
// computed once per step and shared by all layers and heads.
__global__ void rope_table_kernel(const int32_t* __restrict__ tok_pos, int h, double log2_theta, float2* __restrict__ cs,
                                  LaunchStamp stamp) {
  StampScope scope(stamp);
  pdl_enter();
  const int t = blockIdx.x, i = threadIdx.x;
  if (i >= h / 2) return;
  const double inv_freq = exp2(-2.0 * static_cast<double>(i) / static_cast<double>(h) * log2_theta);
  double sn, c;
  sincos(static_cast<double>(tok_pos[t]) * inv_freq, &sn, &c);
  cs[static_cast<int64_t>(t) * (h / 2) + i] = make_float2(static_cast<float>(c), static_cast<float>(sn));
}

int launch_rope_table(const int32_t* tok_pos, int T, int h, float theta, float2* cs, cudaStream_t s, Stamp st) {
  if (T <= 0) return 0;
  SLED_LAUNCH_PDL(rope_table_kernel, dim3(T), dim3(h / 2), 0, s, tok_pos, h, log2(static_cast<double>(theta)), cs, dev_stamp(st));
  return 1;
}

// ------------------------------------------------------ RoPE + cache write --
// grid (T, (Hq + 2 Hkv) / 4), blocks of (h/2, 4) threads: thread (i, y) owns the pair (2i, 2i+1) of one head.
// Cache layout of one layer: [page][Hkv][page_size][h]; slot = page * page_size + offset.
template <typename AT, typename KT>
__global__ void rope_kv_kernel(const float* __restrict__ partial, int n_split, int64_t split_stride,
                               const float2* __restrict__ cs, const int32_t* __restrict__ tok_slot, int Hq, int Hkv,
                               int h, int page_size, AT* __restrict__ q_out, KT* __restrict__ kpool,
                               KT* __restrict__ vpool, LaunchStamp stamp) {
  StampScope scope(stamp);
  pdl_enter();
  const int t = blockIdx.x, head = blockIdx.y * blockDim.y + threadIdx.y, i = threadIdx.x;
  if (head >= Hq + 2 * Hkv) return;
  const int n_cols = (Hq + 2 * Hkv) * h;
  const int64_t src = static_cast<int64_t>(t) * n_cols + head * h + 2 * i;
  float a = 0.f, b = 0.f;
#pragma unroll 8
  for (int sp = 0; sp < n_split; ++sp) {
    const float2 v = __ldcg(reinterpret_cast<const float2*>(partial + sp * split_stride + src));
    a += v.x;
    b += v.y;
  }
  if (head < Hq + Hkv) {
    const float2 c = cs[static_cast<int64_t>(t) * (h / 2) + i];
    const float ra = a * c.x - b * c.y, rb = a * c.y + b * c.x;
    a = ra;
    b = rb;
  }
  if (head < Hq) {
    AT* dst = q_out + (static_cast<int64_t>(t) * Hq + head) * h + 2 * i;
    dst[0] = from_f32<AT>(a);
    dst[1] = from_f32<AT>(b);
  } else {
    const bool is_k = head < Hq + Hkv;
    const int kvh = is_k ? head - Hq : head - Hq - Hkv;
    const int slot = tok_slot[t];
    const int64_t off = ((static_cast<int64_t>(slot / page_size) * Hkv + kvh) * page_size + slot % page_size) * h + 2 * i;
    KT* dst = (is_k ? kpool : vpool) + off;
    dst[0] = from_f32<KT>(a);
    dst[1] = from_f32<KT>(b);
  }
}

int launch_rope_kv(const float* partial, int n_split, int64_t split_stride, const float2* cs, const int32_t* tok_slot,
                   int T, int Hq, int Hkv, int h, int page_size, void* q_out, int adtype, void* kpool, void* vpool,
                   int kvdtype, cudaStream_t s, Stamp st) {
  if (T <= 0) return 0;
  dim3 grid(T, (Hq + 2 * Hkv + 3) / 4);
  if (adtype == BF16 && kvdtype == BF16)
    SLED_LAUNCH_PDL((rope_kv_kernel<__nv_bfloat16, __nv_bfloat16>), grid, dim3(h / 2, 4), 0, s, partial, n_split, split_stride, cs, tok_slot,
                    Hq, Hkv, h, page_size, static_cast<__nv_bfloat16*>(q_out), static_cast<__nv_bfloat16*>(kpool), static_cast<__nv_bfloat16*>(vpool), dev_stamp(st));
  else if (adtype == F32 && kvdtype == F32)
    SLED_LAUNCH_PDL((rope_kv_kernel<float, float>), grid, dim3(h / 2, 4), 0, s, partial, n_split, split_stride, cs, tok_slot,
                    Hq, Hkv, h, page_size, static_cast<float*>(q_out), static_cast<float*>(kpool), static_cast<float*>(vpool), dev_stamp(st));
  else if (adtype == F32 && kvdtype == BF16)
    SLED_LAUNCH_PDL((rope_kv_kernel<float, __nv_bfloat16>), grid, dim3(h / 2, 4), 0, s, partial, n_split, split_stride, cs, tok_slot,
                    Hq, Hkv, h, page_size, static_cast<float*>(q_out), static_cast<__nv_bfloat16*>(kpool), static_cast<__nv_bfloat16*>(vpool), dev_stamp(st));
  else
    return -1;
  return 1;
}

// --------------------------------------------------------------------- SwiGLU --
// partial: [split][T][2F], gate and up interleaved (columns 2f and 2f+1):  out = silu(gate) * up
template <typename AT>
__global__ void swiglu_kernel(const float* __restrict__ partial, int n_split, int64_t split_stride, int F,
                              AT* __restrict__ out, LaunchStamp stamp) {
  StampScope scope(stamp);
  pdl_enter();
  const int t = blockIdx.y;
  const int f = blockIdx.x * blockDim.x + threadIdx.x;
  if (f >= F) return;
  const int64_t row = static_cast<int64_t>(t) * 2 * F;
  float g = 0.f, u = 0.f;
  for (int sp = 0; sp < n_split; ++sp) {
    const float2 gu = __ldcg(reinterpret_cast<const float2*>(partial + sp * split_stride + row + 2 * f));
    g += gu.x;
    u += gu.y;
  }
  out[static_cast<int64_t>(t) * F + f] = from_f32<AT>(g / (1.f + __expf(-g)) * u);
}

int launch_swiglu(const float* partial, int n_split, int64_t split_stride, int T, int F, void* out, int adtype,
                  cudaStream_t s, Stamp st) {
  if (T <= 0) return 0;
  dim3 grid((F + 255) / 256, T);
  if (adtype == BF16)
    SLED_LAUNCH_PDL(swiglu_kernel<__nv_bfloat16>, grid, dim3(256), 0, s, partial, n_split, split_stride, F, static_cast<__nv_bfloat16*>(out), dev_stamp(st));
  else
    SLED_LAUNCH_PDL(swiglu_kernel<float>, grid, dim3(256), 0, s, partial, n_split, split_stride, F, static_cast<float*>(out), dev_stamp(st));
  return 1;
}

// -------------------------------------------------- cache scatter / gather --
template <typename KT, bool TO_POOL>
__global__ void kv_move_kernel(KT* __restrict__ pool, KT* __restrict__ flat, const int32_t* __restrict__ slots, int Hkv,
                               int h, int page_size) {
  const int n = blockIdx.x, kvh = blockIdx.y;
  const int slot = slots[n];
  const int64_t po = ((static_cast<int64_t>(slot / page_size) * Hkv + kvh) * page_size + slot % page_size) * h;
  const int64_t fo = (static_cast<int64_t>(n) * Hkv + kvh) * h;
  for (int i = threadIdx.x; i < h; i += blockDim.x) {
    if (TO_POOL) pool[po + i] = flat[fo + i];
    else flat[fo + i] = pool[po + i];
  }
}

int launch_kv_scatter(const void* src, const int32_t* slots, int n, int Hkv, int h, int page_size, void* pool,
                      int kvdtype, cudaStream_t s) {
  if (n <= 0) return 0;
  dim3 grid(n, Hkv);
  if (kvdtype == BF16)
    kv_move_kernel<__nv_bfloat16, true><<<grid, 64, 0, s>>>(static_cast<__nv_bfloat16*>(pool),
        const_cast<__nv_bfloat16*>(static_cast<const __nv_bfloat16*>(src)), slots, Hkv, h, page_size);
  else
    kv_move_kernel<float, true><<<grid, 64, 0, s>>>(static_cast<float*>(pool),
        const_cast<float*>(static_cast<const float*>(src)), slots, Hkv, h, page_size);
  return 1;
}

int launch_kv_gather(const void* pool, const int32_t* slots, int n, int Hkv, int h, int page_size, void* dst,
                     int kvdtype, cudaStream_t s) {
  if (n <= 0) return 0;
  dim3 grid(n, Hkv);
  if (kvdtype == BF16)
    kv_move_kernel<__nv_bfloat16, false><<<grid, 64, 0, s>>>(
        const_cast<__nv_bfloat16*>(static_cast<const __nv_bfloat16*>(pool)), static_cast<__nv_bfloat16*>(dst), slots,
        Hkv, h, page_size);
  else
    kv_move_kernel<float, false><<<grid, 64, 0, s>>>(const_cast<float*>(static_cast<const float*>(pool)),
                                                     static_cast<float*>(dst), slots, Hkv, h, page_size);
  return 1;
}

// ------------------------------------------------------------ CUDA-core GEMM --
// out[z][t][n] = sum over the z-th K slice of A[t][k] * W[n][k], fp32 accumulation.
// 32 x 64 output tile per block of 256 threads (2 x 4 outputs per thread), K step 32.
template <typename AT, typename WT>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const AT* __restrict__ A, const WT* __restrict__ W, int T, int N,
                                                        int K, int k_per_split, float* __restrict__ out,
                                                        int64_t split_stride, LaunchStamp stamp) {
  StampScope scope(stamp);
  pdl_enter();
  constexpr int BM = 32, BN = 64, BK = 32;
  __shared__ float As[BK][BM + 1];
  __shared__ float Ws[BK][BN + 1];
  const int t0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int k_begin = blockIdx.z * k_per_split, k_end = min(K, k_begin + k_per_split);
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;  // tx -> 4 columns, ty -> 2 rows
  float acc[2][4] = {};
  for (int k0 = k_begin; k0 < k_end; k0 += BK) {
    for (int e = threadIdx.x; e < BM * BK; e += 256) {
      const int m = e / BK, kk = e % BK;
      const int t = t0 + m, k = k0 + kk;
      As[kk][m] = (t < T && k < k_end) ? to_f32(A[static_cast<int64_t>(t) * K + k]) : 0.f;
    }
    for (int e = threadIdx.x; e < BN * BK; e += 256) {
      const int n = e / BK, kk = e % BK;
      const int nn = n0 + n, k = k0 + kk;
      Ws[kk][n] = (nn < N && k < k_end) ? to_f32(W[static_cast<int64_t>(nn) * K + k]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[2], w[4];
#pragma unroll
      for (int i = 0; i < 2; ++i) a[i] = As[kk][ty * 2 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) w[j] = Ws[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
  float* o = out + blockIdx.z * split_stride;
  for (int i = 0; i < 2; ++i)
    for (int j = 0; j < 4; ++j) {
      const int t = t0 + ty * 2 + i, n = n0 + tx * 4 + j;
      if (t < T && n < N) o[static_cast<int64_t>(t) * N + n] = acc[i][j];
    }
}

int launch_gemm_simt(const void* A, int adtype, const void* W, int wdtype, int T, int N, int K, int n_split,
                     float* out, int64_t split_stride, cudaStream_t s, Stamp st) {
  if (T <= 0) return 0;
  if (n_split < 1) n_split = 1;
  int k_per_split = ((K + n_split - 1) / n_split + 31) / 32 * 32;
  dim3 grid((N + 63) / 64, (T + 31) / 32, n_split);
  if (adtype == F32 && wdtype == F32)
    SLED_LAUNCH_PDL((gemm_simt_kernel<float, float>), grid, dim3(256), 0, s, static_cast<const float*>(A),
                    static_cast<const float*>(W), T, N, K, k_per_split, out, split_stride, dev_stamp(st));
  else if (adtype == BF16 && wdtype == BF16)
    SLED_LAUNCH_PDL((gemm_simt_kernel<__nv_bfloat16, __nv_bfloat16>), grid, dim3(256), 0, s,
                    static_cast<const __nv_bfloat16*>(A), static_cast<const __nv_bfloat16*>(W), T, N, K, k_per_split, out,
                    split_stride, dev_stamp(st));
  else
    return -1;
  return 1;
}

}  // namespace sled
