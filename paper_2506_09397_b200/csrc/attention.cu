// Ragged verification attention over the paged KV cache.
//
// A verification request brings q_len = k+1 new tokens; query j attends to the whole
// cached prefix and, causally, to the new tokens 0..j.  With grouped-query attention the
// q_len * (Hq/Hkv) query rows that share one KV head are processed together, so each
// cached key/value is fetched once per work item.  Work items are (request, KV head,
// chunk of keys): long contexts are split over several blocks and their partial results
// (running maximum, normaliser, unnormalised output) merged afterwards.
//
// This file holds the CUDA-core kernel (any storage type, used by the fp32
// configuration) and the merge kernel.
#include "common.cuh"
#include "fp8_split.cuh"
#include "kernels.h"

namespace sled {

namespace {

constexpr int kTileKeys = 32;
constexpr int kRowsPerPass = 64;  // 256 threads, 4 per query row

template <typename KT> __device__ __forceinline__ void load_row_chunk(const KT* src, float* dst);
// 16 bytes of a cache row -> shared floats
template <> __device__ __forceinline__ void load_row_chunk<float>(const float* src, float* dst) {
  const float4 v = *reinterpret_cast<const float4*>(src);
  dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
}
template <> __device__ __forceinline__ void load_row_chunk<__nv_bfloat16>(const __nv_bfloat16* src, float* dst) {
  const uint4 v = *reinterpret_cast<const uint4*>(src);
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    dst[2 * i] = __uint_as_float(w[i] << 16);
    dst[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

template <typename KT, typename AT, int H>
__global__ void __launch_bounds__(256) attn_simt_kernel(AttnArgs a) {
  constexpr int DPT = H / 4;       // head dims per thread
  constexpr int NCH = DPT / 4;     // float4 chunks per thread; thread part p owns chunks p + 4c
  constexpr int EPV = 16 / sizeof(KT);  // storage elements per 16-byte load
  __shared__ __align__(16) float Ks[kTileKeys][H];
  __shared__ __align__(16) float Vs[kTileKeys][H];
  StampScope scope(LaunchStamp{a.stamp.begin, a.stamp.end});
  pdl_enter();

  const int4 item = a.items[blockIdx.x];
  const int req = item.x, kvh = item.y, key_start = item.z, key_count = item.w;
  const int group = a.Hq / a.Hkv;
  const int row0 = a.cu_q[req], q_len = a.cu_q[req + 1] - row0;
  const int n_rows = q_len * group;
  const int kv_base = a.kv_base[req];
  const int32_t* pages = a.page_table + a.pt_off[req];
  const KT* kpool = static_cast<const KT*>(a.kpool);
  const KT* vpool = static_cast<const KT*>(a.vpool);
  const AT* qbuf = static_cast<const AT*>(a.q);
  const bool split = a.req_chunks[req] > 1;
  const int chunk_idx = key_start / a.req_chunk_keys[req];
  const float scale = rsqrtf(static_cast<float>(H)) * 1.4426950408889634f;  // scores in log2 units

  const int part = threadIdx.x & 3;
  for (int rbase = 0; rbase < n_rows; rbase += kRowsPerPass) {
    const int r = rbase + (threadIdx.x >> 2);
    const bool valid = r < n_rows;
    const int j = valid ? r / group : 0;
    const int head = kvh * group + (valid ? r % group : 0);
    const int t = row0 + j;
    float q[DPT], o[DPT];
    {
      const AT* qrow = qbuf + (static_cast<int64_t>(t) * a.Hq + head) * H;
#pragma unroll
      for (int c = 0; c < NCH; ++c)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          q[c * 4 + e] = valid ? to_f32(qrow[(part + 4 * c) * 4 + e]) * scale : 0.f;
          o[c * 4 + e] = 0.f;
        }
    }
    float m = -INFINITY, l = 0.f;
    const int last_visible = kv_base + j;  // highest key index this query may see

    for (int tile = 0; tile < key_count; tile += kTileKeys) {
      __syncthreads();
      // cooperative load of up to 32 keys and values of this KV head
      for (int e = threadIdx.x; e < kTileKeys * (H / EPV); e += blockDim.x) {
        const int kr = e / (H / EPV), cv = e % (H / EPV);
        const int kk = key_start + tile + kr;
        if (tile + kr < key_count) {
          const int page = pages[kk / a.page_size];
          const int64_t off = ((static_cast<int64_t>(page) * a.Hkv + kvh) * a.page_size + kk % a.page_size) * H + cv * EPV;
          load_row_chunk<KT>(kpool + off, &Ks[kr][cv * EPV]);
          load_row_chunk<KT>(vpool + off, &Vs[kr][cv * EPV]);
        } else {
          // past the chunk: these rows are masked below, but their probability 0 still multiplies what is stored
          // here, and shared memory left by an earlier block may hold NaN
#pragma unroll
          for (int z = 0; z < EPV; ++z) { Ks[kr][cv * EPV + z] = 0.f; Vs[kr][cv * EPV + z] = 0.f; }
        }
      }
      __syncthreads();
      const int n_here = min(kTileKeys, key_count - tile);
      float s[kTileKeys];
      float tmax = -INFINITY;
#pragma unroll
      for (int kr = 0; kr < kTileKeys; ++kr) {
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
          const float4 kv4 = *reinterpret_cast<const float4*>(&Ks[kr][(part + 4 * c) * 4]);
          dot = fmaf(q[c * 4 + 0], kv4.x, dot);
          dot = fmaf(q[c * 4 + 1], kv4.y, dot);
          dot = fmaf(q[c * 4 + 2], kv4.z, dot);
          dot = fmaf(q[c * 4 + 3], kv4.w, dot);
        }
        dot += __shfl_xor_sync(0xffffffffu, dot, 1);
        dot += __shfl_xor_sync(0xffffffffu, dot, 2);
        const bool seen = kr < n_here && (key_start + tile + kr) <= last_visible;
        s[kr] = seen ? dot : -INFINITY;
        tmax = fmaxf(tmax, s[kr]);
      }
      const float m_new = fmaxf(m, tmax);
      if (m_new == -INFINITY) continue;  // nothing visible yet (uniform over the 4 threads of a row)
      const float alpha = exp2f(m - m_new);
      l *= alpha;
#pragma unroll
      for (int d = 0; d < DPT; ++d) o[d] *= alpha;
#pragma unroll
      for (int kr = 0; kr < kTileKeys; ++kr) {
        const float p = exp2f(s[kr] - m_new);  // 0 for masked keys
        l += p;
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
          const float4 vv = *reinterpret_cast<const float4*>(&Vs[kr][(part + 4 * c) * 4]);
          o[c * 4 + 0] = fmaf(p, vv.x, o[c * 4 + 0]);
          o[c * 4 + 1] = fmaf(p, vv.y, o[c * 4 + 1]);
          o[c * 4 + 2] = fmaf(p, vv.z, o[c * 4 + 2]);
          o[c * 4 + 3] = fmaf(p, vv.w, o[c * 4 + 3]);
        }
      }
      m = m_new;
    }

    if (valid) {
      if (!split) {
        const float inv = 1.f / l;
        AT* orow = static_cast<AT*>(a.out) + (static_cast<int64_t>(t) * a.Hq + head) * H;
#pragma unroll
        for (int c = 0; c < NCH; ++c)
#pragma unroll
          for (int e = 0; e < 4; ++e) orow[(part + 4 * c) * 4 + e] = from_f32<AT>(o[c * 4 + e] * inv);
      } else {
        const int64_t prow = static_cast<int64_t>(a.tok_part[t] + chunk_idx) * a.Hq + head;
        float* dst = a.part_acc + prow * H;
#pragma unroll
        for (int c = 0; c < NCH; ++c)
          *reinterpret_cast<float4*>(dst + (part + 4 * c) * 4) =
              make_float4(o[c * 4 + 0], o[c * 4 + 1], o[c * 4 + 2], o[c * 4 + 3]);
        if (part == 0) {
          a.part_ml[prow * 2] = m;
          a.part_ml[prow * 2 + 1] = l;
        }
      }
    }
  }
}

// Merge of the per-chunk partial results of split requests: grid (T, Hq), h threads.
template <typename AT>
__global__ void attn_merge_kernel(AttnArgs a) {
  StampScope scope(LaunchStamp{a.stamp_merge.begin, a.stamp_merge.end});
  pdl_enter();
  const int t = blockIdx.x, head = blockIdx.y, i = threadIdx.x;
  const int n = a.req_chunks[a.tok_req[t]];
  if (n <= 1) return;
  const int64_t first = static_cast<int64_t>(a.tok_part[t]);
  float M = -INFINITY;
  for (int c = 0; c < n; ++c) M = fmaxf(M, a.part_ml[((first + c) * a.Hq + head) * 2]);
  float num = 0.f, den = 0.f;
  for (int c = 0; c < n; ++c) {
    const int64_t prow = (first + c) * a.Hq + head;
    const float mc = a.part_ml[prow * 2];
    if (mc == -INFINITY) continue;  // this chunk held no visible key
    const float w = exp2f(mc - M);
    den = fmaf(w, a.part_ml[prow * 2 + 1], den);
    num = fmaf(w, a.part_acc[prow * a.h + i], num);
  }
  static_cast<AT*>(a.out)[(static_cast<int64_t>(t) * a.Hq + head) * a.h + i] = from_f32<AT>(num / den);
}

// The merge and the split in one launch (bf16 outputs; one block per token, four consecutive elements of the token's
// [Hq][h] row per thread): a token of a split request has its chunks merged exactly as attn_merge_kernel does, any
// other token's output is read back; then the row maximum, the token's scale, and the two e4m3 parts.
__global__ void attn_merge_split_kernel(AttnArgs a) {
  __shared__ float red[32];
  StampScope scope(LaunchStamp{a.stamp_merge.begin, a.stamp_merge.end});
  pdl_enter();
  const int t = blockIdx.x, e0 = threadIdx.x * 4, head = e0 / a.h, i = e0 % a.h;
  const int row_len = a.Hq * a.h;
  __nv_bfloat16* orow = static_cast<__nv_bfloat16*>(a.out) + static_cast<int64_t>(t) * row_len;
  const int n = a.part_acc ? a.req_chunks[a.tok_req[t]] : 1;
  float y[4];
  if (n <= 1) {
    const uint2 v = *reinterpret_cast<const uint2*>(orow + e0);
    y[0] = __uint_as_float(v.x << 16); y[1] = __uint_as_float(v.x & 0xffff0000u);
    y[2] = __uint_as_float(v.y << 16); y[3] = __uint_as_float(v.y & 0xffff0000u);
  } else {
    const int64_t first = static_cast<int64_t>(a.tok_part[t]);
    float M = -INFINITY;
    for (int c = 0; c < n; ++c) M = fmaxf(M, a.part_ml[((first + c) * a.Hq + head) * 2]);
    float num[4] = {0.f, 0.f, 0.f, 0.f}, den = 0.f;
    for (int c = 0; c < n; ++c) {
      const int64_t prow = (first + c) * a.Hq + head;
      const float mc = a.part_ml[prow * 2];
      if (mc == -INFINITY) continue;  // this chunk held no visible key
      const float w = exp2f(mc - M);
      den = fmaf(w, a.part_ml[prow * 2 + 1], den);
      const float4 acc = *reinterpret_cast<const float4*>(a.part_acc + prow * a.h + i);
      num[0] = fmaf(w, acc.x, num[0]); num[1] = fmaf(w, acc.y, num[1]);
      num[2] = fmaf(w, acc.z, num[2]); num[3] = fmaf(w, acc.w, num[3]);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const __nv_bfloat16 r = __float2bfloat16_rn(num[j] / den);
      orow[e0 + j] = r;
      y[j] = __bfloat162float(r);
    }
  }
  float amax = fmaxf(fmaxf(fabsf(y[0]), fabsf(y[1])), fmaxf(fabsf(y[2]), fabsf(y[3])));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = 0.f;
  for (int w = 0; w < (blockDim.x + 31) / 32; ++w) amax = fmaxf(amax, red[w]);
  const float s8 = token_scale_e4m3(amax);
  const float inv = 1.f / s8;
  if (threadIdx.x == 0) a.out8_scale[t] = s8;
  uint32_t h0, l0, h1, l1;
  split_pair_e4m3(y[0] * inv, y[1] * inv, h0, l0);
  split_pair_e4m3(y[2] * inv, y[3] * inv, h1, l1);
  *reinterpret_cast<uint32_t*>(a.out8 + static_cast<int64_t>(t) * row_len + e0) = h0 | (h1 << 16);
  *reinterpret_cast<uint32_t*>(a.out8 + static_cast<int64_t>(a.out8_lo_row0 + t) * row_len + e0) = l0 | (l1 << 16);
}

template <typename KT, typename AT>
int launch_typed(const AttnArgs& a, cudaStream_t s) {
  if (a.h == 64)
    SLED_LAUNCH_PDL((attn_simt_kernel<KT, AT, 64>), dim3(a.n_items), dim3(256), 0, s, a);
  else if (a.h == 128)
    SLED_LAUNCH_PDL((attn_simt_kernel<KT, AT, 128>), dim3(a.n_items), dim3(256), 0, s, a);
  else if (a.h == 32)
    SLED_LAUNCH_PDL((attn_simt_kernel<KT, AT, 32>), dim3(a.n_items), dim3(256), 0, s, a);
  else
    return -1;
  return 1;
}

}  // namespace

int launch_attention(const AttnArgs& a, cudaStream_t s, bool* split_done) {
  if (split_done) *split_done = false;
  if (a.n_items <= 0 || a.T <= 0) return 0;
  int n = -1;
  if (a.use_tc && a.kvdtype == BF16 && a.adtype == BF16 && a.map_k && a.page_size == 16 && a.h == 128)
    n = launch_attention_tc(a, s);    // tcgen05 kernel
  else if (a.kvdtype == BF16 && a.adtype == BF16 && a.map_k && a.page_size == 16 && (a.h == 64 || a.h == 128))
    n = launch_attention_mma(a, s);   // warp-level tensor-core kernel
  else if (a.kvdtype == BF16 && a.adtype == BF16) n = launch_typed<__nv_bfloat16, __nv_bfloat16>(a, s);
  else if (a.kvdtype == F32 && a.adtype == F32) n = launch_typed<float, float>(a, s);
  else if (a.kvdtype == BF16 && a.adtype == F32) n = launch_typed<__nv_bfloat16, float>(a, s);
  if (n < 0) return n;
  const int row_len = a.Hq * a.h;
  if (a.out8 && a.out8_scale && a.adtype == BF16 && a.h % 4 == 0 && row_len / 4 <= 1024 && (row_len / 4) % 32 == 0) {
    SLED_LAUNCH_PDL(attn_merge_split_kernel, dim3(a.T), dim3(row_len / 4), 0, s, a);
    if (split_done) *split_done = true;
    return n + 1;
  }
  if (a.part_acc) {  // some request was split
    dim3 grid(a.T, a.Hq);
    if (a.adtype == BF16) SLED_LAUNCH_PDL(attn_merge_kernel<__nv_bfloat16>, grid, dim3(a.h), 0, s, a);
    else SLED_LAUNCH_PDL(attn_merge_kernel<float>, grid, dim3(a.h), 0, s, a);
    ++n;
  }
  return n;
}

}  // namespace sled
