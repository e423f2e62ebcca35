// Host-callable launchers of the device kernels.  Every launcher only enqueues work on
// the given stream and returns the number of kernels it launched (negative: bad argument).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace sled {

enum DType { F32 = 0, BF16 = 1 };

// Device addresses that receive a launch's begin / end time (see common.cuh); null members: no stamps.
struct Stamp {
  unsigned long long* begin = nullptr;
  unsigned long long* end = nullptr;
};

// ---- elementwise / small kernels (kernels_small.cu)
int launch_embed(const void* table, int wdtype, const int32_t* ids, int T, int d, float* x, cudaStream_t s,
                 Stamp st = Stamp());
// x += sum_s partial[s] (if partial), then out = RMSNorm(x) * gain in the activation type
// out8 / lo_row0 / scale8 (optional, bf16 only): the outputs once more as two e4m3 parts per element and a scale per
// token, where the kernel can do it (*split_done tells)
int launch_add_rmsnorm(float* x, const float* partial, int n_split, int64_t split_stride, const void* gain, int wdtype,
                       float eps, int T, int d, void* out, int adtype, cudaStream_t s, Stamp st = Stamp(),
                       uint8_t* out8 = nullptr, int lo_row0 = 0, float* scale8 = nullptr, bool* split_done = nullptr);
int launch_rope_table(const int32_t* tok_pos, int T, int h, float theta, float2* cs, cudaStream_t s, Stamp st = Stamp());
// sums the QKV partials, rotates Q and K, writes Q to q_out and K, V into their cache slots
int launch_rope_kv(const float* partial, int n_split, int64_t split_stride, const float2* cs, const int32_t* tok_slot,
                   int T, int Hq, int Hkv, int h, int page_size, void* q_out, int adtype, void* kpool, void* vpool,
                   int kvdtype, cudaStream_t s, Stamp st = Stamp());
int launch_swiglu(const float* partial, int n_split, int64_t split_stride, int T, int F, void* out, int adtype,
                  cudaStream_t s, Stamp st = Stamp());
// contiguous [n][Hkv][h] <-> paged cache of one layer
int launch_kv_scatter(const void* src, const int32_t* slots, int n, int Hkv, int h, int page_size, void* pool,
                      int kvdtype, cudaStream_t s);
int launch_kv_gather(const void* pool, const int32_t* slots, int n, int Hkv, int h, int page_size, void* dst,
                     int kvdtype, cudaStream_t s);

// ---- fp32 / generic CUDA-core GEMM (kernels_small.cu): out[s][T][N] = A[T][Kslice_s] . W[N][Kslice_s]^T
int launch_gemm_simt(const void* A, int adtype, const void* W, int wdtype, int T, int N, int K, int n_split,
                     float* out, int64_t split_stride, cudaStream_t s, Stamp st = Stamp());

// ---- ragged verification attention over the paged cache (attention.cu)
struct AttnArgs {
  const int4* items;  // {request, kv head, first key, key count}
  int n_items;
  const void* q;      // [T][Hq][h] activation type
  void* out;          // [T][Hq][h] activation type
  const void* kpool;  // one layer: [page][Hkv][page_size][h]
  const void* vpool;
  const int32_t* cu_q;       // [B+1]
  const int32_t* kv_base;    // [B] cached tokens before the step: query j sees keys 0 .. kv_base + j
  const int32_t* page_table; // flat
  const int32_t* pt_off;     // [B+1]
  const int32_t* tok_req;    // [T]
  const int32_t* tok_part;   // [T] first partial-result row of a token (tokens of split requests only)
  const int32_t* req_chunks; // [B] number of key chunks of a request
  const int32_t* req_chunk_keys; // [B] keys per chunk of a request (a multiple of 64)
  float* part_acc;           // [rows][Hq][h]
  float* part_ml;            // [rows][Hq][2]
  int T, Hq, Hkv, h, page_size;
  int adtype, kvdtype;
  // tensor-core path (bf16 cache, 16-token pages): tensor maps over this layer's K and V pool
  // viewed as [page*Hkv*16 + slot][h], and a device word that records a bounded wait running out
  const CUtensorMap* map_k = nullptr;
  const CUtensorMap* map_v = nullptr;
  int32_t* error = nullptr;
  Stamp stamp, stamp_merge;   // of the attention kernel and of the merge kernel that may follow it
  int use_tc = 0;             // 1: every item has at most 48 query rows and head_dim is 128: the tcgen05 kernel runs
  // optional (bf16 activations): the output once more as two e4m3 parts per element and a scale per token, the
  // operand format of the fp8 linear layers - hi rows at out8[t], lo rows at out8[out8_lo_row0 + t]
  uint8_t* out8 = nullptr;
  int out8_lo_row0 = 0;
  float* out8_scale = nullptr;
};
// *split_done (optional) tells whether out8 / out8_scale were written
int launch_attention(const AttnArgs& a, cudaStream_t s, bool* split_done = nullptr);
// warp-level tensor-core kernel alone (attention_mma.cu); returns 1 or a negative value
int launch_attention_mma(const AttnArgs& a, cudaStream_t s);
// tcgen05 kernel alone (attention_tc.cu): head_dim 128, at most 48 query rows per item; returns 1 or a negative value
int launch_attention_tc(const AttnArgs& a, cudaStream_t s);

// ---- fused vocabulary softmax + acceptance + corrective / bonus draw (accept.cu)
struct AcceptArgs {
  const float* logits;        // [rows][V]
  const int32_t* cu_q;        // [B+1] first row of each request
  const int32_t* ids;         // [rows] fed tokens: drafts of request i are ids[cu_q[i]+1 ..]
  const void* const* q_rows;  // [B] device pointer to the request's [k][V] draft distributions (may hold null)
  int q_bf16;                 // 1: the rows are bf16, 0: fp32
  const uint32_t* ctx_lo;     // [B]
  const uint32_t* ctx_hi;     // [B]
  const int32_t* pos0;        // [B] absolute index of the pending token
  int32_t* results;           // [B][3] n_accepted, next_token, status
  int B, V;
  float inv_tau;
  int greedy;
  uint64_t seed;
  Stamp stamp;
};
int launch_accept(const AcceptArgs& a, cudaStream_t s);

}  // namespace sled
