// Tensor-core linear layer for bf16 weights: out[s][t][n] = sum over K-slice s of A[t][k] * W[n][k].
// tcgen05.mma with the weight rows on the M side (128 per tile) and the step's tokens on the N
// side, operands brought to shared memory by TMA, fp32 accumulators in tensor memory.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace sled {

struct TcWeight {       // [N][K] bf16 weights, stored as 128 x 64 tiles of 16 KB (see tc_weight_init)
  CUtensorMap map;      // over the tiled array seen as rows of 128 bytes; box = one tile, 128-byte swizzle
  int N = 0, K = 0;
  bool ready = false;
  // 8-bit weights instead (tc_weight_init_f8): e4m3 bytes as 128 x 128 tiles of 16 KB behind map8 and one fp32 scale
  // per output row
  CUtensorMap map8;
  const float* scale = nullptr;
  bool f8 = false;
  // 4-bit weights (tc_weight_init_f4): e2m1 nibbles, two per byte, as 128 x 128 tiles of 8 KB behind map8 (whose
  // element type makes the copy spread every 8 bytes of nibbles over 16 bytes of shared memory, the form the fp8
  // kind of MMA reads 4-bit operands in); f8 is set as well: everything but the weight operand is the 8-bit path
  bool f4 = false;
};

struct TcActivation8 {  // an activation tensor as two e4m3 parts per element and one fp32 scale per token (see
                        // tc_split_rows_launch): [2 * rows][K] bytes - hi rows first, lo rows from row `rows` on
  CUtensorMap map[4];   // boxes of 128 (k) x {32, 64, 96, 128} rows
  uint8_t* data = nullptr;
  float* scale = nullptr;   // [rows]
  int rows = 0, K = 0;
};

constexpr int kTokenTiles = 6;
struct TcActivation {   // [rows][K] bf16, row-major, device memory; rows is a multiple of 256
  CUtensorMap map[kTokenTiles];   // boxes of 64 (k) x {32, 64, 96, 128, 160, 256} rows
  int rows = 0, K = 0;
};

enum { kEpiStore = 0, kEpiSwiglu = 1 };
struct TcEpilogue {       // what happens to the finished sums (see emit16 in gemm_tc.cu)
  int mode = kEpiStore;
  __nv_bfloat16* act_out = nullptr;   // kEpiSwiglu: [T][act_ld] activations for the down projection
  int act_ld = 0;
  // benchmark mode: device words that receive the time the launch's first block began / its last block ended
  unsigned long long* stamp_begin = nullptr;
  unsigned long long* stamp_end = nullptr;
};

// 2D bf16 tensor map over a row-major [rows][cols] array: boxes of 64 columns x box_rows rows, 128-byte swizzle
int tma_map_bf16_rows(CUtensorMap* map, const void* dev_ptr, long long rows, int cols, int box_rows);
// Bytes of the tiled copy of an [N][K] matrix, and its construction from the row-major matrix (both in
// device memory; `tiled` 16-byte aligned, tc_weight_tiled_bytes(N, K) long).  The row-major copy is not
// needed afterwards.  Synchronises the device.
size_t tc_weight_tiled_bytes(int N, int K);
int tc_weight_init(TcWeight* w, const void* rowmajor, void* tiled, int N, int K);
// The same for e4m3 bytes [N][K] (row-major, device; K a multiple of 16) with `scale` [N] fp32 (device; must stay
// valid): W[n][k] = scale[n] * e4m3(byte).  `tiled` holds tc_weight_f8_tiled_bytes(N, K) bytes.  The byte patterns
// 0x7f / 0xff (NaN in e4m3) must not occur.
size_t tc_weight_f8_tiled_bytes(int N, int K);
int tc_weight_init_f8(TcWeight* w, const void* rowmajor_bytes, void* tiled, const float* scale, int N, int K);
// The same for e2m1 nibbles [N][K / 2] bytes (row-major, device; element k of a row in byte k / 2, even k in the low
// half; K a multiple of 16): W[n][k] = scale[n] * e2m1(nibble).  `tiled` (32-byte aligned) holds
// tc_weight_f4_tiled_bytes(N, K) bytes.
size_t tc_weight_f4_tiled_bytes(int N, int K);
int tc_weight_init_f4(TcWeight* w, const void* rowmajor_nibbles, void* tiled, const float* scale, int N, int K);
// `data`: 2 * rows * K bytes, `scale`: rows floats (device, zero-initialised by the caller); rows a multiple of 128
int tc_activation8_init(TcActivation8* a, void* data, float* scale, int rows, int K);
// a[T][K] bf16 (device) -> the two e4m3 parts and the token scales of `dst`; returns kernels launched or < 0
int tc_split_rows_launch(const void* a_bf16, int T, const TcActivation8& dst, cudaStream_t s,
                         unsigned long long* stamp_begin, unsigned long long* stamp_end);
int tc_gemm_split_f8(int T, int N, int K, int n_sm);
// out[slice][T][N] = scale_t * scale_n * (hi + lo)[T][K slice] . W8[N][K slice]^T
int tc_gemm_f8_launch(const TcActivation8& a, const TcWeight& w, int T, int n_split, float* out, int64_t split_stride,
                      int32_t* error, const TcEpilogue& epi, cudaStream_t s);
void tc_weight_free(TcWeight* w);
int tc_activation_init(TcActivation* a, const void* dev_ptr, int rows, int K);
// number of partial-sum slices [slice][T][N] a launch leaves behind for this shape (bf16 weights; tc_gemm_split_f8:
// 8-bit weights)
int tc_gemm_split(int T, int N, int K, int n_sm);
// out[slice][T][N] = A[T][K slice] . W[N][K slice]^T; returns kernels launched (1) or a negative value;
// `error` is a device word set if a bounded wait ran out
int tc_gemm_launch(const TcActivation& a, const TcWeight& w, int T, int n_split, float* out, int64_t split_stride,
                   int32_t* error, const TcEpilogue& epi, cudaStream_t s);

// Self-test: launches a kernel whose bounded wait (limit in clock cycles, at most the kernels' own limit) runs out
// on a barrier nobody signals and records code 9 in *error.  Returns kernels launched (1) or a negative value.
int tc_wait_probe_launch(int32_t* error, long long limit_cycles, cudaStream_t s);

}  // namespace sled
