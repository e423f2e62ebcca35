// Tensor-core linear layer for bf16 weights: out[s][t][n] = sum over K-slice s of A[t][k] * W[n][k].
// tcgen05.mma with the weight rows on the M side (128 per tile) and the step's tokens on the N
// side, operands brought to shared memory by TMA, fp32 accumulators in tensor memory.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace sled {

struct TcWeight {       // [N][K] bf16, row-major, device memory
  CUtensorMap map;      // box 64 (k) x 128 (rows), 128-byte swizzle
  int N = 0, K = 0;
  bool ready = false;
};

struct TcActivation {   // [rows][K] bf16, row-major, device memory; rows is a multiple of 256
  CUtensorMap map[3];   // boxes of 64 (k) x {64, 128, 256} rows
  int rows = 0, K = 0;
};

// 2D bf16 tensor map over a row-major [rows][cols] array: boxes of 64 columns x box_rows rows, 128-byte swizzle
int tma_map_bf16_rows(CUtensorMap* map, const void* dev_ptr, long long rows, int cols, int box_rows);
int tc_weight_init(TcWeight* w, const void* dev_ptr, int N, int K);
void tc_weight_free(TcWeight* w);
int tc_activation_init(TcActivation* a, const void* dev_ptr, int rows, int K);
// number of K slices the launch below will use for this shape (each slice leaves one partial sum)
int tc_gemm_split(int T, int N, int K, int n_sm);
// returns kernels launched (1) or a negative value; `error` is a device word set if a bounded wait ran out
int tc_gemm_launch(const TcActivation& a, const TcWeight& w, int T, int n_split, float* out, int64_t split_stride,
                   int32_t* error, int n_sm, cudaStream_t s);

}  // namespace sled
