// Shared device helpers of the verification library (storage types, reductions).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace sled {

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// sum over the block; every thread gets the result.  scratch: >= 32 floats of shared memory.
__device__ __forceinline__ float block_sum(float v, float* scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  float t = lane < nw ? scratch[lane] : 0.f;
  return warp_sum(t);
}

// Programmatic dependent launch.  Every kernel of a verification step is launched so that it may
// begin while its predecessor in the stream drains; it lets its own successor do the same at once
// and must call pdl_wait() before it touches anything an earlier kernel wrote (and before it exits,
// so that "this grid is complete" always implies "everything before it is complete").
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_enter() {
  pdl_launch_dependents();
  pdl_wait();
}

// Optional device-side timestamps of a launch (benchmark mode): when the first block began and when the last one
// ended, in nanoseconds of the GPU's global timer.  Unlike events between kernels they leave the overlap of
// neighbouring launches (programmatic dependent launch) as it is.  `begin` starts at ~0, `end` at 0; a null
// pointer switches the stamps off.
struct LaunchStamp {
  unsigned long long* begin;
  unsigned long long* end;
};
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void stamp_begin(const LaunchStamp& s) {
  if (s.begin && threadIdx.x == 0 && threadIdx.y == 0) atomicMin(s.begin, global_ns());
}
__device__ __forceinline__ void stamp_end(const LaunchStamp& s) {
  if (s.end && threadIdx.x == 0 && threadIdx.y == 0) atomicMax(s.end, global_ns());
}
// stamps the end when the scope is left, whichever return is taken
struct StampScope {
  LaunchStamp s;
  __device__ __forceinline__ explicit StampScope(const LaunchStamp& st) : s(st) { stamp_begin(s); }
  __device__ __forceinline__ ~StampScope() { stamp_end(s); }
};

}  // namespace sled

// Launch with the programmatic-serialization attribute (host side).  `kern` must be a concrete
// __global__ function (template arguments spelled out).
#define SLED_LAUNCH_PDL(kern, grid_, block_, smem_, stream_, ...)                                  \
  do {                                                                                         \
    cudaLaunchConfig_t cfg__{};                                                                \
    cfg__.gridDim = (grid_);                                                                    \
    cfg__.blockDim = (block_);                                                                  \
    cfg__.dynamicSmemBytes = (smem_);                                                           \
    cfg__.stream = (stream_);                                                                   \
    cudaLaunchAttribute attr__[1];                                                             \
    attr__[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                         \
    attr__[0].val.programmaticStreamSerializationAllowed = 1;                                  \
    cfg__.attrs = attr__;                                                                      \
    cfg__.numAttrs = 1;                                                                        \
    cudaLaunchKernelEx(&cfg__, kern, __VA_ARGS__);                                             \
  } while (0)
