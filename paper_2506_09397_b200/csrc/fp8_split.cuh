// An activation as two e4m3 numbers: x = hi + lo with hi = e4m3(x) and lo = e4m3(x - hi), for |x| <= 448
// (x = a / s_t with the token's scale s_t = max|a| / 448).  The products of fp8 MMAs with hi and with lo are exact
// in fp32, so their sum carries eight significant bits of a - what a bf16 operand would.
#pragma once
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include <cstdint>

namespace sled {

// two values at once; the low byte of each result belongs to x0
__device__ __forceinline__ void split_pair_e4m3(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  const __nv_fp8x2_storage_t hq = __nv_cvt_float2_to_fp8x2(make_float2(x0, x1), __NV_SATFINITE, __NV_E4M3);
  const float2 hf = __half22float2(__half2(__nv_cvt_fp8x2_to_halfraw2(hq, __NV_E4M3)));
  const __nv_fp8x2_storage_t lq = __nv_cvt_float2_to_fp8x2(make_float2(x0 - hf.x, x1 - hf.y), __NV_SATFINITE, __NV_E4M3);
  hi = hq;
  lo = lq;
}

__device__ __forceinline__ float token_scale_e4m3(float amax) { return amax > 0.f ? amax / 448.f : 1.f; }

}  // namespace sled
