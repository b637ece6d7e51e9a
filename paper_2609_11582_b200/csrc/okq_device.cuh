// Warp-level building blocks shared by the quantise and decode kernels.
#pragma once
#include "okq_layout.cuh"

namespace okq {

// ||x||_2 of the 128-vector spread 4 channels per lane; adjacent-pair summation tree.
__device__ __forceinline__ float warp_norm(float4 x) {
  float s = __fadd_rn(__fadd_rn(__fmul_rn(x.x, x.x), __fmul_rn(x.y, x.y)),
                      __fadd_rn(__fmul_rn(x.z, x.z), __fmul_rn(x.w, x.w)));
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) s = __fadd_rn(s, __shfl_xor_sync(0xffffffffu, s, d));
  float n = __fsqrt_rn(s);
  return n > 65504.0f ? 65504.0f : n;
}

__device__ __forceinline__ float4 load_row4(const __half* row, int lane) {
  uint2 raw = *reinterpret_cast<const uint2*>(row + 4 * lane);
  __half2 lo = *reinterpret_cast<__half2*>(&raw.x), hi = *reinterpret_cast<__half2*>(&raw.y);
  float2 a = __half22float2(lo), b = __half22float2(hi);
  return make_float4(a.x, a.y, b.x, b.y);
}

// Unnormalised Sylvester FWHT of a 128-vector held 4 consecutive channels per lane.
__device__ __forceinline__ float4 warp_fwht(float4 y, int lane) {
  float a0 = __fadd_rn(y.x, y.y), a1 = __fsub_rn(y.x, y.y), a2 = __fadd_rn(y.z, y.w), a3 = __fsub_rn(y.z, y.w);
  float v[4] = {__fadd_rn(a0, a2), __fadd_rn(a1, a3), __fsub_rn(a0, a2), __fsub_rn(a1, a3)};
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    bool upper = (lane & d) != 0;
#pragma unroll
    for (int k = 0; k < 4; k++) {
      float p = __shfl_xor_sync(0xffffffffu, v[k], d);
      v[k] = upper ? __fsub_rn(p, v[k]) : __fadd_rn(v[k], p);
    }
  }
  return make_float4(v[0], v[1], v[2], v[3]);
}

}  // namespace okq
