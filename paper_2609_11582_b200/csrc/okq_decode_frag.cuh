// Device helpers shared by the tensor-core decode kernels (split-K kernels and the combine kernel): mma.sync and
// cp.async wrappers, the fp16 hi/lo product split, and the rotated query fragments.
#pragma once
#include "okq_common.cuh"
#include "okq_device.cuh"
#include "okq_decode_shared.cuh"

namespace okq {

__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem));
}
__device__ __forceinline__ void cp_async8(void* smem, const void* gmem) {
  uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(s), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

// hardware barrier shared by the two warps of a pair (ids 1..8; id 0 is __syncthreads)
__device__ __forceinline__ void pair_barrier(int pair) {
  asm volatile("bar.sync %0, 64;\n" ::"r"(pair + 1) : "memory");
}

__device__ __forceinline__ uint32_t h2u(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ __half2 u2h(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

// fp16 pair (lo half = a, hi half = b), saturating instead of overflowing to infinity
__device__ __forceinline__ uint32_t pack_sat(float a, float b) {
  uint32_t r;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;\n" : "=r"(r) : "f"(b), "f"(a));
  return r;
}

// hi/lo split of the product q * x (q = qh + ql, x an exact fp16 pair): hi = rn(qh*x),
// lo = rn(ql*x + (qh*x - hi)); the inner fma recovers the rounding error of hi exactly.
__device__ __forceinline__ void split_product(__half2 qh, __half2 ql, __half2 x, uint32_t& hi, uint32_t& lo) {
  __half2 h = __hmul2(qh, x);
  __half2 e = __hfma2(qh, x, __hneg2(h));
  hi = h2u(h);
  lo = h2u(__hfma2(ql, x, e));
}

// The group's rotated queries q' = H D q / sqrt(128) as mma A-fragment registers, computed by one warp in
// registers (q: the group's query rows [group][128], signs: the layer's Hadamard signs): lane (g, t) holds head
// g, channels 8 r + 2 t + {0, 1} for r = 0..15, so the transform's
// butterflies over channel bits 0 and 3..6 stay inside the lane and those over bits 1..2 are two shuffles.
// Each pair is scaled into the fp16 range (2^kh, per head), pre-divided by 4^(r&3) (the position scale of
// the matching code field) and split into an fp16 high and low part.  fsc = 2^(24-kh) * sm_scale * log2(e).
__device__ __forceinline__ void query_fragments(const __half* q, const float* signs, int G, float sm_scale, int lane,
                                                uint2 (&qreg)[16], float& fsc) {
  const int g = lane >> 2, t = lane & 3;
  float x[16][2];
  if (g < G) {
    const __half* qrow = q + (size_t)g * D + 2 * t;
    const float* srow = signs + 2 * t;
#pragma unroll
    for (int r = 0; r < 16; r++) {
      const float2 qv = __half22float2(*reinterpret_cast<const __half2*>(qrow + 8 * r));
      const float2 sv = *reinterpret_cast<const float2*>(srow + 8 * r);
      x[r][0] = qv.x * sv.x; x[r][1] = qv.y * sv.y;
    }
  } else {
#pragma unroll
    for (int r = 0; r < 16; r++) x[r][0] = x[r][1] = 0.f;
  }
#pragma unroll
  for (int r = 0; r < 16; r++) {   // channel bit 0
    const float a = x[r][0], b = x[r][1];
    x[r][0] = a + b; x[r][1] = a - b;
  }
#pragma unroll
  for (int d = 1; d < 4; d <<= 1) {   // channel bits 1, 2: lanes t ^ d
    const bool upper = (lane & d) != 0;
#pragma unroll
    for (int r = 0; r < 16; r++)
#pragma unroll
      for (int e = 0; e < 2; e++) {
        const float p = __shfl_xor_sync(0xffffffffu, x[r][e], d);
        x[r][e] = upper ? p - x[r][e] : x[r][e] + p;
      }
  }
#pragma unroll
  for (int s = 1; s < 16; s <<= 1)   // channel bits 3..6
#pragma unroll
    for (int r = 0; r < 16; r++)
      if (!(r & s)) {
#pragma unroll
        for (int e = 0; e < 2; e++) {
          const float a = x[r][e], b = x[r + s][e];
          x[r][e] = a + b; x[r + s][e] = a - b;
        }
      }
  float mx = 0.f;
#pragma unroll
  for (int r = 0; r < 16; r++) {
    x[r][0] *= RSQRT_D; x[r][1] *= RSQRT_D;
    mx = fmaxf(mx, fmaxf(fabsf(x[r][0]), fabsf(x[r][1])));
  }
  mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
  mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
  int ex = 0;
  if (mx > 0.f) frexpf(mx, &ex);           // mx < 2^ex
  const int kh = 14 - ex;                  // |q'| * 2^kh < 2^14
  const float up = exp2f((float)kh);
  fsc = exp2f((float)(24 - kh)) * sm_scale * 1.4426950408889634f;
#pragma unroll
  for (int r = 0; r < 16; r++) {
    const float sc = up / (float)(1 << (2 * (r & 3)));
    const float x0 = x[r][0] * sc, x1 = x[r][1] * sc;
    const __half2 hi2 = __floats2half2_rn(x0, x1);
    const float2 hf = __half22float2(hi2);
    qreg[r] = make_uint2(h2u(hi2), h2u(__floats2half2_rn(x0 - hf.x, x1 - hf.y)));
  }
}

}  // namespace okq
