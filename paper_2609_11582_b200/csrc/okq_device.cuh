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

// ---- MXFP4 metadata: E2M1 elements {0, .5, 1, 1.5, 2, 3, 4, 6} (sign in bit 3) times 2^k

// smallest k in [-23, 12] with 6 * 2^k >= amax  (6 * 2^k = 0.75 * 2^(k+3))
__device__ __forceinline__ int mx_scale_exp(float amax) {
  int k = -23;
  if (amax > 0.0f) {
    int e;
    const float f = frexpf(amax, &e);
    k = f <= 0.75f ? e - 3 : e - 2;
  }
  return max(-23, min(12, k));
}

__device__ __forceinline__ float mx_grid(int idx) {
  return idx < 4 ? 0.5f * (float)idx : (idx == 4 ? 2.0f : (idx == 5 ? 3.0f : (idx == 6 ? 4.0f : 6.0f)));
}

// nibble of x on the grid * 2^k, rounded down (up = false) or up (up = true); |x| <= 6 * 2^k
__device__ __forceinline__ unsigned mx_encode(float x, int k, bool up) {
  const float q = ldexpf(x, -k);   // exact
  const float a = fabsf(q);
  // magnitude index: largest grid value <= a, or smallest grid value >= a
  const int lo = (a >= 0.5f) + (a >= 1.0f) + (a >= 1.5f) + (a >= 2.0f) + (a >= 3.0f) + (a >= 4.0f) + (a >= 6.0f);
  const int hi = min(7, (a > 0.0f) + (a > 0.5f) + (a > 1.0f) + (a > 1.5f) + (a > 2.0f) + (a > 3.0f) + (a > 4.0f));
  const bool neg = q < 0.0f;
  const int idx = (up != neg) ? hi : lo;   // rounding up a negative number shrinks its magnitude
  return idx == 0 ? 0u : ((neg ? 8u : 0u) | (unsigned)idx);
}

__device__ __forceinline__ float mx_decode(unsigned nib, int k) {
  const float g = mx_grid((int)(nib & 7u));
  return ldexpf((nib & 8u) ? -g : g, k);
}


// Four E2M1 nibbles (low nibble first) -> two fp16 pairs of the unscaled grid values.  The byte LUT
// holds the high bytes of fp16 {0, .5, 1, 1.5, 2, 3, 4, 6}; their low bytes are zero.
__device__ __forceinline__ void e2m1x4_to_half2(uint32_t x, uint32_t& h01, uint32_t& h23) {
  const uint32_t hb = __byte_perm(0x3E3C3800u, 0x46444240u, x & 0x7777u);
  const uint32_t sg = x & 0x8888u;
  h01 = __byte_perm(hb, 0u, 0x1404u) | ((sg << 12) & 0x8000u) | ((sg << 24) & 0x80000000u);
  h23 = __byte_perm(hb, 0u, 0x3424u) | ((sg << 4) & 0x8000u) | ((sg << 16) & 0x80000000u);
}

// fp16 pair (2^k, 2^k) for k in [-24, 15]
__device__ __forceinline__ uint32_t pow2_half2(int k) {
  const uint32_t h = k >= -14 ? (uint32_t)(k + 15) << 10 : 1u << (k + 24);
  return h | (h << 16);
}

// Decoded (m * 4^j, s) of record positions 4*lane .. 4*lane+3 from the 136 MXFP4 metadata bytes
// (global or shared, 2-byte aligned): four fp16 each, exact; m with the position scale of the fp16 layout.
__device__ __forceinline__ void mx_decode_lane(const unsigned char* meta, int lane, uint2& m4, uint2& s4) {
  const uint32_t xm = *reinterpret_cast<const unsigned short*>(meta + 2 * lane);
  const uint32_t xs = *reinterpret_cast<const unsigned short*>(meta + 64 + 2 * lane);
  const int blk = (lane >> 1) & 3;   // positions 8j .. 8j+7 (mod 32) belong to channel block j
  const uint32_t pm = pow2_half2((int)meta[128 + blk] - 127), ps = pow2_half2((int)meta[132 + blk] - 127);
  uint32_t a, b;
  e2m1x4_to_half2(xm, a, b);
  __half2 r0 = __hmul2(*reinterpret_cast<__half2*>(&a), *reinterpret_cast<const __half2*>(&pm));
  __half2 r1 = __hmul2(*reinterpret_cast<__half2*>(&b), *reinterpret_cast<const __half2*>(&pm));
  // the staged m plane carries the position scale 4^j: positions 4*lane + {0,1} have j = 2*(lane & 1), the
  // other two j + 1 (a second exact multiply: 2^k * 4^j alone may leave the fp16 range)
  const uint32_t q0 = pow2_half2(4 * (lane & 1)), q1 = pow2_half2(4 * (lane & 1) + 2);
  r0 = __hmul2(r0, *reinterpret_cast<const __half2*>(&q0));
  r1 = __hmul2(r1, *reinterpret_cast<const __half2*>(&q1));
  m4 = make_uint2(*reinterpret_cast<uint32_t*>(&r0), *reinterpret_cast<uint32_t*>(&r1));
  e2m1x4_to_half2(xs, a, b);
  r0 = __hmul2(*reinterpret_cast<__half2*>(&a), *reinterpret_cast<const __half2*>(&ps));
  r1 = __hmul2(*reinterpret_cast<__half2*>(&b), *reinterpret_cast<const __half2*>(&ps));
  s4 = make_uint2(*reinterpret_cast<uint32_t*>(&r0), *reinterpret_cast<uint32_t*>(&r1));
}

}  // namespace okq
