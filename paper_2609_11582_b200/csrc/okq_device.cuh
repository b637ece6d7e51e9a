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

// ---- MXFP4 metadata: E2M1 elements {0, .5, 1, 1.5, 2, 3, 4, 6} (sign in bit 3) times 2^k, converted as in
// the OCP microscaling format

// block exponent floor(log2 amax) - 2, clamped to [-23, 12] (-23 for an all-zero block)
__device__ __forceinline__ int mx_scale_exp(float amax) {
  int k = -23;
  if (amax > 0.0f) {
    int e;
    (void)frexpf(amax, &e);   // amax = f * 2^e, f in [0.5, 1)
    k = e - 3;
  }
  return max(-23, min(12, k));
}

__device__ __forceinline__ float mx_grid(int idx) {
  return idx < 4 ? 0.5f * (float)idx : (idx == 4 ? 2.0f : (idx == 5 ? 3.0f : (idx == 6 ? 4.0f : 6.0f)));
}

// nibble of x on the grid * 2^k: nearest grid value, ties to the even mantissa bit (0, 1, 2, 4), magnitudes
// beyond 6 * 2^k saturate.  The decision points are the midpoints of neighbouring grid values; a tie goes up
// exactly when the upper neighbour has the even mantissa bit.
__device__ __forceinline__ unsigned mx_encode(float x, int k) {
  const float q = ldexpf(x, -k);   // exact
  const float a = fabsf(q);
  const int idx = (a > 0.25f) + (a >= 0.75f) + (a > 1.25f) + (a >= 1.75f) + (a > 2.5f) + (a >= 3.5f) + (a > 5.0f);
  return idx == 0 ? 0u : ((q < 0.0f ? 8u : 0u) | (unsigned)idx);
}

__device__ __forceinline__ float mx_decode(unsigned nib, int k) {
  const float g = mx_grid((int)(nib & 7u));
  return ldexpf((nib & 8u) ? -g : g, k);
}


// E2M1 decode by byte permute: a nibble's low three bits select the high byte of the fp16 value
// {0, .5, 1, 1.5, 2, 3, 4, 6} * 4^j (low byte zero; 4^j adds 2 j to the exponent, i.e. 8 j to the high byte
// of the non-zero entries).
__device__ __forceinline__ uint32_t e2m1_lut_lo(int j) { return 0x3E3C3800u + 0x08080800u * (uint32_t)j; }
__device__ __forceinline__ uint32_t e2m1_lut_hi(int j) { return 0x46444240u + 0x08080808u * (uint32_t)j; }

// fp16 pair (2^k, 2^k) from the stored exponent byte k + 127 (k in [-24, 15]): the byte is the exponent
// field of the fp32 number 2^k
__device__ __forceinline__ __half2 pow2_half2(uint32_t byte) {
  const float f = __uint_as_float(byte << 23);
  return __floats2half2_rn(f, f);
}

// Decoded (m * 4^j, s) of record positions 4*lane .. 4*lane+3 from the 136 MXFP4 metadata bytes
// (global or shared, 2-byte aligned): four fp16 each, exact.  m carries the position scale of the fp16
// layout's m plane: positions 4*lane + {0, 1} have j = 2*(lane & 1), the other two j + 1 (folded into the
// lookup: grid * 4^j <= 384, and the product with 2^k, |m| * 4^j <= 64, is an fp16 number).
__device__ __forceinline__ void mx_decode_lane(const unsigned char* meta, int lane, uint2& m4, uint2& s4) {
  const uint32_t xm = *reinterpret_cast<const unsigned short*>(meta + 2 * lane);
  const uint32_t xs = *reinterpret_cast<const unsigned short*>(meta + 64 + 2 * lane);
  const int blk = (lane >> 1) & 3;   // positions 8j .. 8j+7 (mod 32) belong to channel block j
  const __half2 pm = pow2_half2(meta[128 + blk]), ps = pow2_half2(meta[132 + blk]);
  const int j0 = 2 * (lane & 1);
  // magnitudes: bytes 0, 1 of the first lookup (scale 4^j0), bytes 2, 3 of the second (4^(j0+1))
  const uint32_t im = xm & 0x7777u;
  const uint32_t ma = __byte_perm(e2m1_lut_lo(j0), e2m1_lut_hi(j0), im);
  const uint32_t mb = __byte_perm(e2m1_lut_lo(j0 + 1), e2m1_lut_hi(j0 + 1), im);
  // signs: nibble bit 3 of values 0 / 1 -> bits 15 / 31, of values 2 / 3 likewise (the products spread the
  // four sign bits; stray carries stay below the masked bits)
  const uint32_t sg = xm & 0x8888u;
  uint32_t h01 = __byte_perm(ma, 0u, 0x1404u) | ((sg * 0x01001000u) & 0x80008000u);
  uint32_t h23 = __byte_perm(mb, 0u, 0x3424u) | ((sg * 0x00010010u) & 0x80008000u);
  __half2 r0 = __hmul2(*reinterpret_cast<__half2*>(&h01), pm);
  __half2 r1 = __hmul2(*reinterpret_cast<__half2*>(&h23), pm);
  m4 = make_uint2(*reinterpret_cast<uint32_t*>(&r0), *reinterpret_cast<uint32_t*>(&r1));
  // s is never negative
  const uint32_t sa = __byte_perm(e2m1_lut_lo(0), e2m1_lut_hi(0), xs & 0x7777u);
  h01 = __byte_perm(sa, 0u, 0x1404u);
  h23 = __byte_perm(sa, 0u, 0x3424u);
  r0 = __hmul2(*reinterpret_cast<__half2*>(&h01), ps);
  r1 = __hmul2(*reinterpret_cast<__half2*>(&h23), ps);
  s4 = make_uint2(*reinterpret_cast<uint32_t*>(&r0), *reinterpret_cast<uint32_t*>(&r1));
}

}  // namespace okq
