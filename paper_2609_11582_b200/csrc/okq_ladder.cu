// OmniKVQuant at 2, 3 and 4 bits per code over a canonical cache (the bit-width ladder: K2V2 / K3V3 / K4V4).
// Plain CUDA-core kernels that follow the 2-bit path's arithmetic with the number of levels changed:
//   k_ladder_keys    Eq. 2 + Eq. 4: one block per 32-token window of one (sequence, KV head)
//   k_ladder_values  Eq. 6 + Eq. 3: likewise, the rotation as one fused-multiply-add chain per coordinate
//   k_ladder_decode  Eq. 1 in the rotated space: one block per (sequence, KV head) walks the windows
// The value levels are the Lloyd-Max quantiser of N(0, 1/128) with 2^b levels (fixed point of: level = mean of its
// cell, threshold = mid-point of neighbouring levels), held as constants.
#include "../../include/okq_ladder.h"
#include "okq_common.cuh"
#include "okq_device.cuh"

namespace okq {

namespace {

constexpr int GP_L = OKQ_MAX_GROUP;   // padded GQA group

// ascending levels / thresholds for b = 2, 3, 4 (index b - 2); the middle threshold is 0 by symmetry
__constant__ float c_levels[3][16] = {
    {-0x1.116a30p-3f, -0x1.47d908p-5f, 0x1.47d908p-5f, 0x1.116a30p-3f},
    {-0x1.858b36p-3f, -0x1.e68c10p-4f, -0x1.11b402p-4f, -0x1.62ef2ep-6f, 0x1.62ef2ep-6f, 0x1.11b402p-4f, 0x1.e68c10p-4f,
     0x1.858b36p-3f},
    {-0x1.eea6ccp-3f, -0x1.76883ap-3f, -0x1.24e5cep-3f, -0x1.c6cde4p-4f, -0x1.5529e8p-4f, -0x1.db8b5ep-5f, -0x1.18fa1cp-5f,
     -0x1.73df2ap-7f, 0x1.73df2ap-7f, 0x1.18fa1cp-5f, 0x1.db8b5ep-5f, 0x1.5529e8p-4f, 0x1.c6cde4p-4f, 0x1.24e5cep-3f,
     0x1.76883ap-3f, 0x1.eea6ccp-3f}};
__constant__ float c_thresholds[3][16] = {
    {-0x1.636072p-4f, 0.0f, 0x1.636072p-4f},
    {-0x1.3c689ep-3f, -0x1.7c200ap-4f, -0x1.6a6fccp-5f, 0.0f, 0x1.6a6fccp-5f, 0x1.7c200ap-4f, 0x1.3c689ep-3f},
    {-0x1.b29782p-3f, -0x1.4db704p-3f, -0x1.042660p-3f, -0x1.8dfbe6p-4f, -0x1.2177ccp-4f, -0x1.7a42bcp-5f, -0x1.75f1e6p-6f, 0.0f,
     0x1.75f1e6p-6f, 0x1.7a42bcp-5f, 0x1.2177ccp-4f, 0x1.8dfbe6p-4f, 0x1.042660p-3f, 0x1.4db704p-3f, 0x1.b29782p-3f}};
const float h_levels[3][16] = {
    {-0x1.116a30p-3f, -0x1.47d908p-5f, 0x1.47d908p-5f, 0x1.116a30p-3f},
    {-0x1.858b36p-3f, -0x1.e68c10p-4f, -0x1.11b402p-4f, -0x1.62ef2ep-6f, 0x1.62ef2ep-6f, 0x1.11b402p-4f, 0x1.e68c10p-4f,
     0x1.858b36p-3f},
    {-0x1.eea6ccp-3f, -0x1.76883ap-3f, -0x1.24e5cep-3f, -0x1.c6cde4p-4f, -0x1.5529e8p-4f, -0x1.db8b5ep-5f, -0x1.18fa1cp-5f,
     -0x1.73df2ap-7f, 0x1.73df2ap-7f, 0x1.18fa1cp-5f, 0x1.db8b5ep-5f, 0x1.5529e8p-4f, 0x1.c6cde4p-4f, 0x1.24e5cep-3f,
     0x1.76883ap-3f, 0x1.eea6ccp-3f}};
const float h_thresholds[3][16] = {
    {-0x1.636072p-4f, 0.0f, 0x1.636072p-4f},
    {-0x1.3c689ep-3f, -0x1.7c200ap-4f, -0x1.6a6fccp-5f, 0.0f, 0x1.6a6fccp-5f, 0x1.7c200ap-4f, 0x1.3c689ep-3f},
    {-0x1.b29782p-3f, -0x1.4db704p-3f, -0x1.042660p-3f, -0x1.8dfbe6p-4f, -0x1.2177ccp-4f, -0x1.7a42bcp-5f, -0x1.75f1e6p-6f, 0.0f,
     0x1.75f1e6p-6f, 0x1.7a42bcp-5f, 0x1.2177ccp-4f, 0x1.8dfbe6p-4f, 0x1.042660p-3f, 0x1.4db704p-3f, 0x1.b29782p-3f}};

struct LadderView {
  int batch, n_kv_heads, n_q_heads, capacity, bits;
  unsigned char* k_codes;
  __half* k_norm;
  __half* k_meta;
  unsigned char* v_codes;
  __half* v_norm;
  unsigned char* modality;
  __host__ __device__ size_t unit(int b, int h) const { return (size_t)b * n_kv_heads + h; }
  __host__ __device__ int row_bytes() const { return 16 * bits; }
};

// packs the 32 codes cd[0..31] (channels 32 part .. 32 part + 31 of one token) into 4 * bits bytes of its bit stream
__device__ __forceinline__ void pack_quarter(const unsigned char* cd, int bits, unsigned char* dst) {
  unsigned long long lo = 0, hi = 0;
#pragma unroll
  for (int c = 0; c < 32; c++) {
    const int pos = bits * c;
    const unsigned long long v = cd[c];
    if (pos < 64) {
      lo |= v << pos;
      if (pos + bits > 64) hi |= v >> (64 - pos);
    } else {
      hi |= v << (pos - 64);
    }
  }
  const int nb = 4 * bits;   // 8, 12 or 16 bytes
  for (int k = 0; k < nb; k++) dst[k] = (unsigned char)((k < 8 ? lo >> (8 * k) : hi >> (8 * (k - 8))) & 0xffu);
}

// code of channel c in a token's bit stream
__device__ __forceinline__ unsigned load_code(const unsigned char* row, int bits, int c) {
  const int pos = bits * c, byte = pos >> 3;
  const unsigned w = (unsigned)row[byte] | ((unsigned)row[byte + ((pos & 7) + bits > 8 ? 1 : 0)] << 8);
  return (w >> (pos & 7)) & ((1u << bits) - 1u);
}

struct QuantSmem {
  float z[W][D + 1];
  unsigned char code[W][D];
  unsigned char mod[W];
};

// grid (windows, heads, batch), 128 threads
__global__ void __launch_bounds__(128) k_ladder_keys(LadderView cv, const __half* __restrict__ k, long long sb, long long sh,
                                                     long long st, const float* __restrict__ signs) {
  __shared__ QuantSmem sm;
  const int win = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const size_t u = cv.unit(b, h);
  const float4 sg = *reinterpret_cast<const float4*>(signs + 4 * lane);
  for (int kk = 0; kk < 8; kk++) {
    const int i = warp * 8 + kk;
    const float4 x = load_row4(k + b * sb + h * sh + (long long)(win * W + i) * st, lane);
    float n = warp_norm(x);
    const __half nh = __float2half_rn(n);
    const float nf = __half2float(nh);
    const float cinv = nf != 0.0f ? __fdiv_rn(RSQRT_D, nf) : 0.0f;
    const float4 y = warp_fwht(make_float4(__fmul_rn(sg.x, x.x), __fmul_rn(sg.y, x.y), __fmul_rn(sg.z, x.z), __fmul_rn(sg.w, x.w)), lane);
    // a zero vector (norm 0) has z = +0 in every coordinate
    sm.z[i][4 * lane + 0] = nf != 0.0f ? __fmul_rn(y.x, cinv) : 0.0f; sm.z[i][4 * lane + 1] = nf != 0.0f ? __fmul_rn(y.y, cinv) : 0.0f;
    sm.z[i][4 * lane + 2] = nf != 0.0f ? __fmul_rn(y.z, cinv) : 0.0f; sm.z[i][4 * lane + 3] = nf != 0.0f ? __fmul_rn(y.w, cinv) : 0.0f;
    if (lane == 0) cv.k_norm[u * cv.capacity + (size_t)win * W + i] = nh;
  }
  __syncthreads();
  {
    const int c = tid;
    const float L = (float)((1 << cv.bits) - 1);
    float mn = sm.z[0][c], mx = mn;
    for (int i = 1; i < W; i++) { const float v = sm.z[i][c]; mn = fminf(mn, v); mx = fmaxf(mx, v); }
    const __half mh = __float2half_rn(mn);
    const float mf = __half2float(mh);
    float range = __fsub_rn(mx, mf);
    range = range < 0.0f ? 0.0f : range;
    const __half s16 = __float2half_rn(__fdiv_rn(range, L));
    const float sf = __half2float(s16);
    __half* meta = cv.k_meta + ((u * (cv.capacity / W) + win) * D + c) * 2;
    meta[0] = mh; meta[1] = s16;
    const float r = sf > 0.0f ? __fdiv_rn(1.0f, sf) : 0.0f;
    for (int i = 0; i < W; i++) {
      float q = rintf(__fmul_rn(__fsub_rn(sm.z[i][c], mf), r));
      q = q < 0.0f ? 0.0f : (q > L ? L : q);
      sm.code[i][c] = sf > 0.0f ? (unsigned char)q : (unsigned char)0;
    }
  }
  __syncthreads();
  {
    const int i = tid >> 2, part = tid & 3;
    unsigned char* row = cv.k_codes + (u * cv.capacity + (size_t)win * W + i) * cv.row_bytes();
    pack_quarter(&sm.code[i][32 * part], cv.bits, row + 4 * cv.bits * part);
  }
}

struct ValueSmem {
  __align__(16) float x[W][D + 4];   // the window's value rows (fp32), 16-byte aligned rows
  unsigned char code[W][D];
  unsigned char mod[W];
  float inv[W];
  int uniform;
};

__global__ void __launch_bounds__(128) k_ladder_values(LadderView cv, const __half* __restrict__ v, long long sb, long long sh,
                                                       long long st, const unsigned char* __restrict__ modality, int n_tokens,
                                                       const float* __restrict__ R, int n_R) {
  __shared__ ValueSmem sm;
  const int win = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const size_t u = cv.unit(b, h);
  if (tid < W) {
    unsigned m = modality[(size_t)b * n_tokens + win * W + tid];
    m = m > 2 ? 0 : m;
    sm.mod[tid] = (unsigned char)m;
    if (h == 0) cv.modality[(size_t)b * cv.capacity + win * W + tid] = (unsigned char)m;
    const unsigned m0 = __shfl_sync(0xffffffffu, m, 0);
    const int uni = __all_sync(0xffffffffu, m == m0);
    if (tid == 0) sm.uniform = uni;
  }
  for (int kk = 0; kk < 8; kk++) {
    const int i = warp * 8 + kk;
    const float4 x = load_row4(v + b * sb + h * sh + (long long)(win * W + i) * st, lane);
    const float n = warp_norm(x);
    const __half nh = __float2half_rn(n);
    const float nf = __half2float(nh);
    *reinterpret_cast<float4*>(&sm.x[i][4 * lane]) = x;
    if (lane == 0) {
      cv.v_norm[u * cv.capacity + (size_t)win * W + i] = nh;
      sm.inv[i] = nf != 0.0f ? __fdiv_rn(1.0f, nf) : 0.0f;
    }
  }
  __syncthreads();
  {
    // thread = output coordinate c: z_c = (sum_k R_m[c][k] v_k) / norm as one fused-multiply-add chain in ascending k
    const int c = tid, nth = (1 << cv.bits) - 1;
    const float* Rset = R + (size_t)(n_R == 1 ? 0 : h) * 3 * D * D;
    const float* th = c_thresholds[cv.bits - 2];
    if (sm.uniform) {   // one matrix for the window: every row element is read once for the 32 tokens
      const float4* Rrow = reinterpret_cast<const float4*>(Rset + ((size_t)sm.mod[0] * D + c) * D);
      float acc[W];
#pragma unroll
      for (int i = 0; i < W; i++) acc[i] = 0.0f;
      for (int k4 = 0; k4 < D / 4; k4++) {
        const float4 r4 = __ldg(Rrow + k4);
#pragma unroll
        for (int i = 0; i < W; i++) {
          const float4 x4 = *reinterpret_cast<const float4*>(&sm.x[i][4 * k4]);
          float a = acc[i];
          a = __fmaf_rn(r4.x, x4.x, a);
          a = __fmaf_rn(r4.y, x4.y, a);
          a = __fmaf_rn(r4.z, x4.z, a);
          a = __fmaf_rn(r4.w, x4.w, a);
          acc[i] = a;
        }
      }
#pragma unroll
      for (int i = 0; i < W; i++) {
        const float z = __fmul_rn(acc[i], sm.inv[i]);
        int code = 0;
        for (int j = 0; j < nth; j++) code += z > th[j];
        sm.code[i][c] = (unsigned char)code;
      }
    } else {
      for (int i = 0; i < W; i++) {
        const float4* Rrow = reinterpret_cast<const float4*>(Rset + ((size_t)sm.mod[i] * D + c) * D);
        float a = 0.0f;
        for (int k4 = 0; k4 < D / 4; k4++) {
          const float4 r4 = __ldg(Rrow + k4);
          const float4 x4 = *reinterpret_cast<const float4*>(&sm.x[i][4 * k4]);
          a = __fmaf_rn(r4.x, x4.x, a);
          a = __fmaf_rn(r4.y, x4.y, a);
          a = __fmaf_rn(r4.z, x4.z, a);
          a = __fmaf_rn(r4.w, x4.w, a);
        }
        const float z = __fmul_rn(a, sm.inv[i]);
        int code = 0;
        for (int j = 0; j < nth; j++) code += z > th[j];
        sm.code[i][c] = (unsigned char)code;
      }
    }
  }
  __syncthreads();
  {
    const int i = tid >> 2, part = tid & 3;
    unsigned char* row = cv.v_codes + (u * cv.capacity + (size_t)win * W + i) * cv.row_bytes();
    pack_quarter(&sm.code[i][32 * part], cv.bits, row + 4 * cv.bits * part);
  }
}

}  // namespace
}  // namespace okq

namespace okq {
namespace {

constexpr int LD_THREADS = 256;

struct DecodeSmemL {
  float qrot[GP_L][D];        // rotated queries H D q / sqrt(128)
  float wgt[GP_L][D];         // q'_c s_c of the window
  float lev[16];              // value levels
  float m[D], s[D];
  float bias[GP_L];
  float sc[GP_L][W];          // scores, then numerators p * |v|
  float alpha[GP_L];
  float acc[3][GP_L][D];      // end: rotated-basis sums per modality
  float linv[GP_L];
  unsigned char mod[W];
  __align__(16) unsigned char kc[W * 64], vc[W * 64];   // the window's code rows (W * 16 * bits bytes each), staged
};

// grid (heads, batch), 256 threads: warp j = head j for the query rotation and the softmax; thread (c, hh) = channel
// c, heads 4 hh .. 4 hh + 3 for the value sums
__global__ void __launch_bounds__(LD_THREADS) k_ladder_decode(LadderView cv, int n_tokens, const __half* __restrict__ q,
                                                             float sm_scale, const float* __restrict__ signs,
                                                             const float* __restrict__ R, int n_R, float* __restrict__ out) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  DecodeSmemL& sm = *reinterpret_cast<DecodeSmemL*>(smem_raw);
  const int h = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = cv.n_q_heads / cv.n_kv_heads, bits = cv.bits;
  const size_t u = cv.unit(b, h);
  const int rb = cv.row_bytes();
  constexpr float LOG2E = 1.4426950408889634f;
  // rotated queries
  {
    float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
    if (warp < G) {
      const float4 x = load_row4(q + ((size_t)b * cv.n_q_heads + (size_t)h * G + warp) * D, lane);
      const float4 sg = *reinterpret_cast<const float4*>(signs + 4 * lane);
      y = warp_fwht(make_float4(sg.x * x.x, sg.y * x.y, sg.z * x.z, sg.w * x.w), lane);
    }
    sm.qrot[warp][4 * lane + 0] = y.x * RSQRT_D; sm.qrot[warp][4 * lane + 1] = y.y * RSQRT_D;
    sm.qrot[warp][4 * lane + 2] = y.z * RSQRT_D; sm.qrot[warp][4 * lane + 3] = y.w * RSQRT_D;
  }
  if (tid < 16) sm.lev[tid] = c_levels[bits - 2][tid];
  const int c = tid & (D - 1), hh = tid >> 7;
  float acc[3][4];
#pragma unroll
  for (int m = 0; m < 3; m++)
#pragma unroll
    for (int j = 0; j < 4; j++) acc[m][j] = 0.f;
  float run_m = -INFINITY, run_l = 0.f;   // per warp = head (every lane holds the same value)
  __syncthreads();
  const int n_win = n_tokens / W;
  for (int win = 0; win < n_win; win++) {
    const size_t tok0 = u * cv.capacity + (size_t)win * W;
    if (tid < D) {
      const __half* meta = cv.k_meta + ((u * (cv.capacity / W) + win) * D + tid) * 2;
      sm.m[tid] = __half2float(meta[0]); sm.s[tid] = __half2float(meta[1]);
    }
    if (tid < W) sm.mod[tid] = cv.modality[(size_t)b * cv.capacity + (size_t)win * W + tid];
    {   // the window's rows are contiguous: W * rb bytes = 2 * bits * 32 pieces of 16 bytes per side
      const int n16 = W * rb / 16;
      const uint4* ksrc = reinterpret_cast<const uint4*>(cv.k_codes + tok0 * rb);
      const uint4* vsrc = reinterpret_cast<const uint4*>(cv.v_codes + tok0 * rb);
      if (tid < n16) reinterpret_cast<uint4*>(sm.kc)[tid] = ksrc[tid];
      else if (tid >= 128 && tid - 128 < n16) reinterpret_cast<uint4*>(sm.vc)[tid - 128] = vsrc[tid - 128];
    }
    __syncthreads();
    {   // weights and bias of head `warp`
      float bsum = 0.f;
#pragma unroll
      for (int k4 = 0; k4 < 4; k4++) {
        const int cc = 4 * lane + k4;
        const float qv = sm.qrot[warp][cc];
        sm.wgt[warp][cc] = qv * sm.s[cc];
        bsum = fmaf(qv, sm.m[cc], bsum);
      }
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) bsum += __shfl_xor_sync(0xffffffffu, bsum, d);
      if (lane == 0) sm.bias[warp] = bsum;
    }
    __syncthreads();
    // scores: warp w takes tokens 4 w .. 4 w + 3, a lane four channels
    for (int tt = 0; tt < 4; tt++) {
      const int t = 4 * warp + tt;
      const unsigned char* row = sm.kc + t * rb;
      float cd[4];
#pragma unroll
      for (int k4 = 0; k4 < 4; k4++) cd[k4] = (float)load_code(row, bits, 4 * lane + k4);
      const float kn = __half2float(cv.k_norm[tok0 + t]) * sm_scale * LOG2E;
#pragma unroll
      for (int j = 0; j < GP_L; j++) {
        float d = 0.f;
#pragma unroll
        for (int k4 = 0; k4 < 4; k4++) d = fmaf(sm.wgt[j][4 * lane + k4], cd[k4], d);
#pragma unroll
        for (int sft = 1; sft < 32; sft <<= 1) d += __shfl_xor_sync(0xffffffffu, d, sft);
        if (lane == 0) sm.sc[j][t] = (d + sm.bias[j]) * kn;
      }
    }
    __syncthreads();
    {   // online softmax of head `warp` over the window's 32 tokens (lane = token)
      const float x = sm.sc[warp][lane];
      float mx = x;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
      const float m_new = fmaxf(run_m, mx);
      const float al = exp2f(run_m - m_new);
      const float p = exp2f(x - m_new);
      float ps = p;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) ps += __shfl_xor_sync(0xffffffffu, ps, d);
      run_l = run_l * al + ps;
      run_m = m_new;
      sm.sc[warp][lane] = p * __half2float(cv.v_norm[tok0 + lane]);
      if (lane == 0) sm.alpha[warp] = al;
    }
    __syncthreads();
    {   // value sums in the rotated basis of each token's modality
      float al[4];
#pragma unroll
      for (int j = 0; j < 4; j++) al[j] = sm.alpha[4 * hh + j];
#pragma unroll
      for (int m = 0; m < 3; m++)
#pragma unroll
        for (int j = 0; j < 4; j++) acc[m][j] *= al[j];
      for (int t = 0; t < W; t++) {
        const float lv = sm.lev[load_code(sm.vc + t * rb, bits, c)];
        const int md = sm.mod[t];   // the same for every thread: a uniform branch around register-indexed sums
        if (md == 0) {
#pragma unroll
          for (int j = 0; j < 4; j++) acc[0][j] = fmaf(sm.sc[4 * hh + j][t], lv, acc[0][j]);
        } else if (md == 1) {
#pragma unroll
          for (int j = 0; j < 4; j++) acc[1][j] = fmaf(sm.sc[4 * hh + j][t], lv, acc[1][j]);
        } else {
#pragma unroll
          for (int j = 0; j < 4; j++) acc[2][j] = fmaf(sm.sc[4 * hh + j][t], lv, acc[2][j]);
        }
      }
    }
    __syncthreads();
  }
  // R_m^T once per head, then the normalisation
#pragma unroll
  for (int m = 0; m < 3; m++)
#pragma unroll
    for (int j = 0; j < 4; j++) sm.acc[m][4 * hh + j][c] = acc[m][j];
  if (lane == 0) sm.linv[warp] = run_l > 0.f ? 1.0f / run_l : 0.f;
  __syncthreads();
  const float* Rset = R + (size_t)(n_R == 1 ? 0 : h) * 3 * D * D;
  float o[4] = {0.f, 0.f, 0.f, 0.f};
  for (int m = 0; m < 3; m++)
    for (int r = 0; r < D; r++) {
      const float rv = __ldg(Rset + ((size_t)m * D + r) * D + c);
#pragma unroll
      for (int j = 0; j < 4; j++) o[j] = fmaf(rv, sm.acc[m][4 * hh + j][r], o[j]);
    }
#pragma unroll
  for (int j = 0; j < 4; j++) {
    const int head = 4 * hh + j;
    if (head < G) out[((size_t)b * cv.n_q_heads + (size_t)h * G + head) * D + c] = o[j] * sm.linv[head];
  }
}

// TurboQuant codec (Preliminaries, Eq. 2-3): norm, randomised Hadamard rotation, nearest level of the fixed codebook;
// no window statistics, no modality rotation.  32 vectors per block of 128 threads.
__global__ void __launch_bounds__(128) k_turboquant_encode(const __half* __restrict__ x, long long n, int bits,
                                                           const float* __restrict__ signs, unsigned char* __restrict__ codes,
                                                           __half* __restrict__ norms) {
  __shared__ unsigned char code[W][D];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long base = (long long)blockIdx.x * W;
  const float4 sg = *reinterpret_cast<const float4*>(signs + 4 * lane);
  const float* th = c_thresholds[bits - 2];
  const int nth = (1 << bits) - 1;
  for (int kk = 0; kk < 8; kk++) {
    const int i = warp * 8 + kk;
    if (base + i >= n) break;
    const float4 v = load_row4(x + (base + i) * D, lane);
    const float nrm = warp_norm(v);
    const __half nh = __float2half_rn(nrm);
    const float nf = __half2float(nh);
    const float cinv = nf != 0.0f ? __fdiv_rn(RSQRT_D, nf) : 0.0f;
    const float4 y = warp_fwht(make_float4(__fmul_rn(sg.x, v.x), __fmul_rn(sg.y, v.y), __fmul_rn(sg.z, v.z), __fmul_rn(sg.w, v.w)), lane);
    const float z[4] = {nf != 0.0f ? __fmul_rn(y.x, cinv) : 0.0f, nf != 0.0f ? __fmul_rn(y.y, cinv) : 0.0f,
                        nf != 0.0f ? __fmul_rn(y.z, cinv) : 0.0f, nf != 0.0f ? __fmul_rn(y.w, cinv) : 0.0f};
#pragma unroll
    for (int k4 = 0; k4 < 4; k4++) {
      int cd = 0;
      for (int j = 0; j < nth; j++) cd += z[k4] > th[j];
      code[i][4 * lane + k4] = (unsigned char)cd;
    }
    if (lane == 0) norms[base + i] = nh;
  }
  __syncthreads();
  const int i = tid >> 2, part = tid & 3;
  if (base + i < n) pack_quarter(&code[i][32 * part], bits, codes + (base + i) * 16 * bits + 4 * bits * part);
}

// x_hat = |x| H^T level[code], H^T y = diag(signs) Had y / sqrt(128); one warp per vector
__global__ void __launch_bounds__(128) k_turboquant_decode(const unsigned char* __restrict__ codes, const __half* __restrict__ norms,
                                                           long long n, int bits, const float* __restrict__ signs,
                                                           float* __restrict__ x_hat) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long i = (long long)blockIdx.x * 4 + warp;
  if (i >= n) return;
  const unsigned char* row = codes + i * 16 * bits;
  const float* lv = c_levels[bits - 2];
  const float4 y = warp_fwht(make_float4(lv[load_code(row, bits, 4 * lane + 0)], lv[load_code(row, bits, 4 * lane + 1)],
                                         lv[load_code(row, bits, 4 * lane + 2)], lv[load_code(row, bits, 4 * lane + 3)]), lane);
  const float4 sg = *reinterpret_cast<const float4*>(signs + 4 * lane);
  const float f = RSQRT_D * __half2float(norms[i]);
  *reinterpret_cast<float4*>(x_hat + i * D + 4 * lane) = make_float4(sg.x * y.x * f, sg.y * y.y * f, sg.z * y.z * f, sg.w * y.w * f);
}

okq_status check_ladder(const okq_ladder_cache* c, int n_tokens) {
  if (!c) return OKQ_ERR_INVALID_ARG;
  if (c->bits < 2 || c->bits > 4) return OKQ_ERR_UNSUPPORTED;
  if (c->batch <= 0 || c->n_kv_heads <= 0 || c->n_q_heads <= 0 || c->capacity <= 0 || c->capacity % W) return OKQ_ERR_INVALID_ARG;
  if (c->n_q_heads % c->n_kv_heads || c->n_q_heads / c->n_kv_heads > GP_L) return OKQ_ERR_UNSUPPORTED;
  if (n_tokens < 0 || n_tokens % W || n_tokens > c->capacity) return OKQ_ERR_INVALID_ARG;
  if (!c->k_codes || !c->k_norm || !c->k_meta || !c->v_codes || !c->v_norm || !c->modality) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(c->k_codes) || !aligned16(c->k_norm) || !aligned16(c->k_meta) || !aligned16(c->v_codes) || !aligned16(c->v_norm))
    return OKQ_ERR_ALIGNMENT;
  return OKQ_OK;
}

LadderView ladder_view(const okq_ladder_cache* c) {
  LadderView v;
  v.batch = c->batch; v.n_kv_heads = c->n_kv_heads; v.n_q_heads = c->n_q_heads; v.capacity = c->capacity; v.bits = c->bits;
  v.k_codes = static_cast<unsigned char*>(c->k_codes); v.k_norm = static_cast<__half*>(c->k_norm);
  v.k_meta = static_cast<__half*>(c->k_meta); v.v_codes = static_cast<unsigned char*>(c->v_codes);
  v.v_norm = static_cast<__half*>(c->v_norm); v.modality = c->modality;
  return v;
}

}  // namespace
}  // namespace okq

using namespace okq;

extern "C" {

int32_t okq_ladder_codebook(int32_t bits, float* levels, float* thresholds) {
  if (bits < 2 || bits > 4 || !levels || !thresholds) return 0;
  const int n = 1 << bits;
  for (int i = 0; i < n; i++) levels[i] = h_levels[bits - 2][i];
  for (int i = 0; i < n - 1; i++) thresholds[i] = h_thresholds[bits - 2][i];
  return n;
}

okq_status okq_ladder_quantize_keys(const okq_ladder_cache* cache, const void* k_fp16, const int64_t strides[3],
                                    int32_t n_tokens, const float* signs, void* stream) {
  okq_status st = check_ladder(cache, n_tokens);
  if (st != OKQ_OK) return st;
  if (!k_fp16 || !strides || !signs) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(k_fp16) || !aligned16(signs) || strides[0] % 8 || strides[1] % 8 || strides[2] % 8) return OKQ_ERR_ALIGNMENT;
  if (n_tokens == 0) return OKQ_OK;
  const dim3 grid(n_tokens / W, cache->n_kv_heads, cache->batch);
  k_ladder_keys<<<grid, 128, 0, static_cast<cudaStream_t>(stream)>>>(ladder_view(cache), static_cast<const __half*>(k_fp16),
                                                                     strides[0], strides[1], strides[2], signs);
  return launch_status();
}

okq_status okq_ladder_quantize_values(const okq_ladder_cache* cache, const void* v_fp16, const int64_t strides[3],
                                      int32_t n_tokens, const uint8_t* modality, const float* R, int32_t n_R,
                                      void* stream) {
  okq_status st = check_ladder(cache, n_tokens);
  if (st != OKQ_OK) return st;
  if (!v_fp16 || !strides || !modality || !R || (n_R != 1 && n_R != cache->n_kv_heads)) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(v_fp16) || !aligned16(R) || strides[0] % 8 || strides[1] % 8 || strides[2] % 8) return OKQ_ERR_ALIGNMENT;
  if (n_tokens == 0) return OKQ_OK;
  const dim3 grid(n_tokens / W, cache->n_kv_heads, cache->batch);
  k_ladder_values<<<grid, 128, 0, static_cast<cudaStream_t>(stream)>>>(ladder_view(cache), static_cast<const __half*>(v_fp16),
                                                                       strides[0], strides[1], strides[2], modality, n_tokens, R, n_R);
  return launch_status();
}

okq_status okq_ladder_decode_attention(const okq_ladder_cache* cache, int32_t n_tokens, const void* q, float sm_scale,
                                       const float* signs, const float* R, int32_t n_R, float* out, void* stream) {
  okq_status st = check_ladder(cache, n_tokens);
  if (st != OKQ_OK) return st;
  if (!q || !signs || !R || !out || (n_R != 1 && n_R != cache->n_kv_heads)) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(signs) || !aligned16(R) || !aligned16(out)) return OKQ_ERR_ALIGNMENT;
  static thread_local unsigned long long attr_mask = 0;
  int attr_dev = 0;
  if (attr_needed(attr_mask, attr_dev)) {
    cudaError_t e = cudaFuncSetAttribute(k_ladder_decode, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DecodeSmemL));
    if (e != cudaSuccess) { set_last_cuda_error((int)e); return OKQ_ERR_CUDA; }
    attr_done(attr_mask, attr_dev);
  }
  k_ladder_decode<<<dim3(cache->n_kv_heads, cache->batch), LD_THREADS, sizeof(DecodeSmemL), static_cast<cudaStream_t>(stream)>>>(
      ladder_view(cache), n_tokens, static_cast<const __half*>(q), sm_scale, signs, R, n_R, out);
  return launch_status();
}

okq_status okq_turboquant_encode(const void* x_fp16, int64_t n_vectors, int32_t bits, const float* signs, uint8_t* codes,
                                 void* norms, void* stream) {
  if (bits < 2 || bits > 4) return OKQ_ERR_UNSUPPORTED;
  if (n_vectors < 0 || !x_fp16 || !signs || !codes || !norms) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(x_fp16) || !aligned16(signs) || !aligned16(codes)) return OKQ_ERR_ALIGNMENT;
  if (n_vectors == 0) return OKQ_OK;
  if ((n_vectors + W - 1) / W > 0x7fffffffLL) return OKQ_ERR_CAPACITY;
  k_turboquant_encode<<<(unsigned)((n_vectors + W - 1) / W), 128, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __half*>(x_fp16), n_vectors, bits, signs, codes, static_cast<__half*>(norms));
  return launch_status();
}

okq_status okq_turboquant_decode(const uint8_t* codes, const void* norms, int64_t n_vectors, int32_t bits,
                                 const float* signs, float* x_hat, void* stream) {
  if (bits < 2 || bits > 4) return OKQ_ERR_UNSUPPORTED;
  if (n_vectors < 0 || !codes || !norms || !signs || !x_hat) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(codes) || !aligned16(signs) || !aligned16(x_hat)) return OKQ_ERR_ALIGNMENT;
  if (n_vectors == 0) return OKQ_OK;
  if ((n_vectors + 3) / 4 > 0x7fffffffLL) return OKQ_ERR_CAPACITY;
  k_turboquant_decode<<<(unsigned)((n_vectors + 3) / 4), 128, 0, static_cast<cudaStream_t>(stream)>>>(
      codes, static_cast<const __half*>(norms), n_vectors, bits, signs, x_hat);
  return launch_status();
}

}  // extern "C"
