// Offline calibration of the per-modality value rotations (Eq. 5, R_m = H U_m^T).
//
//   k_calib_rows / k_calib_cols   alpha = softmax(q k^T * scale) in 64 x 64 tiles on the tensor cores
//                                 (mma.sync, fp16 products, fp32 sums): first the row maximum and
//                                 normaliser, then the column sums of alpha^2
//   k_calib_wsum                  w_j: fixed-order sum of the per-(query tile, head) column sums
//   k_calib_wmax, k_calib_moments C_m = sum w_j v_j^T v_j, tensor cores, values staged transposed
//   k_calib_csum                  fixed-order sum of the per-chunk partial moments
//   k_calib_eigen                 cyclic Jacobi (fp64, one block), ordering, signs, R = H U^T
#include "../../include/okq_calib.h"
#include "okq_common.cuh"

namespace okq {
namespace {

constexpr int TQ = 64;          // queries per block (4 warps x 16 rows) and keys per tile
constexpr int KS_STRIDE = D + 8;  // halves per staged key row: 272 bytes, conflict-free fragment reads

__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// One pass over the key tiles of a 64-query block of one head.
//   PASS 0: row maximum m and normaliser l of the softmax -> rowstat[(g * n + i) * 2 + {0, 1}]
//   PASS 1: column sums of alpha^2 over the block's queries -> partial[(itile * G + g) * n + j]
// grid (n_itiles, G), 128 threads.
template <int PASS>
__global__ void __launch_bounds__(128) k_calib_pass(const __half* __restrict__ q, const __half* __restrict__ k, int G, int n,
                                                   float scale, int causal, float* __restrict__ rowstat,
                                                   float* __restrict__ partial) {
  __shared__ __align__(16) __half ks[TQ * KS_STRIDE];
  __shared__ float colsum[4][TQ];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int itile = blockIdx.x, head = blockIdx.y;
  const int i0 = itile * TQ + warp * 16 + g, i1 = i0 + 8;   // this lane's two query rows
  // A fragments of the queries: rows i0 / i1, 8 k-steps of 16 channels
  uint32_t qa[8][4];
  const __half* qh = q + (size_t)head * n * D;
#pragma unroll
  for (int s = 0; s < 8; s++) {
    const int c = 16 * s + 2 * t;
    qa[s][0] = i0 < n ? *reinterpret_cast<const uint32_t*>(qh + (size_t)i0 * D + c) : 0u;
    qa[s][1] = i1 < n ? *reinterpret_cast<const uint32_t*>(qh + (size_t)i1 * D + c) : 0u;
    qa[s][2] = i0 < n ? *reinterpret_cast<const uint32_t*>(qh + (size_t)i0 * D + c + 8) : 0u;
    qa[s][3] = i1 < n ? *reinterpret_cast<const uint32_t*>(qh + (size_t)i1 * D + c + 8) : 0u;
  }
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  if (PASS == 1) {
    if (i0 < n) { m0 = rowstat[((size_t)head * n + i0) * 2]; l0 = 1.0f / rowstat[((size_t)head * n + i0) * 2 + 1]; }
    if (i1 < n) { m1 = rowstat[((size_t)head * n + i1) * 2]; l1 = 1.0f / rowstat[((size_t)head * n + i1) * 2 + 1]; }
  }
  const int n_jt = causal ? itile + 1 : (n + TQ - 1) / TQ;
  for (int jt = 0; jt < n_jt; jt++) {
    __syncthreads();   // the previous tile's fragments and column sums have been consumed
    for (int idx = tid; idx < TQ * (D / 8); idx += 128) {
      const int r = idx >> 4, c8 = idx & 15, j = jt * TQ + r;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (j < n) v = *reinterpret_cast<const uint4*>(k + (size_t)j * D + c8 * 8);
      *reinterpret_cast<uint4*>(&ks[r * KS_STRIDE + c8 * 8]) = v;
    }
    __syncthreads();
    float s[8][4];
#pragma unroll
    for (int nt = 0; nt < 8; nt++) {
      float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int st = 0; st < 8; st++) {
        const __half* kr = &ks[(nt * 8 + g) * KS_STRIDE + 16 * st + 2 * t];
        mma16816(d, qa[st][0], qa[st][1], qa[st][2], qa[st][3], *reinterpret_cast<const uint32_t*>(kr),
                 *reinterpret_cast<const uint32_t*>(kr + 8));
      }
      // d[0], d[1]: row i0, keys j, j+1;  d[2], d[3]: row i1
      const int j = jt * TQ + nt * 8 + 2 * t;
#pragma unroll
      for (int e = 0; e < 4; e++) {
        const int jj = j + (e & 1), ii = (e & 2) ? i1 : i0;
        const bool live = jj < n && ii < n && (!causal || jj <= ii);
        s[nt][e] = live ? d[e] * scale : -INFINITY;
      }
    }
    if (PASS == 0) {
      float t0 = -INFINITY, t1 = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 8; nt++) {
        t0 = fmaxf(t0, fmaxf(s[nt][0], s[nt][1]));
        t1 = fmaxf(t1, fmaxf(s[nt][2], s[nt][3]));
      }
      t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, 1)); t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, 2));
      t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, 1)); t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, 2));
      const float n0 = fmaxf(m0, t0), n1 = fmaxf(m1, t1);
      float a0 = 0.f, a1 = 0.f;
#pragma unroll
      for (int nt = 0; nt < 8; nt++) {
        if (n0 != -INFINITY) a0 += expf(s[nt][0] - n0) + expf(s[nt][1] - n0);
        if (n1 != -INFINITY) a1 += expf(s[nt][2] - n1) + expf(s[nt][3] - n1);
      }
      a0 += __shfl_xor_sync(0xffffffffu, a0, 1); a0 += __shfl_xor_sync(0xffffffffu, a0, 2);
      a1 += __shfl_xor_sync(0xffffffffu, a1, 1); a1 += __shfl_xor_sync(0xffffffffu, a1, 2);
      l0 = (m0 == -INFINITY ? 0.f : l0 * expf(m0 - n0)) + a0; m0 = n0;
      l1 = (m1 == -INFINITY ? 0.f : l1 * expf(m1 - n1)) + a1; m1 = n1;
    } else {
#pragma unroll
      for (int nt = 0; nt < 8; nt++) {
        float c0 = 0.f, c1 = 0.f;   // keys j, j+1: squares of this lane's two rows
        if (s[nt][0] != -INFINITY) { const float a = expf(s[nt][0] - m0) * l0; c0 += a * a; }
        if (s[nt][2] != -INFINITY) { const float a = expf(s[nt][2] - m1) * l1; c0 += a * a; }
        if (s[nt][1] != -INFINITY) { const float a = expf(s[nt][1] - m0) * l0; c1 += a * a; }
        if (s[nt][3] != -INFINITY) { const float a = expf(s[nt][3] - m1) * l1; c1 += a * a; }
#pragma unroll
        for (int dl = 4; dl < 32; dl <<= 1) {   // over the eight row groups g
          c0 += __shfl_xor_sync(0xffffffffu, c0, dl);
          c1 += __shfl_xor_sync(0xffffffffu, c1, dl);
        }
        if (g == 0) { colsum[warp][nt * 8 + 2 * t] = c0; colsum[warp][nt * 8 + 2 * t + 1] = c1; }
      }
      __syncthreads();
      if (tid < TQ) {
        const int j = jt * TQ + tid;
        if (j < n)
          partial[((size_t)itile * G + head) * n + j] = (colsum[0][tid] + colsum[1][tid]) + (colsum[2][tid] + colsum[3][tid]);
      }
    }
  }
  if (PASS == 0 && t == 0) {
    if (i0 < n) { rowstat[((size_t)head * n + i0) * 2] = m0; rowstat[((size_t)head * n + i0) * 2 + 1] = l0; }
    if (i1 < n) { rowstat[((size_t)head * n + i1) * 2] = m1; rowstat[((size_t)head * n + i1) * 2 + 1] = l1; }
  }
}

// w_j = sum over (query tile, head) of the column sums, in index order.  One thread per key.
__global__ void k_calib_wsum(const float* __restrict__ partial, int G, int n, int causal, float* __restrict__ w) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n) return;
  const int n_it = (n + TQ - 1) / TQ;
  float acc = 0.f;
  for (int it = causal ? j / TQ : 0; it < n_it; it++)
    for (int g = 0; g < G; g++) acc += partial[((size_t)it * G + g) * n + j];
  w[j] = acc;
}

// ---------------------------------------------------------------- weighted moments

constexpr int MT = 32;             // tokens per staged tile (two k-steps)
constexpr int VT_STRIDE = MT + 8;  // halves per transposed row: 80 bytes
constexpr int MAX_CHUNKS = 64;     // token ranges (blocks) per modality

// exponent e with 2^e >= max_j w_j (0 when all weights are 0): the weights are used as w_j * 2^-e <= 1
__global__ void k_calib_wmax(const float* __restrict__ w, int n, int* __restrict__ e_out) {
  __shared__ float red[32];
  float mx = 0.f;
  for (int j = threadIdx.x; j < n; j += blockDim.x) mx = fmaxf(mx, w[j]);
  for (int d = 16; d; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < (int)(blockDim.x >> 5); i++) mx = fmaxf(mx, red[i]);
    int e = 0;
    if (mx > 0.f) { frexpf(mx, &e); }   // mx = f * 2^e, f in [0.5, 1)
    *e_out = e;
  }
}

// grid (n_chunks, 3), 256 threads: block (chunk, m) adds the tokens of modality m in its token range into
// a 128 x 128 partial moment matrix.  Warp w owns rows 16 w .. 16 w + 15 (all 128 columns).
__global__ void __launch_bounds__(256) k_calib_moments(const __half* __restrict__ v, const float* __restrict__ w,
                                                      const unsigned char* __restrict__ modality, int n, int n_chunks,
                                                      const int* __restrict__ w_exp, float* __restrict__ partial) {
  __shared__ __align__(16) __half vt[D * VT_STRIDE];    // values, transposed: [channel][token]
  __shared__ __align__(16) __half xh[D * VT_STRIDE];    // w v, high fp16 term
  __shared__ __align__(16) __half xl[D * VT_STRIDE];    // w v, low fp16 term
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int chunk = blockIdx.x, m = blockIdx.y;
  const int n_tiles = (n + MT - 1) / MT;
  const int per = (n_tiles + n_chunks - 1) / n_chunks;
  const int t_begin = chunk * per, t_end = min(n_tiles, t_begin + per);
  const float wscale = exp2f((float)-(*w_exp));
  float acc[16][4];
#pragma unroll
  for (int nt = 0; nt < 16; nt++)
#pragma unroll
    for (int e = 0; e < 4; e++) acc[nt][e] = 0.f;
  for (int tile = t_begin; tile < t_end; tile++) {
    __syncthreads();
    for (int idx = tid; idx < MT * (D / 8); idx += 256) {
      const int r = idx >> 4, c8 = idx & 15, j = tile * MT + r;
      uint4 raw = make_uint4(0u, 0u, 0u, 0u);
      float wj = 0.f;
      if (j < n) {
        unsigned mm = modality[j];
        mm = mm > 2 ? 0 : mm;
        if ((int)mm == m) { raw = *reinterpret_cast<const uint4*>(v + (size_t)j * D + c8 * 8); wj = w[j] * wscale; }
      }
      const __half* hv = reinterpret_cast<const __half*>(&raw);
#pragma unroll
      for (int u = 0; u < 8; u++) {
        const float x = __half2float(hv[u]) * wj;
        const __half hi = __float2half_rn(x);
        vt[(c8 * 8 + u) * VT_STRIDE + r] = hv[u];
        xh[(c8 * 8 + u) * VT_STRIDE + r] = hi;
        xl[(c8 * 8 + u) * VT_STRIDE + r] = __float2half_rn(x - __half2float(hi));
      }
    }
    __syncthreads();
#pragma unroll
    for (int st = 0; st < MT / 16; st++) {
      const int row0 = (16 * warp + g) * VT_STRIDE + 16 * st + 2 * t, row1 = row0 + 8 * VT_STRIDE;
      const uint32_t h0 = *reinterpret_cast<const uint32_t*>(&xh[row0]), h1 = *reinterpret_cast<const uint32_t*>(&xh[row1]);
      const uint32_t h2 = *reinterpret_cast<const uint32_t*>(&xh[row0 + 8]), h3 = *reinterpret_cast<const uint32_t*>(&xh[row1 + 8]);
      const uint32_t l0 = *reinterpret_cast<const uint32_t*>(&xl[row0]), l1 = *reinterpret_cast<const uint32_t*>(&xl[row1]);
      const uint32_t l2 = *reinterpret_cast<const uint32_t*>(&xl[row0 + 8]), l3 = *reinterpret_cast<const uint32_t*>(&xl[row1 + 8]);
#pragma unroll
      for (int nt = 0; nt < 16; nt++) {
        const __half* br = &vt[(nt * 8 + g) * VT_STRIDE + 16 * st + 2 * t];
        const uint32_t b0 = *reinterpret_cast<const uint32_t*>(br), b1 = *reinterpret_cast<const uint32_t*>(br + 8);
        mma16816(acc[nt], h0, h1, h2, h3, b0, b1);
        mma16816(acc[nt], l0, l1, l2, l3, b0, b1);
      }
    }
  }
  float* out = partial + ((size_t)chunk * 3 + m) * D * D;
#pragma unroll
  for (int nt = 0; nt < 16; nt++) {
    const int col = nt * 8 + 2 * t, r0 = 16 * warp + g;
    *reinterpret_cast<float2*>(&out[r0 * D + col]) = make_float2(acc[nt][0], acc[nt][1]);
    *reinterpret_cast<float2*>(&out[(r0 + 8) * D + col]) = make_float2(acc[nt][2], acc[nt][3]);
  }
}

// C = 2^e * (sum of the partial matrices in chunk order), made exactly symmetric.  One thread per element pair.
__global__ void k_calib_csum(const float* __restrict__ partial, int n_chunks, const int* __restrict__ w_exp,
                             float* __restrict__ C) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= 3 * D * D) return;
  const int m = idx / (D * D), a = (idx / D) % D, b = idx % D;
  if (b < a) return;
  float s0 = 0.f, s1 = 0.f;
  for (int c = 0; c < n_chunks; c++) {
    s0 += partial[((size_t)c * 3 + m) * D * D + a * D + b];
    s1 += partial[((size_t)c * 3 + m) * D * D + b * D + a];
  }
  const float val = 0.5f * (s0 + s1) * exp2f((float)*w_exp);
  C[(size_t)m * D * D + a * D + b] = val;
  C[(size_t)m * D * D + b * D + a] = val;
}

// ---------------------------------------------------------------- eigenbasis and rotation

constexpr int EIG_THREADS = 1024;
constexpr int MAX_SWEEPS = 30;

// Cyclic Jacobi on a symmetric 128 x 128 matrix in fp64, one block.  A lives in shared memory (128 KB), the
// accumulated rotations as V^T (row l = eigenvector l) in global memory.  A sweep is 127 rounds of 64
// disjoint pairs (round-robin pairing); a round computes its 64 rotations, then applies them to the rows
// and to the columns of A and to the rows of V^T.  Stops after a sweep in which no rotation was needed.
// Then: eigenvalues in descending order, every eigenvector with its largest-magnitude component positive,
// R = H U^T with H = Had_128 diag(signs) / sqrt(128).
__global__ void __launch_bounds__(EIG_THREADS) k_calib_eigen(const float* __restrict__ C, const float* __restrict__ signs,
                                                           double* __restrict__ vt, float* __restrict__ R,
                                                           float* __restrict__ lambda, int* __restrict__ sweeps_out) {
  extern __shared__ __align__(16) unsigned char eig_raw[];
  double* A = reinterpret_cast<double*>(eig_raw);                 // [128][128]
  __shared__ double rc[64], rs[64];
  __shared__ int rp[64], rq[64];
  __shared__ int rotated;
  __shared__ int order[D];
  __shared__ double flip[D];
  const int tid = threadIdx.x;
  for (int idx = tid; idx < D * D; idx += EIG_THREADS) {
    const int a = idx / D, b = idx % D;
    A[idx] = 0.5 * ((double)C[a * D + b] + (double)C[b * D + a]);
    vt[idx] = a == b ? 1.0 : 0.0;
  }
  // the scale below which an off-diagonal element is left alone
  __shared__ double tiny;
  if (tid == 0) {
    double tr = 0.0;
    for (int i = 0; i < D; i++) tr += fabs((double)C[i * D + i]);
    tiny = tr * 1e-18;
  }
  __syncthreads();
  int sweeps = 0;
  for (; sweeps < MAX_SWEEPS; sweeps++) {
    if (tid == 0) rotated = 0;
    __syncthreads();
    for (int round = 0; round < D - 1; round++) {
      if (tid < 64) {
        int p, q;
        if (tid == 0) { p = round; q = D - 1; }
        else { p = (round + tid) % (D - 1); q = (round - tid + (D - 1)) % (D - 1); }
        if (p > q) { const int x = p; p = q; q = x; }
        const double apq = A[p * D + q], app = A[p * D + p], aqq = A[q * D + q];
        double c = 1.0, s = 0.0;
        if (fabs(apq) > tiny && fabs(apq) > 1e-17 * sqrt(fabs(app * aqq))) {
          const double tau = (aqq - app) / (2.0 * apq);
          const double tt = (tau >= 0.0 ? 1.0 : -1.0) / (fabs(tau) + sqrt(1.0 + tau * tau));
          c = 1.0 / sqrt(1.0 + tt * tt);
          s = tt * c;
          rotated = 1;
        }
        rc[tid] = c; rs[tid] = s; rp[tid] = p; rq[tid] = q;
      }
      __syncthreads();
      // rows: A <- J^T A, and V^T <- J^T V^T (the rows of V^T are the eigenvector estimates)
      for (int idx = tid; idx < 64 * D; idx += EIG_THREADS) {
        const int kk = idx >> 7, j = idx & (D - 1);
        const double c = rc[kk], s = rs[kk];
        if (s != 0.0) {
          const int p = rp[kk], q = rq[kk];
          const double ap = A[p * D + j], aq = A[q * D + j];
          A[p * D + j] = c * ap - s * aq;
          A[q * D + j] = s * ap + c * aq;
          const double vp = vt[p * D + j], vq = vt[q * D + j];
          vt[p * D + j] = c * vp - s * vq;
          vt[q * D + j] = s * vp + c * vq;
        }
      }
      __syncthreads();
      // columns: A <- A J
      for (int idx = tid; idx < 64 * D; idx += EIG_THREADS) {
        const int kk = idx & 63, i = idx >> 6;
        const double c = rc[kk], s = rs[kk];
        if (s != 0.0) {
          const int p = rp[kk], q = rq[kk];
          const double ap = A[i * D + p], aq = A[i * D + q];
          A[i * D + p] = c * ap - s * aq;
          A[i * D + q] = s * ap + c * aq;
        }
      }
      __syncthreads();
    }
    if (!rotated) break;
    __syncthreads();
  }
  if (tid == 0 && sweeps_out) *sweeps_out = sweeps;
  // descending order (ties by index) and sign convention
  if (tid < D) {
    const double li = A[tid * D + tid];
    int rank = 0;
    for (int j = 0; j < D; j++) {
      const double lj = A[j * D + j];
      rank += (lj > li) || (lj == li && j < tid);
    }
    order[rank] = tid;
    double best = 0.0, val = 1.0;
    for (int j = 0; j < D; j++) {
      const double x = vt[tid * D + j];
      if (fabs(x) > best) { best = fabs(x); val = x; }
    }
    flip[tid] = val < 0.0 ? -1.0 : 1.0;
  }
  __syncthreads();
  if (tid < D) lambda[tid] = (float)A[order[tid] * D + order[tid]];
  // R[c][k] = sum_l H[c][l] * U[k][l], U[k][l] = component k of the l-th eigenvector (in sorted order)
  for (int idx = tid; idx < D * D; idx += EIG_THREADS) {
    const int c = idx / D, k = idx % D;
    double acc = 0.0;
    for (int l = 0; l < D; l++) {
      const int src = order[l];
      const double h = ((__popc(c & l) & 1) ? -1.0 : 1.0) * (double)signs[l];
      acc += h * flip[src] * vt[src * D + k];
    }
    R[idx] = (float)(acc * 0.08838834764831845);   // 1 / sqrt(128)
  }
}

size_t attn_bytes(int group, int n) {
  const size_t n_it = (size_t)(n + TQ - 1) / TQ;
  return ((size_t)group * n * 2 + n_it * group * n) * sizeof(float);
}
size_t moments_bytes() { return (size_t)MAX_CHUNKS * 3 * D * D * sizeof(float) + 16; }
constexpr size_t EIGEN_BYTES = (size_t)D * D * sizeof(double);

}  // namespace
}  // namespace okq

using namespace okq;

extern "C" {

size_t okq_calib_workspace_bytes(int32_t group, int32_t n) {
  if (group <= 0 || n <= 0) return 0;
  size_t b = attn_bytes(group, n);
  if (moments_bytes() > b) b = moments_bytes();
  if (EIGEN_BYTES > b) b = EIGEN_BYTES;
  return (b + 255) & ~(size_t)255;
}

okq_status okq_calib_attention_weights(const void* q_fp16, const void* k_fp16, int32_t group, int32_t n,
                                       float sm_scale, int32_t causal, void* workspace, size_t workspace_bytes,
                                       float* w_out, void* stream) {
  if (!q_fp16 || !k_fp16 || !w_out || !workspace || group <= 0 || n <= 0) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(q_fp16) || !aligned16(k_fp16) || !aligned16(workspace) || !aligned16(w_out)) return OKQ_ERR_ALIGNMENT;
  if (workspace_bytes < attn_bytes(group, n)) return OKQ_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  float* rowstat = static_cast<float*>(workspace);
  float* partial = rowstat + (size_t)group * n * 2;
  const dim3 grid((n + TQ - 1) / TQ, group);
  const __half* q = static_cast<const __half*>(q_fp16);
  const __half* k = static_cast<const __half*>(k_fp16);
  k_calib_pass<0><<<grid, 128, 0, s>>>(q, k, group, n, sm_scale, causal, rowstat, partial);
  k_calib_pass<1><<<grid, 128, 0, s>>>(q, k, group, n, sm_scale, causal, rowstat, partial);
  k_calib_wsum<<<(n + 127) / 128, 128, 0, s>>>(partial, group, n, causal, w_out);
  return launch_status();
}

okq_status okq_calib_moments(const void* v_fp16, const float* w, const uint8_t* modality, int32_t n,
                             void* workspace, size_t workspace_bytes, float* C_out, void* stream) {
  if (!v_fp16 || !w || !modality || !C_out || !workspace || n <= 0) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(v_fp16) || !aligned16(workspace) || !aligned16(C_out)) return OKQ_ERR_ALIGNMENT;
  if (workspace_bytes < moments_bytes()) return OKQ_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  float* partial = static_cast<float*>(workspace);
  int* w_exp = reinterpret_cast<int*>(partial + (size_t)MAX_CHUNKS * 3 * D * D);
  const int n_tiles = (n + MT - 1) / MT;
  const int n_chunks = n_tiles < MAX_CHUNKS ? n_tiles : MAX_CHUNKS;
  k_calib_wmax<<<1, 1024, 0, s>>>(w, n, w_exp);
  k_calib_moments<<<dim3(n_chunks, 3), 256, 0, s>>>(static_cast<const __half*>(v_fp16), w, modality, n, n_chunks, w_exp, partial);
  k_calib_csum<<<(3 * D * D + 255) / 256, 256, 0, s>>>(partial, n_chunks, w_exp, C_out);
  return launch_status();
}

okq_status okq_calib_rotation(const float* C, const float* signs, void* workspace, size_t workspace_bytes,
                              float* R_out, float* lambda_out, int32_t* sweeps_out, void* stream) {
  if (!C || !signs || !workspace || !R_out || !lambda_out) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(C) || !aligned16(workspace) || !aligned16(R_out)) return OKQ_ERR_ALIGNMENT;
  if (workspace_bytes < EIGEN_BYTES) return OKQ_ERR_WORKSPACE;
  static thread_local unsigned long long attr_mask = 0;
  int attr_dev = 0;
  if (attr_needed(attr_mask, attr_dev)) {
    cudaError_t e = cudaFuncSetAttribute(k_calib_eigen, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)EIGEN_BYTES);
    if (e != cudaSuccess) { set_last_cuda_error((int)e); return OKQ_ERR_CUDA; }
    attr_done(attr_mask, attr_dev);
  }
  k_calib_eigen<<<1, EIG_THREADS, EIGEN_BYTES, static_cast<cudaStream_t>(stream)>>>(C, signs, static_cast<double*>(workspace), R_out,
                                                                                  lambda_out, sweeps_out);
  return launch_status();
}

}  // extern "C"
