// Quantise-and-append kernels: fp16 keys/values -> window records (Eq. 2, 3, 4, 6), the
// streaming append with its fp16 tail, and conversion to/from the canonical arrays.
//
// Every floating-point step that decides a stored bit is written with the explicitly
// rounded intrinsics (__fmul_rn, __fadd_rn, ...), which the compiler never contracts into
// fused multiply-adds, so the stored codes, norms and (m, s) pairs do not depend on
// compiler flags.  The one place that is *defined* with fused multiply-adds is the value
// rotation: one __fmaf_rn chain per output coordinate, input index ascending.
#include "okq_common.cuh"
#include "okq_device.cuh"

namespace okq {

constexpr int ZS = 144;  // row stride (floats) of the per-window staging buffers: neighbouring rows 16 banks apart

// Position of channel c inside a staged key row: the four 4-float chunks of every 16-channel block are
// rotated by (block >> 1), which makes the three access patterns of the key quantiser (16-byte stores of a
// block per thread, 8-byte accesses with stride 16 channels, 8-byte reads of the code-word order) free of
// shared-memory bank conflicts.
__device__ __forceinline__ int zpos(int c) {
  return (c & ~15) + 4 * ((((c >> 2) & 3) + ((c >> 5) & 3)) & 3) + (c & 3);
}

struct WindowSmem {
  float z[W * ZS];        // rotated keys, or fp32 values
  float a[D];             // keys: decoded minimum m; values: unused
  float b[D];             // keys: 1/s (0 when s == 0)
  float inv[W];           // values: 1/norm per token (0 for a zero vector)
  unsigned char code[W * D];  // values: one code per byte
  unsigned char mod[W];
  int uniform;
};

// Key window: rows(i) = rows + i*stride, i = 0..31.  128 threads.
//
// The 128-point transform is done in two in-register halves around one shared-memory transpose:
// eight threads per token first hold 16 consecutive channels each (stages h = 1, 2, 4, 8, and the
// first four levels of the norm's summation tree), then each holds the 2 x 8 channels that differ in
// the three high index bits (stages h = 16, 32, 64).  The stage order, and with it every rounding,
// is that of the plain butterfly loop.
// two fp32 values in one 64-bit register and the packed arithmetic on them (each half rounds like the scalar op)
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}

__device__ void quantize_key_window(const __half* rows, long long stride, const float* __restrict__ signs,
                                    unsigned char* rec, unsigned char* body, int fmt, WindowSmem& sm) {
  const int tid = threadIdx.x;
  __half* knorm = reinterpret_cast<__half*>(body + B_KNORM);
  const int a = tid & 7;          // which 16-channel block (first half) / which channel pair (second half)
  uint64_t sgp[8];   // the signs of the thread's 16 channels, two per register
#pragma unroll
  for (int q = 0; q < 4; q++) {
    const float4 s4 = *reinterpret_cast<const float4*>(signs + 16 * a + 4 * q);
    sgp[2 * q] = pack2(s4.x, s4.y); sgp[2 * q + 1] = pack2(s4.z, s4.w);
  }
#pragma unroll 1
  for (int round = 0; round < 2; round++) {
    const int i = (tid >> 3) + 16 * round;   // token; its eight threads are neighbours in one warp
    float* zrow = &sm.z[i * ZS];
    float y[16];
    {
      const uint4* src = reinterpret_cast<const uint4*>(rows + (long long)i * stride + 16 * a);
      const uint4 r0 = src[0], r1 = src[1];
      const __half2* h0 = reinterpret_cast<const __half2*>(&r0);
      const __half2* h1 = reinterpret_cast<const __half2*>(&r1);
#pragma unroll
      for (int q = 0; q < 4; q++) {
        const float2 f0 = __half22float2(h0[q]), f1 = __half22float2(h1[q]);
        y[2 * q] = f0.x; y[2 * q + 1] = f0.y; y[8 + 2 * q] = f1.x; y[8 + 2 * q + 1] = f1.y;
      }
    }
    // Two channels per instruction (add / sub / mul .f32x2: each half is the same IEEE operation as the
    // scalar one, so the results do not change): P[i] = (y[2i], y[2i+1]).
    uint64_t P[8];
#pragma unroll
    for (int q = 0; q < 8; q++) P[q] = pack2(y[2 * q], y[2 * q + 1]);
    // norm: adjacent-pair tree (4 levels here, 3 across the eight threads)
    float t[16];
#pragma unroll
    for (int q = 0; q < 8; q++) unpack2(mul2(P[q], P[q]), t[2 * q], t[2 * q + 1]);
#pragma unroll
    for (int n = 8; n >= 1; n >>= 1)
#pragma unroll
      for (int c = 0; c < n; c++) t[c] = __fadd_rn(t[2 * c], t[2 * c + 1]);
    float ssum = t[0];
    ssum = __fadd_rn(ssum, __shfl_xor_sync(0xffffffffu, ssum, 1));
    ssum = __fadd_rn(ssum, __shfl_xor_sync(0xffffffffu, ssum, 2));
    ssum = __fadd_rn(ssum, __shfl_xor_sync(0xffffffffu, ssum, 4));
    float nrm = __fsqrt_rn(ssum);
    nrm = nrm > 65504.0f ? 65504.0f : nrm;
    const __half nh = __float2half_rn(nrm);
    const float nf = __half2float(nh);
    if (a == 0) knorm[norm_pos(i)] = nh;
    const float cinv = nf != 0.0f ? __fdiv_rn(RSQRT_D, nf) : 0.0f;
    // D x, then stages h = 1, 2, 4, 8 inside the 16-channel block: h = 1 pairs the two halves of one P[i]
    // (scalar), h = 2, 4, 8 pair P[i] with P[i + h/2]
#pragma unroll
    for (int q = 0; q < 8; q++) {
      float lo, hi;
      unpack2(mul2(sgp[q], P[q]), lo, hi);
      P[q] = pack2(__fadd_rn(lo, hi), __fsub_rn(lo, hi));
    }
#pragma unroll
    for (int hh = 1; hh < 8; hh <<= 1)
#pragma unroll
      for (int j = 0; j < 8; j++)
        if ((j & hh) == 0) {
          const uint64_t p = P[j], q2 = P[j + hh];
          P[j] = add2(p, q2);
          P[j + hh] = sub2(p, q2);
        }
#pragma unroll
    for (int q = 0; q < 4; q++)
      *reinterpret_cast<ulonglong2*>(&zrow[zpos(16 * a + 4 * q)]) = make_ulonglong2(P[2 * q], P[2 * q + 1]);
    __syncwarp();
    // second half: channels 16*u + 2*a + e, u = 0..7: stages h = 16, 32, 64 act on u; Q[u] = both e
    uint64_t Q[8];
#pragma unroll
    for (int u = 0; u < 8; u++) Q[u] = *reinterpret_cast<const uint64_t*>(&zrow[zpos(16 * u + 2 * a)]);
#pragma unroll
    for (int hh = 1; hh < 8; hh <<= 1)
#pragma unroll
      for (int j = 0; j < 8; j++)
        if ((j & hh) == 0) {
          const uint64_t p = Q[j], q2 = Q[j + hh];
          Q[j] = add2(p, q2);
          Q[j + hh] = sub2(p, q2);
        }
    __syncwarp();   // every thread of the token has read the first-half values before they are overwritten
    const uint64_t cinv2 = pack2(cinv, cinv);
#pragma unroll
    for (int u = 0; u < 8; u++)
      *reinterpret_cast<uint64_t*>(&zrow[zpos(16 * u + 2 * a)]) = nf != 0.0f ? mul2(Q[u], cinv2) : 0ull;
  }
  __syncthreads();
  {  // per channel: window minimum and step (Eq. 4)
    int c = tid;
    const int cp = zpos(c);
    float mn = sm.z[cp], mx = mn;
#pragma unroll 8
    for (int i = 1; i < W; i++) {
      float v = sm.z[i * ZS + cp];
      if (v < mn) mn = v;
      if (v > mx) mx = v;
    }
    if (fmt == FMT_FP16) {
      __half mh = __float2half_rn(mn);
      float mf = __half2float(mh);
      float range = __fsub_rn(mx, mf);
      if (range < 0.0f) range = 0.0f;
      __half sh = __float2half_rn(__fdiv_rn(range, 3.0f));
      float sf = __half2float(sh);
      sm.a[c] = mf;
      sm.b[c] = sf > 0.0f ? __fdiv_rn(1.0f, sf) : 0.0f;
      int p = meta_pos(c);
      reinterpret_cast<__half*>(rec + OFF_KM)[p] = __float2half_rn(mf * (float)(1 << (2 * meta_shift(c))));   // exact
      reinterpret_cast<__half*>(rec + OFF_KS)[p] = sh;
    } else {
      // MXFP4: a warp is one block of 32 consecutive channels; nearest-even conversion of m, then of s
      const int lane = tid & 31, blk = tid >> 5;
      float amax = fabsf(mn);
#pragma unroll
      for (int d = 16; d; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
      const int km = mx_scale_exp(amax);
      const unsigned mnib = mx_encode(mn, km);
      const float mf = mx_decode(mnib, km);
      float range = __fsub_rn(mx, mf);
      if (range < 0.0f) range = 0.0f;
      const float sraw = __fdiv_rn(range, 3.0f);
      float smax = sraw;
#pragma unroll
      for (int d = 16; d; d >>= 1) smax = fmaxf(smax, __shfl_xor_sync(0xffffffffu, smax, d));
      const int ks = mx_scale_exp(smax);
      const unsigned snib = mx_encode(sraw, ks);
      const float sf = mx_decode(snib, ks);
      sm.a[c] = mf;
      sm.b[c] = sf > 0.0f ? __fdiv_rn(1.0f, sf) : 0.0f;
      const int p = meta_pos(c);
      sm.code[p] = (unsigned char)mnib;          // nibbles in record order, packed two per byte below
      sm.code[D + p] = (unsigned char)snib;
      if (lane == 0) { rec[128 + blk] = (unsigned char)(km + 127); rec[132 + blk] = (unsigned char)(ks + 127); }
    }
  }
  __syncthreads();
  if (fmt == FMT_MXFP4) {
    // 128 bytes: m nibbles [0, 64), s nibbles [64, 128)
    rec[tid] = (unsigned char)(sm.code[2 * tid] | (sm.code[2 * tid + 1] << 4));
  }
  // codes: a thread keeps the (m, 1/s) of the 16 channels of "its" word position (t, ww) in registers
  // and packs that word for two tokens
  {
    uint32_t* words = reinterpret_cast<uint32_t*>(body + B_KCODE);
    const int t = tid & 3, ww = (tid >> 2) & 1, tg = tid >> 3;   // tokens tg and tg + 16
    uint64_t mch[8], rch[8];   // (m, 1/s) of the channel pairs 2q, 2q+1 of the word
#pragma unroll
    for (int q = 0; q < 8; q++) {
      const int c0 = 16 * ((ww * 8 + q) >> 1) + 8 * (q & 1) + 2 * t;
      mch[q] = *reinterpret_cast<const uint64_t*>(&sm.a[c0]);
      rch[q] = *reinterpret_cast<const uint64_t*>(&sm.b[c0]);
    }
    // code = clamp(rint((z - m) / s), 0, 3).  Clamping first gives the same integer (rounding is monotone and
    // keeps 0 and 3), and adding 1.5 * 2^23 to a value in [0, 3] rounds it to nearest-even into the low
    // mantissa bits; the sixteen 2-bit fields are then summed with integer shift-adds and the sixteen
    // copies of the constant's bit pattern are taken off at the end (all modulo 2^32).
    constexpr float MAGIC = 12582912.0f;                 // 1.5 * 2^23, bit pattern 0x4B400000
    constexpr uint32_t MAGIC_SUM = 0x4B400000u * 0x55555555u;   // sum over the sixteen field positions 4^j
    const uint64_t magic2 = pack2(MAGIC, MAGIC);
#pragma unroll
    for (int k = 0; k < 2; k++) {
      const int i = tg + 16 * k;
      uint32_t word = 0;
#pragma unroll
      for (int q = 0; q < 8; q++) {
        const int c0 = 16 * ((ww * 8 + q) >> 1) + 8 * (q & 1) + 2 * t;
        const uint64_t z2 = *reinterpret_cast<const uint64_t*>(&sm.z[i * ZS + zpos(c0)]);
        float u0, u1;
        unpack2(mul2(sub2(z2, mch[q]), rch[q]), u0, u1);
        float r0, r1;
        unpack2(add2(pack2(fminf(fmaxf(u0, 0.0f), 3.0f), fminf(fmaxf(u1, 0.0f), 3.0f)), magic2), r0, r1);
        word += __float_as_uint(r0) << (8 * (q >> 2) + 2 * (q & 3));
        word += __float_as_uint(r1) << (16 + 8 * (q >> 2) + 2 * (q & 3));
      }
      word -= MAGIC_SUM;
      // word index of (token i, t, ww): [i >> 4][lane 4*(i & 7) + t][(i >> 3) & 1][ww]
      words[kword_index((i >> 4) * 128 + (4 * (i & 7) + t) * 4 + ((i >> 3) & 1) * 2 + ww)] = word;
    }
  }
  __syncthreads();
}

// Value window.  mod[] must already be in sm.mod and sm.uniform set.  Rset = R + rsel*3*D*D.
__device__ void quantize_value_window(const __half* rows, long long stride, const float* __restrict__ Rset,
                                      unsigned char* body, WindowSmem& sm) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  __half* vnorm = reinterpret_cast<__half*>(body + B_VNORM);
  for (int k = 0; k < 8; k++) {
    int i = warp * 8 + k;
    float4 x = load_row4(rows + (long long)i * stride, lane);
    float n = warp_norm(x);
    __half nh = __float2half_rn(n);
    float nf = __half2float(nh);
    *reinterpret_cast<float4*>(&sm.z[i * ZS + 4 * lane]) = x;
    if (lane == 0) {
      vnorm[norm_pos(i)] = nh;
      sm.inv[i] = nf != 0.0f ? __fdiv_rn(1.0f, nf) : 0.0f;
    }
  }
  __syncthreads();
  {
    const int c = tid;
    if (sm.uniform) {
      const float4* Rrow = reinterpret_cast<const float4*>(Rset + ((size_t)sm.mod[0] * D + c) * D);
      float acc[W];
#pragma unroll
      for (int i = 0; i < W; i++) acc[i] = 0.0f;
      for (int k4 = 0; k4 < D / 4; k4++) {
        float4 r4 = __ldg(Rrow + k4);
#pragma unroll
        for (int i = 0; i < W; i++) {
          float4 x4 = *reinterpret_cast<const float4*>(&sm.z[i * ZS + 4 * k4]);
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
        float z = __fmul_rn(acc[i], sm.inv[i]);
        sm.code[i * D + c] = (unsigned char)((z > -CB_THRESH) + (z > 0.0f) + (z > CB_THRESH));
      }
    } else {
      for (int i = 0; i < W; i++) {
        const float4* Rrow = reinterpret_cast<const float4*>(Rset + ((size_t)sm.mod[i] * D + c) * D);
        float a = 0.0f;
        for (int k4 = 0; k4 < D / 4; k4++) {
          float4 r4 = __ldg(Rrow + k4);
          float4 x4 = *reinterpret_cast<const float4*>(&sm.z[i * ZS + 4 * k4]);
          a = __fmaf_rn(r4.x, x4.x, a);
          a = __fmaf_rn(r4.y, x4.y, a);
          a = __fmaf_rn(r4.z, x4.z, a);
          a = __fmaf_rn(r4.w, x4.w, a);
        }
        float z = __fmul_rn(a, sm.inv[i]);
        sm.code[i * D + c] = (unsigned char)((z > -CB_THRESH) + (z > 0.0f) + (z > CB_THRESH));
      }
    }
  }
  __syncthreads();
  uint32_t* words = reinterpret_cast<uint32_t*>(body + B_VCODE);
  for (int wi = tid; wi < 256; wi += 128) {
    int mu = (wi >> 7) * 4 + (wi & 3);
    int l = (wi & 127) >> 2;
    int g = l >> 2, t = l & 3;
    uint32_t word = 0;
#pragma unroll
    for (int q = 0; q < 8; q++) {
      int sh = q >> 2, j = q & 3;
#pragma unroll
      for (int e = 0; e < 2; e++) {
        int i = 16 * (j >> 1) + 8 * (j & 1) + 2 * t + e;
        int c = 16 * mu + 8 * sh + g;
        word |= (uint32_t)sm.code[i * D + c] << (16 * e + 8 * sh + 2 * j);
      }
    }
    words[vword_index(wi)] = word;
  }
  __syncthreads();
}

__device__ __forceinline__ void stage_modality(const unsigned char* mod32, WindowSmem& sm) {
  if (threadIdx.x < 32) {
    unsigned char m = mod32[threadIdx.x];
    m = m > 2 ? 0 : m;  // anything that is not audio / video counts as text
    sm.mod[threadIdx.x] = m;
    unsigned char m0 = __shfl_sync(0xffffffffu, m, 0);
    int uni = __all_sync(0xffffffffu, m == m0);
    if (threadIdx.x == 0) sm.uniform = uni;
  }
  __syncthreads();
}

// ---------------------------------------------------------------- bulk kernels

__global__ void __launch_bounds__(128) k_quantize_keys(CacheView cv, int layer, const __half* __restrict__ k,
                                                      long long sb, long long sh, long long st,
                                                      const float* __restrict__ signs) {
  __shared__ WindowSmem sm;
  int win = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const __half* rows = k + b * sb + h * sh + (long long)win * W * st;
  quantize_key_window(rows, st, signs, cv.meta(layer, b, h, win), cv.body(layer, b, h, win), cv.fmt, sm);
}

__global__ void __launch_bounds__(128) k_quantize_values(CacheView cv, int layer, const __half* __restrict__ v,
                                                        long long sb, long long sh, long long st,
                                                        const unsigned char* __restrict__ modality, int n_tokens,
                                                        const float* __restrict__ R, int n_R) {
  __shared__ WindowSmem sm;
  int win = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  stage_modality(modality + (size_t)b * n_tokens + (size_t)win * W, sm);
  const __half* rows = v + b * sb + h * sh + (long long)win * W * st;
  const float* Rset = R + (size_t)(n_R == 1 ? 0 : h) * 3 * D * D;
  quantize_value_window(rows, st, Rset, cv.body(layer, b, h, win), sm);
}

// raw tokens behind the packed ones + seq_len (+ modality for the value call); grid (n_kv_heads, batch, slices),
// 128 threads.  Token t goes to slot t mod (slots of the schedule).
__global__ void k_bulk_tail(CacheView cv, int layer, const __half* __restrict__ src, long long sb, long long sh,
                            long long st, int n_tokens, int is_value, const unsigned char* __restrict__ modality) {
  const int h = blockIdx.x, b = blockIdx.y;
  const int n_packed = is_value ? cv.v_packed(n_tokens) : cv.k_packed(n_tokens);
  const int n_tail = n_tokens - n_packed;
  __half* dst = is_value ? cv.v_tail + cv.v_tail_off(layer, b, h) : cv.k_tail + cv.k_tail_off(layer, b, h);
  const int per = (n_tail + gridDim.z - 1) / gridDim.z;      // tokens per slice
  const int i0 = blockIdx.z * per, i1 = min(n_tail, i0 + per);
  for (int idx = i0 * (D / 8) + threadIdx.x; idx < i1 * (D / 8); idx += blockDim.x) {
    const int t = n_packed + idx / (D / 8), c8 = idx % (D / 8);
    const int slot = is_value ? cv.v_slot(t) : cv.k_slot(t);
    reinterpret_cast<uint4*>(dst + slot * D)[c8] =
        *reinterpret_cast<const uint4*>(src + b * sb + h * sh + (long long)t * st + c8 * 8);
  }
  if (blockIdx.z == 0 && h == 0 && threadIdx.x == 0) cv.seq_len[layer * cv.batch + b] = n_tokens;
  if (modality) {   // the sequence's modality bytes, spread over the (head, slice) blocks of the sequence
    const int stride = gridDim.x * gridDim.z * blockDim.x;
    for (int i = (h * gridDim.z + blockIdx.z) * blockDim.x + threadIdx.x; i < n_tokens; i += stride) {
      const unsigned char m = modality[(size_t)b * n_tokens + i];
      cv.modality[(size_t)b * cv.capacity + i] = m > 2 ? 0 : m;
    }
  }
}

// ---------------------------------------------------------------- append

constexpr int APPEND_ARRIVAL = 1 << 24;   // one arrived block in the transient count kept in seq_len's top byte

// grid (n_kv_heads, batch, layer_count), 128 threads
__global__ void __launch_bounds__(128) k_append(CacheView cv, int layer0, const __half* __restrict__ k_new,
                                               const __half* __restrict__ v_new,
                                               const unsigned char* __restrict__ mod_new,
                                               const float* __restrict__ signs, const float* __restrict__ R,
                                               int n_R) {
  __shared__ WindowSmem sm;
  __shared__ int s_pos;
  int h = blockIdx.x, b = blockIdx.y, li = blockIdx.z, layer = layer0 + li;
  // The n_kv_heads blocks of a (layer, sequence) all need the position before any of them may advance it.
  // Each block counts itself in the top byte of seq_len while reading it; the block that finds the others
  // already counted stores the new length (which also clears the count): by then every block has its copy.
  if (threadIdx.x == 0) {
    int* len = cv.seq_len + layer * cv.batch + b;
    const int old = atomicAdd(len, APPEND_ARRIVAL);
    const int p = old & (APPEND_ARRIVAL - 1);
    if (old / APPEND_ARRIVAL == cv.n_kv_heads - 1) *len = p < cv.capacity ? p + 1 : p;
    s_pos = p;
  }
  __syncthreads();
  const int pos = s_pos;
  if (pos >= cv.capacity) {
    if (threadIdx.x == 0) atomicCAS(cv.status, 0, (int)OKQ_ERR_CAPACITY);
    return;
  }
  size_t src = (((size_t)li * cv.batch + b) * cv.n_kv_heads + h) * D;
  __half* kt = cv.k_tail + cv.k_tail_off(layer, b, h);
  __half* vt = cv.v_tail + cv.v_tail_off(layer, b, h);
  unsigned char mnew = mod_new[b];
  mnew = mnew > 2 ? 0 : mnew;
  const int kslot = cv.k_slot(pos), vslot = cv.v_slot(pos);
  if (threadIdx.x < 16) reinterpret_cast<uint4*>(kt + kslot * D)[threadIdx.x] = reinterpret_cast<const uint4*>(k_new + src)[threadIdx.x];
  else if (threadIdx.x < 32) reinterpret_cast<uint4*>(vt + vslot * D)[threadIdx.x - 16] = reinterpret_cast<const uint4*>(v_new + src)[threadIdx.x - 16];
  if (h == 0 && threadIdx.x == 32) cv.modality[(size_t)b * cv.capacity + pos] = mnew;
  // windows that the schedule packs now that the sequence holds pos + 1 tokens
  const int kw0 = cv.k_packed(pos) / W, kw1 = cv.k_packed(pos + 1) / W;
  const int vw0 = cv.v_packed(pos) / W, vw1 = cv.v_packed(pos + 1) / W;
  if (kw0 == kw1 && vw0 == vw1) return;
  __syncthreads();  // the new token is now visible to the whole block
  for (int win = kw0; win < kw1; win++)   // the window's 32 raw keys sit in consecutive slots
    quantize_key_window(kt + cv.k_slot(win * W) * D, D, signs + (size_t)li * D, cv.meta(layer, b, h, win),
                        cv.body(layer, b, h, win), cv.fmt, sm);
  const float* Rset = R + ((size_t)li * n_R + (n_R == 1 ? 0 : h)) * 3 * D * D;
  for (int win = vw0; win < vw1; win++) {
    __syncthreads();
    if (threadIdx.x < 32) {
      const int t = win * W + threadIdx.x;   // the newest token's modality may not have reached global memory yet
      unsigned char m = t == pos ? mnew : cv.modality[(size_t)b * cv.capacity + t];
      sm.mod[threadIdx.x] = m;
      unsigned char m0 = __shfl_sync(0xffffffffu, m, 0);
      int uni = __all_sync(0xffffffffu, m == m0);
      if (threadIdx.x == 0) sm.uniform = uni;
    }
    __syncthreads();
    quantize_value_window(vt + cv.v_slot(win * W) * D, D, Rset, cv.body(layer, b, h, win), sm);
  }
}

// ---------------------------------------------------------------- canonical <-> physical

// grid (capacity/32, n_kv_heads, batch), 128 threads
__global__ void k_export(CacheView cv, int layer, unsigned char* k_codes, __half* k_norm, __half* k_meta,
                         unsigned char* v_codes, __half* v_norm, unsigned char* k_mx) {
  int win = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const unsigned char* rec = cv.meta(layer, b, h, win);
  const unsigned char* body = cv.body(layer, b, h, win);
  size_t unit = (size_t)b * cv.n_kv_heads + h;
  size_t tok0 = unit * cv.capacity + (size_t)win * W;
  const uint32_t* kw = reinterpret_cast<const uint32_t*>(body + B_KCODE);
  const uint32_t* vw = reinterpret_cast<const uint32_t*>(body + B_VCODE);
  for (int idx = threadIdx.x; idx < W * 32; idx += blockDim.x) {
    int i = idx >> 5, byte = idx & 31;
    unsigned kb = 0, vb = 0;
    for (int k = 0; k < 4; k++) {
      int c = byte * 4 + k, word, bit;
      kcode_pos(i, c, word, bit);
      kb |= ((kw[word] >> bit) & 3u) << (2 * k);
      vcode_pos(i, c, word, bit);
      vb |= ((vw[word] >> bit) & 3u) << (2 * k);
    }
    k_codes[(tok0 + i) * 32 + byte] = (unsigned char)kb;
    v_codes[(tok0 + i) * 32 + byte] = (unsigned char)vb;
  }
  if (threadIdx.x < W) {
    k_norm[tok0 + threadIdx.x] = reinterpret_cast<const __half*>(body + B_KNORM)[norm_pos(threadIdx.x)];
    v_norm[tok0 + threadIdx.x] = reinterpret_cast<const __half*>(body + B_VNORM)[norm_pos(threadIdx.x)];
  }
  {
    int c = threadIdx.x, p = meta_pos(c);
    size_t o = ((unit * cv.n_windows() + win) * D + c) * 2;
    if (cv.fmt == FMT_FP16) {
      k_meta[o] = __float2half_rn(__half2float(reinterpret_cast<const __half*>(rec + OFF_KM)[p]) /
                                  (float)(1 << (2 * meta_shift(c))));   // exact
      k_meta[o + 1] = reinterpret_cast<const __half*>(rec + OFF_KS)[p];
    } else {   // decode the MXFP4 pair; every decoded value is an fp16 number
      const unsigned mnib = (rec[p >> 1] >> (4 * (p & 1))) & 15u, snib = (rec[64 + (p >> 1)] >> (4 * (p & 1))) & 15u;
      k_meta[o] = __float2half_rn(mx_decode(mnib, (int)rec[128 + (c >> 5)] - 127));
      k_meta[o + 1] = __float2half_rn(mx_decode(snib, (int)rec[132 + (c >> 5)] - 127));
      if (k_mx) {   // stored bytes in natural channel order: nibble of channel c in byte c/2
        unsigned char* dst = k_mx + (unit * cv.n_windows() + win) * MX_META_BYTES;
        __shared__ unsigned char nb[2 * D];
        nb[c] = (unsigned char)mnib; nb[D + c] = (unsigned char)snib;
        __syncthreads();
        dst[c] = (unsigned char)(nb[2 * c] | (nb[2 * c + 1] << 4));
        if (c < 8) dst[128 + c] = rec[128 + c];
      }
    }
  }
}

__global__ void k_import(CacheView cv, int layer, const unsigned char* k_codes, const __half* k_norm,
                         const __half* k_meta, const unsigned char* v_codes, const __half* v_norm) {
  int win = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  unsigned char* rec = cv.meta(layer, b, h, win);   // fp16 metadata only
  size_t unit = (size_t)b * cv.n_kv_heads + h;
  size_t tok0 = unit * cv.capacity + (size_t)win * W;
  __shared__ uint32_t kw[256], vw[256];
  for (int i = threadIdx.x; i < 256; i += blockDim.x) { kw[i] = 0; vw[i] = 0; }
  __syncthreads();
  for (int idx = threadIdx.x; idx < W * 32; idx += blockDim.x) {
    int i = idx >> 5, byte = idx & 31;
    unsigned kb = k_codes[(tok0 + i) * 32 + byte], vb = v_codes[(tok0 + i) * 32 + byte];
    for (int k = 0; k < 4; k++) {
      int c = byte * 4 + k, word, bit;
      kcode_pos(i, c, word, bit);
      atomicOr(&kw[word], ((kb >> (2 * k)) & 3u) << bit);
      vcode_pos(i, c, word, bit);
      atomicOr(&vw[word], ((vb >> (2 * k)) & 3u) << bit);
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 256; i += blockDim.x) {
    reinterpret_cast<uint32_t*>(rec + OFF_KCODE)[i] = kw[i];
    reinterpret_cast<uint32_t*>(rec + OFF_VCODE)[i] = vw[i];
  }
  if (threadIdx.x < W) {
    reinterpret_cast<__half*>(rec + OFF_KNORM)[norm_pos(threadIdx.x)] = k_norm[tok0 + threadIdx.x];
    reinterpret_cast<__half*>(rec + OFF_VNORM)[norm_pos(threadIdx.x)] = v_norm[tok0 + threadIdx.x];
  }
  {
    int c = threadIdx.x, p = meta_pos(c);
    size_t o = ((unit * cv.n_windows() + win) * D + c) * 2;
    reinterpret_cast<__half*>(rec + OFF_KM)[p] = __float2half_rn(__half2float(k_meta[o]) * (float)(1 << (2 * meta_shift(c))));
    reinterpret_cast<__half*>(rec + OFF_KS)[p] = k_meta[o + 1];
  }
}

okq_status launch_quantize_values_tc(const CacheView& cv, int layer, const __half* v, const int64_t strides[3],
                                     const unsigned char* modality, int n_tokens, int n_win, const float* R, int n_R,
                                     int n_sm, cudaStream_t s, long long wait_limit = 0, int skip_tile = -1);

constexpr int TAIL_SLICES = 16;   // blocks per (sequence, head) that share the copy of the modality bytes

static okq_status check_bulk(const okq_cache* c, int32_t layer, const void* x, const int64_t strides[3],
                             int32_t n_tokens) {
  okq_status st = check_cache(c, true);
  if (st != OKQ_OK) return st;
  if (!strides || layer < 0 || layer >= c->n_layers || n_tokens < 0) return OKQ_ERR_INVALID_ARG;
  if (!x && n_tokens > 0) return OKQ_ERR_INVALID_ARG;  // an empty prefill may pass a null tensor
  if (n_tokens > c->capacity) return OKQ_ERR_CAPACITY;
  if (!aligned16(x) || strides[0] % 8 || strides[1] % 8 || strides[2] % 8) return OKQ_ERR_ALIGNMENT;
  return OKQ_OK;
}

}  // namespace okq

using namespace okq;

extern "C" {

okq_status okq_quantize_keys(const okq_cache* cache, int32_t layer, const void* k_fp16, const int64_t strides[3],
                             int32_t n_tokens, const float* signs, void* stream) {
  okq_status st = check_bulk(cache, layer, k_fp16, strides, n_tokens);
  if (st != OKQ_OK) return st;
  if (!signs) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(signs)) return OKQ_ERR_ALIGNMENT;
  CacheView cv = make_view(cache);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __half* k = static_cast<const __half*>(k_fp16);
  int n_win = cv.k_packed(n_tokens) / W;
  if (n_win > 0) {
    dim3 grid(n_win, cv.n_kv_heads, cv.batch);
    k_quantize_keys<<<grid, 128, 0, s>>>(cv, layer, k, strides[0], strides[1], strides[2], signs);
  }
  k_bulk_tail<<<dim3(cv.n_kv_heads, cv.batch, 1), 128, 0, s>>>(cv, layer, k, strides[0], strides[1], strides[2],
                                                              n_tokens, 0, nullptr);
  return launch_status();
}

okq_status okq_quantize_values(const okq_cache* cache, int32_t layer, const void* v_fp16, const int64_t strides[3],
                               int32_t n_tokens, const uint8_t* modality, const float* R, int32_t n_R,
                               void* stream) {
  okq_status st = check_bulk(cache, layer, v_fp16, strides, n_tokens);
  if (st != OKQ_OK) return st;
  if ((!modality && n_tokens > 0) || !R) return OKQ_ERR_INVALID_ARG;
  if (n_R != 1 && n_R != cache->n_kv_heads) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(R)) return OKQ_ERR_ALIGNMENT;
  CacheView cv = make_view(cache);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __half* v = static_cast<const __half*>(v_fp16);
  int n_win = cv.v_packed(n_tokens) / W;
  if (n_win > 0) {
    dim3 grid(n_win, cv.n_kv_heads, cv.batch);
    k_quantize_values<<<grid, 128, 0, s>>>(cv, layer, v, strides[0], strides[1], strides[2], modality, n_tokens, R,
                                           n_R);
  }
  k_bulk_tail<<<dim3(cv.n_kv_heads, cv.batch, TAIL_SLICES), 128, 0, s>>>(cv, layer, v, strides[0], strides[1], strides[2],
                                                                        n_tokens, 1, n_tokens > 0 ? modality : nullptr);
  return launch_status();
}

okq_status okq_quantize_values_bulk(const okq_cache* cache, int32_t layer, const void* v_fp16,
                                    const int64_t strides[3], int32_t n_tokens, const uint8_t* modality,
                                    const float* R, int32_t n_R, void* stream) {
  okq_status st = check_bulk(cache, layer, v_fp16, strides, n_tokens);
  if (st != OKQ_OK) return st;
  if ((!modality && n_tokens > 0) || !R) return OKQ_ERR_INVALID_ARG;
  if (n_R != 1 && n_R != cache->n_kv_heads) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(R)) return OKQ_ERR_ALIGNMENT;
  CacheView cv = make_view(cache);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __half* v = static_cast<const __half*>(v_fp16);
  st = launch_quantize_values_tc(cv, layer, v, strides, modality, n_tokens, cv.v_packed(n_tokens) / W, R, n_R, sm_count(), s);
  if (st != OKQ_OK) return st;
  k_bulk_tail<<<dim3(cv.n_kv_heads, cv.batch, TAIL_SLICES), 128, 0, s>>>(cv, layer, v, strides[0], strides[1], strides[2],
                                                                        n_tokens, 1, n_tokens > 0 ? modality : nullptr);
  return launch_status();
}

okq_status okq_debug_bulk_timeout(const okq_cache* cache, int32_t layer, const void* v_fp16, const int64_t strides[3],
                                  int32_t n_tokens, const uint8_t* modality, const float* R, int32_t n_R,
                                  int64_t limit_clocks, void* stream) {
  okq_status st = check_bulk(cache, layer, v_fp16, strides, n_tokens);
  if (st != OKQ_OK) return st;
  if (!modality || !R || (n_R != 1 && n_R != cache->n_kv_heads) || limit_clocks <= 0) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(R)) return OKQ_ERR_ALIGNMENT;
  CacheView cv = make_view(cache);
  st = launch_quantize_values_tc(cv, layer, static_cast<const __half*>(v_fp16), strides, modality, n_tokens,
                                 cv.v_packed(n_tokens) / W, R, n_R, sm_count(), static_cast<cudaStream_t>(stream),
                                 (long long)limit_clocks, 0);
  return st != OKQ_OK ? st : launch_status();
}

okq_status okq_append(const okq_cache* cache, int32_t layer, int32_t layer_count, const void* k_new,
                      const void* v_new, const uint8_t* modality_new, const float* signs, const float* R,
                      int32_t n_R, void* stream) {
  okq_status st = check_cache(cache, true);
  if (st != OKQ_OK) return st;
  if (!k_new || !v_new || !modality_new || !signs || !R) return OKQ_ERR_INVALID_ARG;
  if (layer < 0 || layer_count <= 0 || layer + layer_count > cache->n_layers) return OKQ_ERR_INVALID_ARG;
  if (n_R != 1 && n_R != cache->n_kv_heads) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(signs) || !aligned16(R)) return OKQ_ERR_ALIGNMENT;
  CacheView cv = make_view(cache);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // the kernel counts a sequence's blocks in the top byte of its seq_len entry while it runs
  if (cache->capacity >= APPEND_ARRIVAL || cache->n_kv_heads > 127) return OKQ_ERR_UNSUPPORTED;
  k_append<<<dim3(cv.n_kv_heads, cv.batch, layer_count), 128, 0, s>>>(
      cv, layer, static_cast<const __half*>(k_new), static_cast<const __half*>(v_new), modality_new, signs, R, n_R);
  return launch_status();
}

okq_status okq_cache_export(const okq_cache* cache, int32_t layer, uint8_t* k_codes, void* k_norm, void* k_meta,
                            uint8_t* v_codes, void* v_norm, void* stream) {
  okq_status st = check_cache(cache, true);
  if (st != OKQ_OK) return st;
  if (layer < 0 || layer >= cache->n_layers || !k_codes || !k_norm || !k_meta || !v_codes || !v_norm)
    return OKQ_ERR_INVALID_ARG;
  CacheView cv = make_view(cache);
  k_export<<<dim3(cv.capacity / W, cv.n_kv_heads, cv.batch), 128, 0, static_cast<cudaStream_t>(stream)>>>(
      cv, layer, k_codes, static_cast<__half*>(k_norm), static_cast<__half*>(k_meta), v_codes,
      static_cast<__half*>(v_norm), nullptr);
  return launch_status();
}

okq_status okq_cache_export_mx(const okq_cache* cache, int32_t layer, uint8_t* k_codes, void* k_norm, void* k_meta,
                               uint8_t* k_mx, uint8_t* v_codes, void* v_norm, void* stream) {
  okq_status st = check_cache(cache, true);
  if (st != OKQ_OK) return st;
  if (cache->meta_format != OKQ_META_MXFP4) return OKQ_ERR_UNSUPPORTED;
  if (layer < 0 || layer >= cache->n_layers || !k_codes || !k_norm || !k_meta || !k_mx || !v_codes || !v_norm)
    return OKQ_ERR_INVALID_ARG;
  CacheView cv = make_view(cache);
  k_export<<<dim3(cv.capacity / W, cv.n_kv_heads, cv.batch), 128, 0, static_cast<cudaStream_t>(stream)>>>(
      cv, layer, k_codes, static_cast<__half*>(k_norm), static_cast<__half*>(k_meta), v_codes,
      static_cast<__half*>(v_norm), k_mx);
  return launch_status();
}

okq_status okq_cache_import(const okq_cache* cache, int32_t layer, const uint8_t* k_codes, const void* k_norm,
                            const void* k_meta, const uint8_t* v_codes, const void* v_norm, void* stream) {
  okq_status st = check_cache(cache, true);
  if (st != OKQ_OK) return st;
  if (cache->meta_format != OKQ_META_FP16) return OKQ_ERR_UNSUPPORTED;   // fp16 (m, s) need not lie on the MX grid
  if (layer < 0 || layer >= cache->n_layers || !k_codes || !k_norm || !k_meta || !v_codes || !v_norm)
    return OKQ_ERR_INVALID_ARG;
  CacheView cv = make_view(cache);
  k_import<<<dim3(cv.capacity / W, cv.n_kv_heads, cv.batch), 128, 0, static_cast<cudaStream_t>(stream)>>>(
      cv, layer, k_codes, static_cast<const __half*>(k_norm), static_cast<const __half*>(k_meta), v_codes,
      static_cast<const __half*>(v_norm));
  return launch_status();
}

}  // extern "C"
