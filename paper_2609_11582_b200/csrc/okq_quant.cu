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

constexpr int ZS = 132;  // row stride (floats) of the per-window staging buffers

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
__device__ void quantize_key_window(const __half* rows, long long stride, const float* __restrict__ signs,
                                    unsigned char* rec, WindowSmem& sm) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const float4 sg = *reinterpret_cast<const float4*>(signs + 4 * lane);
  __half* knorm = reinterpret_cast<__half*>(rec + OFF_KNORM);
  for (int k = 0; k < 8; k++) {
    int i = warp * 8 + k;
    float4 x = load_row4(rows + (long long)i * stride, lane);
    float n = warp_norm(x);
    __half nh = __float2half_rn(n);
    float nf = __half2float(nh);
    float4 y = make_float4(__fmul_rn(sg.x, x.x), __fmul_rn(sg.y, x.y), __fmul_rn(sg.z, x.z), __fmul_rn(sg.w, x.w));
    y = warp_fwht(y, lane);
    float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    if (nf != 0.0f) {
      float cinv = __fdiv_rn(RSQRT_D, nf);
      z = make_float4(__fmul_rn(y.x, cinv), __fmul_rn(y.y, cinv), __fmul_rn(y.z, cinv), __fmul_rn(y.w, cinv));
    }
    *reinterpret_cast<float4*>(&sm.z[i * ZS + 4 * lane]) = z;
    if (lane == 0) knorm[norm_pos(i)] = nh;
  }
  __syncthreads();
  {  // per channel: window minimum and step (Eq. 4)
    int c = tid;
    float mn = sm.z[c], mx = mn;
    for (int i = 1; i < W; i++) {
      float v = sm.z[i * ZS + c];
      if (v < mn) mn = v;
      if (v > mx) mx = v;
    }
    __half mh = __float2half_rn(mn);
    float mf = __half2float(mh);
    float range = __fsub_rn(mx, mf);
    if (range < 0.0f) range = 0.0f;
    __half sh = __float2half_rn(__fdiv_rn(range, 3.0f));
    float sf = __half2float(sh);
    sm.a[c] = mf;
    sm.b[c] = sf > 0.0f ? __fdiv_rn(1.0f, sf) : 0.0f;
    int p = meta_pos(c);
    reinterpret_cast<__half*>(rec + OFF_KM)[p] = mh;
    reinterpret_cast<__half*>(rec + OFF_KS)[p] = sh;
  }
  __syncthreads();
  uint32_t* words = reinterpret_cast<uint32_t*>(rec + OFF_KCODE);
  for (int wi = tid; wi < 256; wi += 128) {
    int h2 = wi >> 7, rem = wi & 127;
    int l = rem >> 2, tt = (rem >> 1) & 1, ww = rem & 1;
    int g = l >> 2, t = l & 3;
    int i = g + 8 * (2 * h2 + tt);
    uint32_t word = 0;
#pragma unroll
    for (int q = 0; q < 8; q++) {
      int r = ww * 8 + q;
      int kappa = r >> 1, pair = r & 1;
#pragma unroll
      for (int e = 0; e < 2; e++) {
        int c = 16 * kappa + 8 * pair + 2 * t + e;
        float qv = rintf(__fmul_rn(__fsub_rn(sm.z[i * ZS + c], sm.a[c]), sm.b[c]));
        uint32_t code = qv < 0.0f ? 0u : (qv > 3.0f ? 3u : (uint32_t)qv);
        word |= code << (16 * e + 8 * (q >> 2) + 2 * (q & 3));
      }
    }
    words[wi] = word;
  }
  __syncthreads();
}

// Value window.  mod[] must already be in sm.mod and sm.uniform set.  Rset = R + rsel*3*D*D.
__device__ void quantize_value_window(const __half* rows, long long stride, const float* __restrict__ Rset,
                                      unsigned char* rec, WindowSmem& sm) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  __half* vnorm = reinterpret_cast<__half*>(rec + OFF_VNORM);
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
  uint32_t* words = reinterpret_cast<uint32_t*>(rec + OFF_VCODE);
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
    words[wi] = word;
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
  quantize_key_window(rows, st, signs, cv.record(layer, b, h, win), sm);
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
  quantize_value_window(rows, st, Rset, cv.record(layer, b, h, win), sm);
}

// raw tail copy + seq_len (+ modality for the value call); grid (n_kv_heads, batch), 128 threads
__global__ void k_bulk_tail(CacheView cv, int layer, const __half* __restrict__ src, long long sb, long long sh,
                            long long st, int n_tokens, __half* tail, const unsigned char* __restrict__ modality) {
  int h = blockIdx.x, b = blockIdx.y;
  int n_packed = n_tokens & ~(W - 1);
  int n_tail = n_tokens - n_packed;
  __half* dst = tail + cv.tail_off(layer, b, h);
  for (int idx = threadIdx.x; idx < n_tail * (D / 8); idx += blockDim.x) {
    int i = idx / (D / 8), c8 = idx % (D / 8);
    reinterpret_cast<uint4*>(dst + i * D)[c8] =
        *reinterpret_cast<const uint4*>(src + b * sb + h * sh + (long long)(n_packed + i) * st + c8 * 8);
  }
  if (h == 0) {
    if (threadIdx.x == 0) cv.seq_len[layer * cv.batch + b] = n_tokens;
    if (modality)
      for (int i = threadIdx.x; i < n_tokens; i += blockDim.x) {
        unsigned char m = modality[(size_t)b * n_tokens + i];
        cv.modality[(size_t)b * cv.capacity + i] = m > 2 ? 0 : m;
      }
  }
}

// ---------------------------------------------------------------- append

// grid (n_kv_heads, batch, layer_count), 128 threads
__global__ void __launch_bounds__(128) k_append(CacheView cv, int layer0, const __half* __restrict__ k_new,
                                               const __half* __restrict__ v_new,
                                               const unsigned char* __restrict__ mod_new,
                                               const float* __restrict__ signs, const float* __restrict__ R,
                                               int n_R) {
  __shared__ WindowSmem sm;
  int h = blockIdx.x, b = blockIdx.y, li = blockIdx.z, layer = layer0 + li;
  int pos = cv.seq_len[layer * cv.batch + b];
  if (pos >= cv.capacity) {
    if (threadIdx.x == 0) atomicCAS(cv.status, 0, (int)OKQ_ERR_CAPACITY);
    return;
  }
  int slot = pos & (W - 1);
  size_t src = (((size_t)li * cv.batch + b) * cv.n_kv_heads + h) * D;
  __half* kt = cv.k_tail + cv.tail_off(layer, b, h);
  __half* vt = cv.v_tail + cv.tail_off(layer, b, h);
  unsigned char mnew = mod_new[b];
  mnew = mnew > 2 ? 0 : mnew;
  if (threadIdx.x < 16) reinterpret_cast<uint4*>(kt + slot * D)[threadIdx.x] = reinterpret_cast<const uint4*>(k_new + src)[threadIdx.x];
  else if (threadIdx.x < 32) reinterpret_cast<uint4*>(vt + slot * D)[threadIdx.x - 16] = reinterpret_cast<const uint4*>(v_new + src)[threadIdx.x - 16];
  if (h == 0 && threadIdx.x == 32) cv.modality[(size_t)b * cv.capacity + pos] = mnew;
  if (slot != W - 1) return;
  __syncthreads();  // the 32nd token of the window is now visible to the whole block
  unsigned char* rec = cv.record(layer, b, h, pos / W);
  quantize_key_window(kt, D, signs + (size_t)li * D, rec, sm);
  if (threadIdx.x < 32) {
    unsigned char m = threadIdx.x == W - 1 ? mnew : cv.modality[(size_t)b * cv.capacity + (pos - (W - 1)) + threadIdx.x];
    sm.mod[threadIdx.x] = m;
    unsigned char m0 = __shfl_sync(0xffffffffu, m, 0);
    int uni = __all_sync(0xffffffffu, m == m0);
    if (threadIdx.x == 0) sm.uniform = uni;
  }
  __syncthreads();
  const float* Rset = R + ((size_t)li * n_R + (n_R == 1 ? 0 : h)) * 3 * D * D;
  quantize_value_window(vt, D, Rset, rec, sm);
}

__global__ void k_advance(CacheView cv, int layer0, int layer_count) {
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= layer_count * cv.batch) return;
  int* p = cv.seq_len + (size_t)layer0 * cv.batch + idx;
  if (*p < cv.capacity) *p += 1;
}

// ---------------------------------------------------------------- canonical <-> physical

// grid (capacity/32, n_kv_heads, batch), 128 threads
__global__ void k_export(CacheView cv, int layer, unsigned char* k_codes, __half* k_norm, __half* k_meta,
                         unsigned char* v_codes, __half* v_norm) {
  int win = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const unsigned char* rec = cv.record(layer, b, h, win);
  size_t unit = (size_t)b * cv.n_kv_heads + h;
  size_t tok0 = unit * cv.capacity + (size_t)win * W;
  const uint32_t* kw = reinterpret_cast<const uint32_t*>(rec + OFF_KCODE);
  const uint32_t* vw = reinterpret_cast<const uint32_t*>(rec + OFF_VCODE);
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
    k_norm[tok0 + threadIdx.x] = reinterpret_cast<const __half*>(rec + OFF_KNORM)[norm_pos(threadIdx.x)];
    v_norm[tok0 + threadIdx.x] = reinterpret_cast<const __half*>(rec + OFF_VNORM)[norm_pos(threadIdx.x)];
  }
  {
    int c = threadIdx.x, p = meta_pos(c);
    size_t o = ((unit * cv.n_windows() + win) * D + c) * 2;
    k_meta[o] = reinterpret_cast<const __half*>(rec + OFF_KM)[p];
    k_meta[o + 1] = reinterpret_cast<const __half*>(rec + OFF_KS)[p];
  }
}

__global__ void k_import(CacheView cv, int layer, const unsigned char* k_codes, const __half* k_norm,
                         const __half* k_meta, const unsigned char* v_codes, const __half* v_norm) {
  int win = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  unsigned char* rec = cv.record(layer, b, h, win);
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
    reinterpret_cast<__half*>(rec + OFF_KM)[p] = k_meta[o];
    reinterpret_cast<__half*>(rec + OFF_KS)[p] = k_meta[o + 1];
  }
}

okq_status launch_quantize_values_tc(const CacheView& cv, int layer, const __half* v, const int64_t strides[3],
                                     const unsigned char* modality, int n_tokens, const float* R, int n_R,
                                     int n_sm, cudaStream_t s);

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
  int n_win = n_tokens / W;
  if (n_win > 0) {
    dim3 grid(n_win, cv.n_kv_heads, cv.batch);
    k_quantize_keys<<<grid, 128, 0, s>>>(cv, layer, k, strides[0], strides[1], strides[2], signs);
  }
  k_bulk_tail<<<dim3(cv.n_kv_heads, cv.batch), 128, 0, s>>>(cv, layer, k, strides[0], strides[1], strides[2],
                                                           n_tokens, cv.k_tail, nullptr);
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
  int n_win = n_tokens / W;
  if (n_win > 0) {
    dim3 grid(n_win, cv.n_kv_heads, cv.batch);
    k_quantize_values<<<grid, 128, 0, s>>>(cv, layer, v, strides[0], strides[1], strides[2], modality, n_tokens, R,
                                           n_R);
  }
  k_bulk_tail<<<dim3(cv.n_kv_heads, cv.batch), 128, 0, s>>>(cv, layer, v, strides[0], strides[1], strides[2],
                                                           n_tokens, cv.v_tail, n_tokens > 0 ? modality : nullptr);
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
  st = launch_quantize_values_tc(cv, layer, v, strides, modality, n_tokens, R, n_R, sm_count(), s);
  if (st != OKQ_OK) return st;
  k_bulk_tail<<<dim3(cv.n_kv_heads, cv.batch), 128, 0, s>>>(cv, layer, v, strides[0], strides[1], strides[2],
                                                           n_tokens, cv.v_tail, n_tokens > 0 ? modality : nullptr);
  return launch_status();
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
  k_append<<<dim3(cv.n_kv_heads, cv.batch, layer_count), 128, 0, s>>>(
      cv, layer, static_cast<const __half*>(k_new), static_cast<const __half*>(v_new), modality_new, signs, R, n_R);
  int n = layer_count * cv.batch;
  k_advance<<<(n + 127) / 128, 128, 0, s>>>(cv, layer, layer_count);
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
      static_cast<__half*>(v_norm));
  return launch_status();
}

okq_status okq_cache_import(const okq_cache* cache, int32_t layer, const uint8_t* k_codes, const void* k_norm,
                            const void* k_meta, const uint8_t* v_codes, const void* v_norm, void* stream) {
  okq_status st = check_cache(cache, true);
  if (st != OKQ_OK) return st;
  if (layer < 0 || layer >= cache->n_layers || !k_codes || !k_norm || !k_meta || !v_codes || !v_norm)
    return OKQ_ERR_INVALID_ARG;
  CacheView cv = make_view(cache);
  k_import<<<dim3(cv.capacity / W, cv.n_kv_heads, cv.batch), 128, 0, static_cast<cudaStream_t>(stream)>>>(
      cv, layer, k_codes, static_cast<const __half*>(k_norm), static_cast<const __half*>(k_meta), v_codes,
      static_cast<const __half*>(v_norm));
  return launch_status();
}

}  // extern "C"
