// Fused decode attention over the packed cache: split-K kernel + combine kernel.
//
// Scores are taken in the rotated space (q' = H q once per head; q . k_hat =
// norm * (sum_c q'_c m_gc + sum_c q'_c s_gc code_c)), the softmax runs online per warp in
// FlashAttention order, the softmax-weighted codebook levels are accumulated per modality in
// the rotated basis, and the combine kernel merges the splits and applies R_m^T once per
// head.  No fp16 K or V is ever rebuilt.
#include "okq_common.cuh"
#include "okq_device.cuh"
#include "okq_decode_shared.cuh"

namespace okq {

struct WarpSmem {
  __align__(16) unsigned char rec[RECORD_BYTES];
  __align__(16) float w[D][GP];   // per-window weights q'_c * s_gc, position-major
  __align__(16) float p[W][GP];   // softmax numerators times value norm
  unsigned char mod[W];
};

struct DecodeSmem {
  __align__(16) float qrot[GP][D];  // q' in the record's channel order
  __align__(16) float qraw[GP][D];  // q, natural order (for the raw tail)
  WarpSmem warp[4];
  float red_m[4][GP], red_l[4][GP];
  __align__(16) float accbuf[NACC][GP][D];
};

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int d = 16; d; d >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, d));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int d = 16; d; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
  return v;
}

// channel owned by (lane, k): lane = 4*g + a, k = 2*musel + sh  ->  16*(a + 4*musel) + 8*sh + g
__device__ __forceinline__ int own_channel(int lane, int k) {
  int g = lane >> 2, a = lane & 3;
  return 16 * (a + 4 * (k >> 1)) + 8 * (k & 1) + g;
}

// grid (n_splits, n_kv_heads, batch*layer_count), 128 threads
__global__ void __launch_bounds__(128) k_decode_simt(DecodeParams P) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  DecodeSmem& sm = *reinterpret_cast<DecodeSmem*>(smem_raw);
  const CacheView& cv = P.cv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int split = blockIdx.x, h = blockIdx.y;
  const int b = blockIdx.z % cv.batch, li = blockIdx.z / cv.batch, layer = P.layer0 + li;
  const int G = P.group;

  // q' = H q for the group's heads (zero for the padding heads)
  for (int hh = warp; hh < GP; hh += 4) {
    float4 qr = make_float4(0, 0, 0, 0), x = qr;
    if (hh < G) {
      const __half* qrow = P.q + (((size_t)li * cv.batch + b) * cv.n_q_heads + h * G + hh) * D;
      x = load_row4(qrow, lane);
      const float4 sg = *reinterpret_cast<const float4*>(P.signs + (size_t)li * D + 4 * lane);
      qr = warp_fwht(make_float4(x.x * sg.x, x.y * sg.y, x.z * sg.z, x.w * sg.w), lane);
    }
    float v[4] = {qr.x * RSQRT_D, qr.y * RSQRT_D, qr.z * RSQRT_D, qr.w * RSQRT_D};
#pragma unroll
    for (int k = 0; k < 4; k++) sm.qrot[hh][meta_pos(4 * lane + k)] = v[k];
    *reinterpret_cast<float4*>(&sm.qraw[hh][4 * lane]) = x;
  }
  __syncthreads();

  const int seq = cv.seq_len[layer * cv.batch + b];
  const int n_win = seq / W, n_tail = seq - n_win * W;
  const int per = (n_win + P.n_splits - 1) / P.n_splits;
  const int w_begin = split * per, w_end = min(n_win, w_begin + per);

  WarpSmem& ws = sm.warp[warp];
  float run_m[GP], run_l[GP], acc[NACC][GP][4];
#pragma unroll
  for (int j = 0; j < GP; j++) { run_m[j] = -INFINITY; run_l[j] = 0.f; }
#pragma unroll
  for (int a = 0; a < NACC; a++)
#pragma unroll
    for (int j = 0; j < GP; j++)
#pragma unroll
      for (int k = 0; k < 4; k++) acc[a][j][k] = 0.f;

  const float cb[4] = {-CB_OUTER, -CB_INNER, CB_INNER, CB_OUTER};

  for (int win = w_begin + warp; win < w_end; win += 4) {
    if (cv.fmt == FMT_FP16) {
      const unsigned char* rec = cv.meta(layer, b, h, win);
      for (int i = lane; i < RECORD_BYTES / 16; i += 32)
        reinterpret_cast<uint4*>(ws.rec)[i] = __ldg(reinterpret_cast<const uint4*>(rec) + i);
    } else {
      // same staged image as with fp16 metadata: the body behind 512 bytes of decoded (m, s)
      const unsigned char* body = cv.body(layer, b, h, win);
      for (int i = lane; i < BODY_BYTES / 16; i += 32)
        reinterpret_cast<uint4*>(ws.rec + META_BYTES_FP16)[i] = __ldg(reinterpret_cast<const uint4*>(body) + i);
      uint2 m4, s4;
      mx_decode_lane(cv.meta(layer, b, h, win), lane, m4, s4);
      *reinterpret_cast<uint2*>(ws.rec + OFF_KM + 8 * lane) = m4;
      *reinterpret_cast<uint2*>(ws.rec + OFF_KS + 8 * lane) = s4;
    }
    ws.mod[lane] = cv.modality[(size_t)b * cv.capacity + (size_t)win * W + lane];
    __syncwarp();
    // per-window weights and bias
    float bias[GP];
    {
      const __half* mp = reinterpret_cast<const __half*>(ws.rec + OFF_KM);
      const __half* sp = reinterpret_cast<const __half*>(ws.rec + OFF_KS);
#pragma unroll
      for (int j = 0; j < GP; j++) bias[j] = 0.f;
#pragma unroll
      for (int k = 0; k < 4; k++) {
        int p = 4 * lane + k;
        float mf = __half2float(mp[p]) * (1.0f / (float)(1 << (2 * meta_shift_pos(p)))), sf = __half2float(sp[p]);
        float wv[GP];
#pragma unroll
        for (int j = 0; j < GP; j++) {
          float qv = sm.qrot[j][p];
          wv[j] = qv * sf;
          bias[j] = fmaf(qv, mf, bias[j]);
        }
        *reinterpret_cast<float4*>(&ws.w[p][0]) = make_float4(wv[0], wv[1], wv[2], wv[3]);
        *reinterpret_cast<float4*>(&ws.w[p][4]) = make_float4(wv[4], wv[5], wv[6], wv[7]);
      }
#pragma unroll
      for (int j = 0; j < GP; j++) bias[j] = warp_sum(bias[j]);
    }
    __syncwarp();
    // scores: lane = token
    float s[GP];
#pragma unroll
    for (int j = 0; j < GP; j++) s[j] = 0.f;
    {
      const uint32_t* kw = reinterpret_cast<const uint32_t*>(ws.rec + OFF_KCODE);
      int nu = lane >> 3, g = lane & 7;
      for (int t = 0; t < 4; t++) {
        uint2 wd = *reinterpret_cast<const uint2*>(&kw[kword_index((nu >> 1) * 128 + (4 * g + t) * 4 + (nu & 1) * 2)]);
#pragma unroll
        for (int ww = 0; ww < 2; ww++) {
          uint32_t word = ww ? wd.y : wd.x;
#pragma unroll
          for (int qd = 0; qd < 8; qd++) {
#pragma unroll
            for (int e = 0; e < 2; e++) {
              float code = (float)((word >> (16 * e + 8 * (qd >> 2) + 2 * (qd & 3))) & 3u);
              int p = t * 32 + (ww * 8 + qd) * 2 + e;
              float4 w0 = *reinterpret_cast<const float4*>(&ws.w[p][0]);
              float4 w1 = *reinterpret_cast<const float4*>(&ws.w[p][4]);
              s[0] = fmaf(w0.x, code, s[0]); s[1] = fmaf(w0.y, code, s[1]);
              s[2] = fmaf(w0.z, code, s[2]); s[3] = fmaf(w0.w, code, s[3]);
              s[4] = fmaf(w1.x, code, s[4]); s[5] = fmaf(w1.y, code, s[5]);
              s[6] = fmaf(w1.z, code, s[6]); s[7] = fmaf(w1.w, code, s[7]);
            }
          }
        }
      }
    }
    const float kn = __half2float(reinterpret_cast<const __half*>(ws.rec + OFF_KNORM)[norm_pos(lane)]) * P.sm_scale;
    const float vn = __half2float(reinterpret_cast<const __half*>(ws.rec + OFF_VNORM)[norm_pos(lane)]);
    float pw[GP];
#pragma unroll
    for (int j = 0; j < GP; j++) {
      float sc = (s[j] + bias[j]) * kn;
      float mnew = fmaxf(run_m[j], warp_max(sc));
      float alpha = __expf(run_m[j] - mnew);  // exp(-inf) = 0 on the first window
      float pj = __expf(sc - mnew);
      run_l[j] = run_l[j] * alpha + pj;
      run_m[j] = mnew;
      pw[j] = pj * vn;
#pragma unroll
      for (int a = 0; a < 3; a++)
#pragma unroll
        for (int k = 0; k < 4; k++) acc[a][j][k] *= alpha;
    }
    *reinterpret_cast<float4*>(&ws.p[lane][0]) = make_float4(pw[0], pw[1], pw[2], pw[3]);
    *reinterpret_cast<float4*>(&ws.p[lane][4]) = make_float4(pw[4], pw[5], pw[6], pw[7]);
    __syncwarp();
    // values: lane owns 4 channels
    unsigned char m0 = ws.mod[0];
    bool uniform = __all_sync(0xffffffffu, ws.mod[lane] == m0);
    const uint32_t* vw = reinterpret_cast<const uint32_t*>(ws.rec + OFF_VCODE);
    const int gq = lane >> 2, aq = lane & 3;
    for (int mm = 0; mm < 3; mm++) {
      if (uniform ? (mm != m0) : !__any_sync(0xffffffffu, ws.mod[lane] == mm)) continue;
      float tmp[GP][4];
#pragma unroll
      for (int j = 0; j < GP; j++)
#pragma unroll
        for (int k = 0; k < 4; k++) tmp[j][k] = 0.f;
#pragma unroll
      for (int musel = 0; musel < 2; musel++) {
        for (int t = 0; t < 4; t++) {
          uint32_t word = vw[vword_index(musel * 128 + (4 * gq + t) * 4 + aq)];
#pragma unroll
          for (int qd = 0; qd < 8; qd++) {
            int sh = qd >> 2, jj = qd & 3;
#pragma unroll
            for (int e = 0; e < 2; e++) {
              int tok = 16 * (jj >> 1) + 8 * (jj & 1) + 2 * t + e;
              float lvl = cb[(word >> (16 * e + 8 * sh + 2 * jj)) & 3u];
              if (!uniform && ws.mod[tok] != mm) lvl = 0.f;
              float4 p0 = *reinterpret_cast<const float4*>(&ws.p[tok][0]);
              float4 p1 = *reinterpret_cast<const float4*>(&ws.p[tok][4]);
              int k = musel * 2 + sh;
              tmp[0][k] = fmaf(p0.x, lvl, tmp[0][k]); tmp[1][k] = fmaf(p0.y, lvl, tmp[1][k]);
              tmp[2][k] = fmaf(p0.z, lvl, tmp[2][k]); tmp[3][k] = fmaf(p0.w, lvl, tmp[3][k]);
              tmp[4][k] = fmaf(p1.x, lvl, tmp[4][k]); tmp[5][k] = fmaf(p1.y, lvl, tmp[5][k]);
              tmp[6][k] = fmaf(p1.z, lvl, tmp[6][k]); tmp[7][k] = fmaf(p1.w, lvl, tmp[7][k]);
            }
          }
        }
      }
#pragma unroll
      for (int a = 0; a < 3; a++)
        if (a == mm)
#pragma unroll
          for (int j = 0; j < GP; j++)
#pragma unroll
            for (int k = 0; k < 4; k++) acc[a][j][k] += tmp[j][k];
    }
    __syncwarp();
  }

  // raw fp16 tail: last split, warp 0
  if (split == P.n_splits - 1 && warp == 0 && n_tail > 0) {
    const __half* kt = cv.k_tail + cv.k_tail_off(layer, b, h);
    const __half* vt = cv.v_tail + cv.v_tail_off(layer, b, h);
    float s[GP];
#pragma unroll
    for (int j = 0; j < GP; j++) s[j] = 0.f;
    if (lane < n_tail) {
      for (int c8 = 0; c8 < D / 8; c8++) {
        uint4 raw = *reinterpret_cast<const uint4*>(kt + lane * D + c8 * 8);
        const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
        for (int u = 0; u < 4; u++) {
          float2 kv = __half22float2(h2[u]);
#pragma unroll
          for (int j = 0; j < GP; j++) {
            s[j] = fmaf(sm.qraw[j][c8 * 8 + 2 * u], kv.x, s[j]);
            s[j] = fmaf(sm.qraw[j][c8 * 8 + 2 * u + 1], kv.y, s[j]);
          }
        }
      }
    }
    float pw[GP];
#pragma unroll
    for (int j = 0; j < GP; j++) {
      float sc = lane < n_tail ? s[j] * P.sm_scale : -INFINITY;
      float mnew = fmaxf(run_m[j], warp_max(sc));
      float alpha = __expf(run_m[j] - mnew);
      float pj = __expf(sc - mnew);
      run_l[j] = run_l[j] * alpha + pj;
      run_m[j] = mnew;
      pw[j] = pj;
#pragma unroll
      for (int a = 0; a < NACC; a++)
#pragma unroll
        for (int k = 0; k < 4; k++) acc[a][j][k] *= alpha;
    }
    *reinterpret_cast<float4*>(&ws.p[lane][0]) = make_float4(pw[0], pw[1], pw[2], pw[3]);
    *reinterpret_cast<float4*>(&ws.p[lane][4]) = make_float4(pw[4], pw[5], pw[6], pw[7]);
    __syncwarp();
    for (int i = 0; i < n_tail; i++) {
#pragma unroll
      for (int k = 0; k < 4; k++) {
        float v = __half2float(vt[i * D + own_channel(lane, k)]);
#pragma unroll
        for (int j = 0; j < GP; j++) acc[3][j][k] = fmaf(ws.p[i][j], v, acc[3][j][k]);
      }
    }
  }

  // merge the four warps
#pragma unroll
  for (int j = 0; j < GP; j++) {
    float lt = warp_sum(run_l[j]);
    if (lane == 0) { sm.red_m[warp][j] = run_m[j]; sm.red_l[warp][j] = lt; }
  }
  __syncthreads();
  float scale[GP];
#pragma unroll
  for (int j = 0; j < GP; j++) {
    float M = fmaxf(fmaxf(sm.red_m[0][j], sm.red_m[1][j]), fmaxf(sm.red_m[2][j], sm.red_m[3][j]));
    scale[j] = run_m[j] == -INFINITY ? 0.f : __expf(run_m[j] - M);
  }
  for (int wsel = 0; wsel < 4; wsel++) {
    if (warp == wsel) {
#pragma unroll
      for (int a = 0; a < NACC; a++)
#pragma unroll
        for (int j = 0; j < GP; j++)
#pragma unroll
          for (int k = 0; k < 4; k++) {
            float v = acc[a][j][k] * scale[j];
            float* dst = &sm.accbuf[a][j][own_channel(lane, k)];
            *dst = wsel == 0 ? v : *dst + v;
          }
    }
    __syncthreads();
  }
  Partial* out = P.partials + ((((size_t)li * cv.batch + b) * cv.n_kv_heads + h) * P.n_splits + split);
  if (tid < GP) {
    int j = tid;
    float M = fmaxf(fmaxf(sm.red_m[0][j], sm.red_m[1][j]), fmaxf(sm.red_m[2][j], sm.red_m[3][j]));
    float L = 0.f;
    for (int w4 = 0; w4 < 4; w4++)
      L += sm.red_m[w4][j] == -INFINITY ? 0.f : sm.red_l[w4][j] * __expf(sm.red_m[w4][j] - M);
    out->m[j] = M;
    out->l[j] = L;
  }
  const float4* src = reinterpret_cast<const float4*>(&sm.accbuf[0][0][0]);
  float4* dst = reinterpret_cast<float4*>(&out->acc[0][0][0]);
  for (int i = tid; i < NACC * GP * D / 4; i += 128) dst[i] = src[i];
}

// grid (n_kv_heads, batch*layer_count), 128 threads: merge splits, apply R_m^T, normalise
__global__ void __launch_bounds__(128) k_combine(DecodeParams P) {
  __shared__ float vec[3][GP][D];
  __shared__ float Ls[GP];
  const CacheView& cv = P.cv;
  const int h = blockIdx.x, b = blockIdx.y % cv.batch, li = blockIdx.y / cv.batch;
  const int c = threadIdx.x, G = P.group;
  const Partial* parts = P.partials + (((size_t)li * cv.batch + b) * cv.n_kv_heads + h) * P.n_splits;
  float raw[GP];
  for (int j = 0; j < G; j++) {
    float M = -INFINITY;
    for (int s = 0; s < P.n_splits; s++) M = fmaxf(M, parts[s].m[j]);
    float L = 0.f, v[NACC] = {0.f, 0.f, 0.f, 0.f};
    for (int s = 0; s < P.n_splits; s++) {
      float ms = parts[s].m[j];
      if (ms == -INFINITY) continue;
      float e = __expf(ms - M);
      L += parts[s].l[j] * e;
#pragma unroll
      for (int a = 0; a < NACC; a++) v[a] = fmaf(parts[s].acc[a][j][c], e, v[a]);
    }
    vec[0][j][c] = v[0]; vec[1][j][c] = v[1]; vec[2][j][c] = v[2];
    raw[j] = v[3];
    if (c == 0) Ls[j] = L;
  }
  __syncthreads();
  float o[GP];
#pragma unroll
  for (int j = 0; j < GP; j++) o[j] = 0.f;
  const float* Rset = P.R + ((size_t)li * P.n_R + (P.n_R == 1 ? 0 : h)) * 3 * D * D;
  for (int m = 0; m < 3; m++)
    for (int r = 0; r < D; r++) {
      float rv = __ldg(Rset + ((size_t)m * D + r) * D + c);
#pragma unroll
      for (int j = 0; j < GP; j++) o[j] = fmaf(rv, vec[m][j][r], o[j]);
    }
  for (int j = 0; j < G; j++) {
    float L = Ls[j];
    P.out[(((size_t)li * cv.batch + b) * cv.n_q_heads + h * G + j) * D + c] = L > 0.f ? (o[j] + raw[j]) / L : 0.f;
  }
}

static thread_local cudaEvent_t g_ev_before = nullptr, g_ev_after = nullptr;

// Scratch of okq_decode_attention_noalloc: lives in the library's device image, so every GPU
// that loads the library holds these bytes until the process exits.  In host code the name
// below is only a handle; the device address comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_noalloc_scratch[OKQ_NOALLOC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
static void* g_noalloc_ptr[MAX_DEVICES];   // device address of g_noalloc_scratch, per device (0 = not resolved yet)

// Resolves the scratch address on the current device (first call per device only).
static okq_status noalloc_scratch(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { set_last_cuda_error((int)e); return OKQ_ERR_CUDA; }
  if (dev < 0 || dev >= MAX_DEVICES) return OKQ_ERR_UNSUPPORTED;
  void* p = __atomic_load_n(&g_noalloc_ptr[dev], __ATOMIC_ACQUIRE);
  if (!p) {
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess || !p) { set_last_cuda_error((int)e); return OKQ_ERR_CUDA; }
    __atomic_store_n(&g_noalloc_ptr[dev], p, __ATOMIC_RELEASE);   // every thread resolves the same address
  }
  *out = p;
  return OKQ_OK;
}

static int auto_splits(const okq_cache* c, int layer_count) {
  long long units = (long long)layer_count * c->batch * c->n_kv_heads;
  long long want = (2 * 148 + units - 1) / units;
  long long cap = c->capacity / W / 16;
  if (cap < 1) cap = 1;
  if (want > cap) want = cap;
  if (want < 1) want = 1;
  return (int)want;
}

// persistent grid of the tensor-core kernel
static int mma_ctas(const okq_cache* c, int layer_count, int num_splits) {
  if (num_splits <= 0) return sm_count();
  long long n = (long long)num_splits * layer_count * c->batch * c->n_kv_heads;
  return (int)(n > 1024 ? 1024 : n);
}

static size_t simt_workspace(const okq_cache* c, int layer_count, int num_splits) {
  int S = num_splits > 0 ? num_splits : auto_splits(c, layer_count);
  return (size_t)layer_count * c->batch * c->n_kv_heads * S * sizeof(Partial);
}

// one PartialF per (CTA, (sequence, head)) overlap, then one PairPartial per (warp pair, (sequence, head))
// overlap: slot = unit index + CTA (or global pair) index, both non-decreasing along the window axis
static size_t mma_partials_bytes(const okq_cache* c, int layer_count, int num_splits) {
  return ((size_t)layer_count * c->batch * c->n_kv_heads + mma_ctas(c, layer_count, num_splits)) * sizeof(PartialF);
}
static size_t mma_workspace(const okq_cache* c, int layer_count, int num_splits) {
  return mma_partials_bytes(c, layer_count, num_splits) +
         ((size_t)layer_count * c->batch * c->n_kv_heads + (size_t)MMA_PAIRS * mma_ctas(c, layer_count, num_splits)) *
             sizeof(PairPartial);
}

static okq_status check_decode(const okq_cache* cache, int32_t layer, int32_t layer_count, const void* q,
                               const float* signs, const float* R, int32_t n_R, void* workspace,
                               size_t workspace_bytes, int32_t num_splits, float* out) {
  okq_status st = check_cache(cache, true);
  if (st != OKQ_OK) return st;
  if (!q || !signs || !R || !workspace || !out || num_splits < 0) return OKQ_ERR_INVALID_ARG;
  if (layer < 0 || layer_count <= 0 || layer + layer_count > cache->n_layers) return OKQ_ERR_INVALID_ARG;
  if (n_R != 1 && n_R != cache->n_kv_heads) return OKQ_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(signs) || !aligned16(R) || !aligned16(workspace) || !aligned16(out))
    return OKQ_ERR_ALIGNMENT;
  if (workspace_bytes < okq_decode_workspace_bytes(cache, layer_count, num_splits)) return OKQ_ERR_WORKSPACE;
  return OKQ_OK;
}

static DecodeParams make_params(const okq_cache* cache, int32_t layer, int32_t layer_count, const void* q,
                                float sm_scale, const float* signs, const float* R, int32_t n_R, float* out) {
  DecodeParams P;
  P.cv = make_view(cache);
  P.layer0 = layer; P.layer_count = layer_count; P.n_splits = 1;
  P.group = cache->n_q_heads / cache->n_kv_heads;
  P.q = static_cast<const __half*>(q); P.signs = signs; P.R = R; P.n_R = n_R; P.sm_scale = sm_scale;
  P.partials = nullptr; P.partials_f = nullptr; P.pair_parts = nullptr; P.out = out;
  return P;
}

}  // namespace okq

using namespace okq;

extern "C" {

void okq_profile_events(void* before, void* after) {
  g_ev_before = static_cast<cudaEvent_t>(before);
  g_ev_after = static_cast<cudaEvent_t>(after);
}

int32_t okq_decode_select(int32_t impl) {
  const int32_t prev = g_decode_impl;
  if (impl == 0 || impl == 1) g_decode_impl = impl;
  return prev;
}

size_t okq_decode_workspace_bytes(const okq_cache* cache, int32_t layer_count, int32_t num_splits) {
  if (check_cache(cache, false) != OKQ_OK || layer_count <= 0 || num_splits < 0) return 0;
  size_t a = simt_workspace(cache, layer_count, num_splits), b = mma_workspace(cache, layer_count, num_splits);
  return a > b ? a : b;
}

okq_status okq_decode_attention(const okq_cache* cache, int32_t layer, int32_t layer_count, const void* q,
                                float sm_scale, const float* signs, const float* R, int32_t n_R, void* workspace,
                                size_t workspace_bytes, int32_t num_splits, float* out, void* stream) {
  okq_status st = check_decode(cache, layer, layer_count, q, signs, R, n_R, workspace, workspace_bytes, num_splits, out);
  if (st != OKQ_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // one launch covers at most MAX_ENTRIES (layer, sequence) pairs
  const int layers_per_launch = cache->batch >= MAX_ENTRIES ? 1 : MAX_ENTRIES / cache->batch;
  if (cache->batch > MAX_ENTRIES) return OKQ_ERR_UNSUPPORTED;
  const size_t q_stride = (size_t)cache->batch * cache->n_q_heads * D;
  for (int l0 = 0; l0 < layer_count; l0 += layers_per_launch) {
    const int lc = layer_count - l0 < layers_per_launch ? layer_count - l0 : layers_per_launch;
    DecodeParams P = make_params(cache, layer + l0, lc, static_cast<const __half*>(q) + l0 * q_stride, sm_scale,
                                 signs + (size_t)l0 * D, R + (size_t)l0 * n_R * 3 * D * D, n_R, out + l0 * q_stride);
    P.partials_f = static_cast<PartialF*>(workspace);
    P.pair_parts = reinterpret_cast<PairPartial*>(static_cast<unsigned char*>(workspace) +
                                                  mma_partials_bytes(cache, lc, num_splits));
    const int n_cta = mma_ctas(cache, lc, num_splits);
    st = launch_decode_mma(P, n_cta, s, g_ev_before, g_ev_after);
    if (st != OKQ_OK) return st;
  }
  return launch_status();
}

okq_status okq_decode_attention_noalloc(const okq_cache* cache, int32_t layer, int32_t layer_count, const void* q,
                                        float sm_scale, const float* signs, const float* R, int32_t n_R,
                                        int32_t num_splits, float* out, void* stream) {
  okq_status st = check_cache(cache, false);
  if (st != OKQ_OK) return st;
  if (layer_count <= 0 || num_splits < 0) return OKQ_ERR_INVALID_ARG;
  // the largest launch of the call decides how much of the fixed scratch is needed
  const int layers_per_launch = cache->batch >= MAX_ENTRIES ? 1 : MAX_ENTRIES / cache->batch;
  const int lc_max = layer_count < layers_per_launch ? layer_count : layers_per_launch;
  if (mma_workspace(cache, lc_max, num_splits) > (size_t)OKQ_NOALLOC_SCRATCH_BYTES) return OKQ_ERR_WORKSPACE;
  void* scratch = nullptr;
  st = noalloc_scratch(&scratch);
  if (st != OKQ_OK) return st;
  st = check_decode(cache, layer, layer_count, q, signs, R, n_R, scratch, (size_t)-1, num_splits, out);
  if (st != OKQ_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cache->batch > MAX_ENTRIES) return OKQ_ERR_UNSUPPORTED;
  const size_t q_stride = (size_t)cache->batch * cache->n_q_heads * D;
  for (int l0 = 0; l0 < layer_count; l0 += layers_per_launch) {
    const int lc = layer_count - l0 < layers_per_launch ? layer_count - l0 : layers_per_launch;
    DecodeParams P = make_params(cache, layer + l0, lc, static_cast<const __half*>(q) + l0 * q_stride, sm_scale,
                                 signs + (size_t)l0 * D, R + (size_t)l0 * n_R * 3 * D * D, n_R, out + l0 * q_stride);
    P.partials_f = static_cast<PartialF*>(scratch);
    P.pair_parts = reinterpret_cast<PairPartial*>(static_cast<unsigned char*>(scratch) +
                                                  mma_partials_bytes(cache, lc, num_splits));
    st = launch_decode_mma(P, mma_ctas(cache, lc, num_splits), s, nullptr, nullptr);
    if (st != OKQ_OK) return st;
  }
  return launch_status();
}

okq_status okq_decode_attention_simt(const okq_cache* cache, int32_t layer, int32_t layer_count, const void* q,
                                     float sm_scale, const float* signs, const float* R, int32_t n_R,
                                     void* workspace, size_t workspace_bytes, int32_t num_splits, float* out,
                                     void* stream) {
  okq_status st = check_decode(cache, layer, layer_count, q, signs, R, n_R, workspace, workspace_bytes, num_splits, out);
  if (st != OKQ_OK) return st;
  if (cache->schedule != OKQ_SCHEDULE_WINDOW) return OKQ_ERR_UNSUPPORTED;   // the cross-check kernels know one schedule
  DecodeParams P = make_params(cache, layer, layer_count, q, sm_scale, signs, R, n_R, out);
  P.n_splits = num_splits > 0 ? num_splits : auto_splits(cache, layer_count);
  P.partials = static_cast<Partial*>(workspace);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  static thread_local unsigned long long attr_mask = 0;
  int attr_dev = 0;
  if (attr_needed(attr_mask, attr_dev)) {
    cudaError_t e = cudaFuncSetAttribute(k_decode_simt, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DecodeSmem));
    if (e != cudaSuccess) { set_last_cuda_error((int)e); return OKQ_ERR_CUDA; }
    attr_done(attr_mask, attr_dev);
  }
  dim3 grid(P.n_splits, cache->n_kv_heads, cache->batch * layer_count);
  if (g_ev_before) cudaEventRecord(g_ev_before, s);
  k_decode_simt<<<grid, 128, sizeof(DecodeSmem), s>>>(P);
  if (g_ev_after) cudaEventRecord(g_ev_after, s);
  k_combine<<<dim3(cache->n_kv_heads, cache->batch * layer_count), 128, 0, s>>>(P);
  return launch_status();
}

}  // extern "C"
