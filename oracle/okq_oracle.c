/*
 * CPU oracle for the OmniKVQuant hot path.  TEST INFRASTRUCTURE ONLY: it is called by
 * the tests, by the smoke check and by the benchmark's CPU-baseline leg, never by the
 * product path.  It shares no code with the CUDA library.
 *
 * What it computes, and where the paper defines it:
 *   - key quantiser:   norm split + randomised Hadamard rotation (Eq. 2), then per
 *                      32-token window and coordinate the minimum m_gc and scale s_gc
 *                      (Eq. 4), codes on four uniform levels m + s*code;
 *   - value quantiser: norm split, per-modality rotation z = R_m u (Eq. 6), nearest of
 *                      the four fixed Gaussian codebook levels (Eq. 3);
 *   - attention:       softmax(q K^T / sqrt(d)) V (Eq. 1) over the dequantised cache,
 *                      written twice: as the plain definition, and in the order the
 *                      paper's kernel uses (query rotated once per head, Sec. "Temporal
 *                      range adaptation"; inverse value rotation after aggregation,
 *                      Sec. "Modality-aware value rotation").
 *
 * The quantisers are the algorithm step by step in fp32 with every operation rounded
 * on its own (compile with -ffp-contract=off); attention is in double.
 *
 * Readings of points the paper leaves open (all listed in the design notes):
 *   - H = (1/sqrt(128)) * Had_128 * diag(D), Sylvester order, D a +-1 vector;
 *   - the per-vector norm is stored as fp16 for keys and values; the rotated vector is
 *     normalised by the *stored* norm;
 *   - (m, s) are stored as fp16, s = (max - m)/3 is the step; codes are computed
 *     against the stored (decoded) pair, round-half-even, clamped to [0,3];
 *   - the value codebook is the 4-level Lloyd-Max quantiser of N(0, 1/128); a value
 *     exactly on a threshold takes the lower code;
 *   - tokens beyond the last full window stay raw fp16 (the "tail").
 *
 * Parity unpinned: nothing in this file.  (The paper's Recon. MSE / Attn. KL / Output
 * MSE table needs the paper's activations and is not reproduced anywhere.)
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define OKQ_D 128
#define OKQ_W 32

/* ---------------------------------------------------------------- fp16 <-> fp32 */

float okqo_half_to_float(uint16_t h) {
  uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
  uint32_t e = (h >> 10) & 0x1f, m = h & 0x3ff, x;
  if (e == 0) {
    if (m == 0) {
      x = sign;
    } else { /* subnormal: m * 2^-24 */
      float f = (float)m * 0x1p-24f;
      memcpy(&x, &f, 4);
      x |= sign;
    }
  } else if (e == 31) {
    x = sign | 0x7f800000u | (m << 13);
  } else {
    x = sign | ((e + 112) << 23) | (m << 13);
  }
  float f;
  memcpy(&f, &x, 4);
  return f;
}

/* round-to-nearest-even; values >= 65520 become infinity */
uint16_t okqo_float_to_half(float f) {
  uint32_t x;
  memcpy(&x, &f, 4);
  uint16_t sign = (uint16_t)((x >> 16) & 0x8000u);
  uint32_t a = x & 0x7fffffffu;
  if (a >= 0x7f800000u) return (uint16_t)(sign | 0x7c00u | (a > 0x7f800000u ? 0x200u : 0u));
  if (a >= 0x477ff000u) return (uint16_t)(sign | 0x7c00u);
  if (a < 0x38800000u) { /* below 2^-14: half subnormal, unit 2^-24 */
    if (a <= 0x33000000u) return sign; /* <= 2^-25 rounds to zero (tie goes to even) */
    uint32_t e = a >> 23, m = (a & 0x7fffffu) | 0x800000u;
    uint32_t shift = 126 - e; /* 14..24 */
    uint32_t r = m >> shift, rem = m & ((1u << shift) - 1), half = 1u << (shift - 1);
    if (rem > half || (rem == half && (r & 1))) r++;
    return (uint16_t)(sign | r);
  }
  uint32_t e = (a >> 23) - 112, m = a & 0x7fffffu;
  uint32_t r = (e << 10) | (m >> 13), rem = m & 0x1fffu;
  if (rem > 0x1000u || (rem == 0x1000u && (r & 1))) r++;
  return (uint16_t)(sign | r);
}

/* ---------------------------------------------------------------- constants */

/* float(1/sqrt(128)) */
static const float RSQRT_D = 0x1.6a09e6p-4f;
/* Lloyd-Max levels of N(0,1): +-0.4527800346, +-1.5104176085, threshold 0.9815988216,
 * each divided by sqrt(128) and rounded to fp32 (Eq. 3: codebook built from the
 * Gaussian reference N(0, 1/d)). */
static const float CB_A = 0x1.47d908p-5f;   /* 0.040020481 */
static const float CB_B = 0x1.116a3p-3f;    /* 0.133503318 */
static const float CB_T = 0x1.636072p-4f;   /* 0.086761899 */

void okqo_codebook(float levels[4], float* threshold) {
  levels[0] = -CB_B; levels[1] = -CB_A; levels[2] = CB_A; levels[3] = CB_B;
  *threshold = CB_T;
}

/* Storage cost of one token of one KV head with fp16 (m, s) metadata: 32 B key codes +
 * 2 B key norm + 2*2*128/32 = 16 B metadata, 32 B value codes + 2 B value norm.
 * 84 B * 8 / 256 elements = 2.625 bits per element (Table "error comparison",
 * Bits/elem. column, FP16-metadata row). */
int okqo_bytes_per_token_head(void) { return (OKQ_D * 2) / 8 + 2 + (2 * 2 * OKQ_D) / OKQ_W + (OKQ_D * 2) / 8 + 2; }

/* ---------------------------------------------------------------- building blocks */

/* Unnormalised Sylvester-ordered fast Walsh-Hadamard transform, in place, fp32.
 * Stages h = 1, 2, ..., 64; pair (j, j+h) with (j & h) == 0 becomes (a+b, a-b). */
void okqo_fwht128(float* y) {
  for (int h = 1; h < OKQ_D; h <<= 1)
    for (int j = 0; j < OKQ_D; j++)
      if ((j & h) == 0) {
        float a = y[j], b = y[j + h];
        y[j] = a + b;
        y[j + h] = a - b;
      }
}

/* ||x||_2 in fp32 with the adjacent-pair summation tree, rounded to fp16 (clamped to
 * the largest finite half).  Returns the stored half. */
static uint16_t norm_half(const float* x) {
  float t[OKQ_D];
  for (int c = 0; c < OKQ_D; c++) t[c] = x[c] * x[c];
  for (int n = OKQ_D / 2; n >= 1; n >>= 1)
    for (int c = 0; c < n; c++) t[c] = t[2 * c] + t[2 * c + 1];
  float nrm = sqrtf(t[0]);
  if (nrm > 65504.0f) nrm = 65504.0f;
  return okqo_float_to_half(nrm);
}

/* Eq. 2 for one key: stored norm and z = H (k / norm), H = Had * diag(D) / sqrt(128). */
void okqo_key_rotate(const uint16_t* k, const float* signs, uint16_t* norm_out, float* z) {
  float x[OKQ_D], y[OKQ_D];
  for (int c = 0; c < OKQ_D; c++) x[c] = okqo_half_to_float(k[c]);
  uint16_t nh = norm_half(x);
  *norm_out = nh;
  if ((nh & 0x7fff) == 0) {
    for (int c = 0; c < OKQ_D; c++) z[c] = 0.0f;
    return;
  }
  for (int c = 0; c < OKQ_D; c++) y[c] = signs[c] * x[c];
  okqo_fwht128(y);
  float cinv = RSQRT_D / okqo_half_to_float(nh);
  for (int c = 0; c < OKQ_D; c++) z[c] = y[c] * cinv;
}

/* Eq. 4 for one window: z[32][128] -> meta[128][2] = (m, s) as fp16, codes[32][32]
 * (byte c/4 of a token holds channel c at bits 2*(c%4)). */
void okqo_window_quantize(const float* z, uint16_t* meta, uint8_t* codes) {
  memset(codes, 0, OKQ_W * OKQ_D / 4);
  for (int c = 0; c < OKQ_D; c++) {
    float mn = z[c], mx = z[c];
    for (int i = 1; i < OKQ_W; i++) {
      float v = z[i * OKQ_D + c];
      if (v < mn) mn = v;
      if (v > mx) mx = v;
    }
    uint16_t mh = okqo_float_to_half(mn);
    float mf = okqo_half_to_float(mh);
    float range = mx - mf;
    if (range < 0.0f) range = 0.0f; /* m rounded up past a (near-)constant channel */
    uint16_t sh = okqo_float_to_half(range / 3.0f);
    float sf = okqo_half_to_float(sh);
    meta[2 * c] = mh;
    meta[2 * c + 1] = sh;
    if (!(sf > 0.0f)) continue; /* constant channel (or mx below the rounded m): codes 0 */
    float r = 1.0f / sf;
    for (int i = 0; i < OKQ_W; i++) {
      float q = rintf((z[i * OKQ_D + c] - mf) * r); /* round-half-even in the default mode */
      int code = q < 0.0f ? 0 : (q > 3.0f ? 3 : (int)q);
      codes[i * (OKQ_D / 4) + c / 4] |= (uint8_t)(code << (2 * (c % 4)));
    }
  }
}

/* ---------------------------------------------------------------- MXFP4 (m, s) metadata
 *
 * The paper's default metadata format ("MXFP4 metadata by default", Implementation details):
 * m and s are each stored as 4-bit E2M1 elements sharing one 8-bit power-of-two scale (E8M0) per
 * block of 32.  The paper does not say how blocks are formed or how values are rounded; the
 * reading taken here (listed in the design notes):
 *   - a block is 32 consecutive channels of one window, separately for m and for s;
 *   - conversion as in the OCP microscaling format: the block exponent is floor(log2 max|x|) - 2 (2^2 is
 *     the largest power of two of E2M1), clamped to [-23, 12] so that every decoded value grid * 2^k is
 *     exactly an fp16 number; elements are rounded to the nearest value of the grid
 *     {0, .5, 1, 1.5, 2, 3, 4, 6} * 2^k (ties to the even mantissa), magnitudes beyond 6 * 2^k saturate;
 *     a value below m' or above m' + 3 s' takes the end code (codes are clamped to [0, 3] anyway).  With
 *     this conversion the key error grows by a few percent over fp16 metadata, the order of the paper's
 *     error table (0.1833 against 0.1495); rounding m down and s up so that nothing clips doubles it;
 *   - codes are computed against the decoded pair (m', s') exactly as in the fp16 format.
 * 2 * (128 * 4 + 4 * 8) bits per 32-token window = 136 B instead of 512 B: 72.25 B per token per
 * KV head = 2.258 bits per element, the figure the paper prints for its default.
 */
static const float MX_GRID[8] = {0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f};

int okqo_bytes_per_window_mx(void) { return OKQ_W * ((OKQ_D * 2) / 8 + 2 + (OKQ_D * 2) / 8 + 2) + 2 * (OKQ_D / 2 + OKQ_D / 32); }

/* block exponent floor(log2 amax) - 2, clamped to [-23, 12] (-23 for an all-zero block) */
int okqo_mx_scale_exp(float amax) {
  int k = -23;
  if (amax > 0.0f) {
    int e;
    (void)frexpf(amax, &e); /* amax = f * 2^e, f in [0.5, 1): floor(log2 amax) = e - 1 */
    k = e - 1 - 2;          /* the element format's largest power of two is 2^2 */
  }
  if (k < -23) k = -23;
  if (k > 12) k = 12;
  return k;
}

/* nibble (sign << 3 | grid index) of x on the grid * 2^k: nearest grid value, ties to the value with an even
 * mantissa bit (grid indices 0, 2, 4, 6), magnitudes beyond 6 * 2^k saturate to 6 * 2^k */
uint8_t okqo_mx_encode(float x, int k) {
  float q = ldexpf(x, -k); /* exact */
  float a = fabsf(q);
  int best = 0;
  for (int i = 1; i < 8; i++) {
    float d0 = fabsf(a - MX_GRID[best]), d1 = fabsf(a - MX_GRID[i]);
    if (d1 < d0 || (d1 == d0 && (i & 1) == 0)) best = i;
  }
  if (best == 0) return 0; /* no negative zero */
  return (uint8_t)(((q < 0.0f) ? 8 : 0) | best);
}

float okqo_mx_decode(uint8_t nib, int k) {
  float g = MX_GRID[nib & 7];
  return ldexpf((nib & 8) ? -g : g, k);
}

/* Eq. 4 with MXFP4 metadata for one window.  mx: 136 bytes = m nibbles [64] (channel c in byte c/2,
 * low nibble for even c), s nibbles [64], m scales [4] (k + 127), s scales [4].  meta_dec: the decoded
 * (m', s') as fp16 [128][2], the same array the fp16 format stores.  codes as okqo_window_quantize. */
void okqo_window_quantize_mx(const float* z, uint8_t* mx, uint16_t* meta_dec, uint8_t* codes) {
  float mn[OKQ_D], mxv[OKQ_D], md[OKQ_D], sr[OKQ_D], sd[OKQ_D];
  memset(codes, 0, OKQ_W * OKQ_D / 4);
  memset(mx, 0, 136);
  for (int c = 0; c < OKQ_D; c++) {
    mn[c] = mxv[c] = z[c];
    for (int i = 1; i < OKQ_W; i++) {
      float v = z[i * OKQ_D + c];
      if (v < mn[c]) mn[c] = v;
      if (v > mxv[c]) mxv[c] = v;
    }
  }
  for (int b = 0; b < OKQ_D / 32; b++) { /* minima: scale from the block's largest magnitude */
    float amax = 0.0f;
    for (int c = 32 * b; c < 32 * b + 32; c++) if (fabsf(mn[c]) > amax) amax = fabsf(mn[c]);
    int k = okqo_mx_scale_exp(amax);
    mx[128 + b] = (uint8_t)(k + 127);
    for (int c = 32 * b; c < 32 * b + 32; c++) {
      uint8_t nib = okqo_mx_encode(mn[c], k);
      mx[c / 2] |= (uint8_t)(nib << (4 * (c & 1)));
      md[c] = okqo_mx_decode(nib, k);
      float range = mxv[c] - md[c];
      if (range < 0.0f) range = 0.0f;
      sr[c] = range / 3.0f;
    }
  }
  for (int b = 0; b < OKQ_D / 32; b++) { /* steps */
    float amax = 0.0f;
    for (int c = 32 * b; c < 32 * b + 32; c++) if (sr[c] > amax) amax = sr[c];
    int k = okqo_mx_scale_exp(amax);
    mx[132 + b] = (uint8_t)(k + 127);
    for (int c = 32 * b; c < 32 * b + 32; c++) {
      uint8_t nib = okqo_mx_encode(sr[c], k);
      mx[64 + c / 2] |= (uint8_t)(nib << (4 * (c & 1)));
      sd[c] = okqo_mx_decode(nib, k);
    }
  }
  for (int c = 0; c < OKQ_D; c++) {
    meta_dec[2 * c] = okqo_float_to_half(md[c]);     /* exact: every decoded value is an fp16 number */
    meta_dec[2 * c + 1] = okqo_float_to_half(sd[c]);
    if (!(sd[c] > 0.0f)) continue;
    float r = 1.0f / sd[c];
    for (int i = 0; i < OKQ_W; i++) {
      float q = rintf((z[i * OKQ_D + c] - md[c]) * r);
      int code = q < 0.0f ? 0 : (q > 3.0f ? 3 : (int)q);
      codes[i * (OKQ_D / 4) + c / 4] |= (uint8_t)(code << (2 * (c % 4)));
    }
  }
}

/* Key quantiser with MXFP4 metadata over one (layer, sequence, KV head).  mx: [n_windows][136]. */
int64_t okqo_quantize_keys_mx(const uint16_t* k, int64_t n_tokens, const float* signs, uint8_t* codes,
                              uint16_t* norms, uint16_t* meta_dec, uint8_t* mx) {
  int64_t n_win = n_tokens / OKQ_W;
  float* z = (float*)malloc(sizeof(float) * OKQ_W * OKQ_D);
  for (int64_t g = 0; g < n_win; g++) {
    for (int i = 0; i < OKQ_W; i++) {
      int64_t tok = g * OKQ_W + i;
      okqo_key_rotate(k + tok * OKQ_D, signs, norms + tok, z + i * OKQ_D);
    }
    okqo_window_quantize_mx(z, mx + g * 136, meta_dec + g * OKQ_D * 2, codes + g * OKQ_W * (OKQ_D / 4));
  }
  free(z);
  return n_win * OKQ_W;
}

/* Key quantiser over one (layer, sequence, KV head): tokens [0, n_tokens); the first
 * floor(n/32)*32 are packed.  Returns the number of packed tokens. */
int64_t okqo_quantize_keys(const uint16_t* k, int64_t n_tokens, const float* signs,
                           uint8_t* codes, uint16_t* norms, uint16_t* meta) {
  int64_t n_win = n_tokens / OKQ_W;
  float* z = (float*)malloc(sizeof(float) * OKQ_W * OKQ_D);
  for (int64_t g = 0; g < n_win; g++) {
    for (int i = 0; i < OKQ_W; i++) {
      int64_t tok = g * OKQ_W + i;
      okqo_key_rotate(k + tok * OKQ_D, signs, norms + tok, z + i * OKQ_D);
    }
    okqo_window_quantize(z, meta + g * OKQ_D * 2, codes + g * OKQ_W * (OKQ_D / 4));
  }
  free(z);
  return n_win * OKQ_W;
}

/* Eq. 6 for one value: stored norm and z = R_m (v / norm).  Each output coordinate is
 * one chain of fused multiply-adds over k = 0..127 in ascending order. */
void okqo_value_rotate(const uint16_t* v, const float* Rm, uint16_t* norm_out, float* z) {
  float x[OKQ_D];
  for (int c = 0; c < OKQ_D; c++) x[c] = okqo_half_to_float(v[c]);
  uint16_t nh = norm_half(x);
  *norm_out = nh;
  if ((nh & 0x7fff) == 0) {
    for (int c = 0; c < OKQ_D; c++) z[c] = 0.0f;
    return;
  }
  float inv = 1.0f / okqo_half_to_float(nh);
  for (int c = 0; c < OKQ_D; c++) {
    float t = 0.0f;
    for (int kk = 0; kk < OKQ_D; kk++) t = fmaf(Rm[c * OKQ_D + kk], x[kk], t);
    z[c] = t * inv;
  }
}

/* Eq. 3: index of the nearest codebook level, written as three threshold compares. */
static inline int value_code(float z) { return (z > -CB_T) + (z > 0.0f) + (z > CB_T); }

/* Value quantiser over one (layer, sequence, KV head).  R is [3][128][128] row-major,
 * modality[i] in {0 text, 1 audio, 2 video} selects the matrix. */
int64_t okqo_quantize_values(const uint16_t* v, int64_t n_tokens, const uint8_t* modality,
                             const float* R, uint8_t* codes, uint16_t* norms) {
  int64_t n_packed = (n_tokens / OKQ_W) * OKQ_W;
  float z[OKQ_D];
  for (int64_t i = 0; i < n_packed; i++) {
    okqo_value_rotate(v + i * OKQ_D, R + (size_t)modality[i] * OKQ_D * OKQ_D, norms + i, z);
    uint8_t* out = codes + i * (OKQ_D / 4);
    memset(out, 0, OKQ_D / 4);
    for (int c = 0; c < OKQ_D; c++) out[c / 4] |= (uint8_t)(value_code(z[c]) << (2 * (c % 4)));
  }
  return n_packed;
}

/* ---------------------------------------------------------------- dequantisation (double) */

static inline int get_code(const uint8_t* codes, int c) { return (codes[c / 4] >> (2 * (c % 4))) & 3; }

static int popcount7(int x) { int n = 0; for (; x; x >>= 1) n += x & 1; return n; }

/* H[r][c] = (-1)^popcount(r & c) * D_c / sqrt(128), as an explicit matrix in double. */
static void build_H(const float* signs, double* H) {
  double rs = 1.0 / sqrt((double)OKQ_D);
  for (int r = 0; r < OKQ_D; r++)
    for (int c = 0; c < OKQ_D; c++)
      H[r * OKQ_D + c] = ((popcount7(r & c) & 1) ? -1.0 : 1.0) * (double)signs[c] * rs;
}

/* k_hat = norm * H^T z_hat, z_hat_c = m_c + s_c * code_c  (Eq. 3 reconstruction with
 * Eq. 4 inverted).  meta points at the token's window; H is the explicit matrix. */
static void dequant_key_H(const uint8_t* codes, uint16_t norm, const uint16_t* meta,
                          const double* H, double* k_hat) {
  double zh[OKQ_D];
  for (int c = 0; c < OKQ_D; c++)
    zh[c] = (double)okqo_half_to_float(meta[2 * c]) +
            (double)okqo_half_to_float(meta[2 * c + 1]) * (double)get_code(codes, c);
  double n = (double)okqo_half_to_float(norm);
  for (int c = 0; c < OKQ_D; c++) {
    double acc = 0.0;
    for (int r = 0; r < OKQ_D; r++) acc += H[r * OKQ_D + c] * zh[r];
    k_hat[c] = n * acc;
  }
}

void okqo_dequant_key(const uint8_t* codes, uint16_t norm, const uint16_t* meta,
                      const float* signs, double* k_hat) {
  double* H = (double*)malloc(sizeof(double) * OKQ_D * OKQ_D);
  build_H(signs, H);
  dequant_key_H(codes, norm, meta, H, k_hat);
  free(H);
}

/* v_hat = norm * R_m^T cb[code]  (Eq. 6). */
void okqo_dequant_value(const uint8_t* codes, uint16_t norm, const float* Rm, double* v_hat) {
  const double cb[4] = {-(double)CB_B, -(double)CB_A, (double)CB_A, (double)CB_B};
  double n = (double)okqo_half_to_float(norm);
  for (int c = 0; c < OKQ_D; c++) {
    double acc = 0.0;
    for (int r = 0; r < OKQ_D; r++) acc += (double)Rm[r * OKQ_D + c] * cb[get_code(codes, r)];
    v_hat[c] = n * acc;
  }
}

/* ---------------------------------------------------------------- attention (double) */

/*
 * One (sequence, KV head) unit.  q: [G][128] fp16.  Packed tokens [0, n_packed) come from
 * the canonical arrays, tail tokens [n_packed, n_packed + n_tail) are raw fp16.
 * modality: [n_packed + n_tail] (only the packed part is used).  out: [G][128] double.
 * No mask: the decode query attends to every cached token.
 *
 * Definition path (Eq. 1): dequantise every token, then softmax attention.
 */
void okqo_attention_def(const uint16_t* q, int G, int64_t n_packed, const uint8_t* k_codes,
                        const uint16_t* k_norm, const uint16_t* k_meta, const uint8_t* v_codes,
                        const uint16_t* v_norm, const uint8_t* modality, int n_tail,
                        const uint16_t* k_tail, const uint16_t* v_tail, const float* signs,
                        const float* R, double sm_scale, double* out) {
  int64_t n = n_packed + n_tail;
  double* kh = (double*)malloc(sizeof(double) * (size_t)n * OKQ_D);
  double* vh = (double*)malloc(sizeof(double) * (size_t)n * OKQ_D);
  double* s = (double*)malloc(sizeof(double) * (size_t)n);
  double* H = (double*)malloc(sizeof(double) * OKQ_D * OKQ_D);
  build_H(signs, H);
  for (int64_t i = 0; i < n_packed; i++) {
    dequant_key_H(k_codes + i * 32, k_norm[i], k_meta + (i / OKQ_W) * OKQ_D * 2, H, kh + i * OKQ_D);
    okqo_dequant_value(v_codes + i * 32, v_norm[i], R + (size_t)modality[i] * OKQ_D * OKQ_D, vh + i * OKQ_D);
  }
  for (int i = 0; i < n_tail; i++)
    for (int c = 0; c < OKQ_D; c++) {
      kh[(n_packed + i) * OKQ_D + c] = (double)okqo_half_to_float(k_tail[i * OKQ_D + c]);
      vh[(n_packed + i) * OKQ_D + c] = (double)okqo_half_to_float(v_tail[i * OKQ_D + c]);
    }
  for (int h = 0; h < G; h++) {
    double qd[OKQ_D], mx = -INFINITY, sum = 0.0;
    for (int c = 0; c < OKQ_D; c++) qd[c] = (double)okqo_half_to_float(q[h * OKQ_D + c]);
    for (int64_t i = 0; i < n; i++) {
      double a = 0.0;
      for (int c = 0; c < OKQ_D; c++) a += qd[c] * kh[i * OKQ_D + c];
      s[i] = a * sm_scale;
      if (s[i] > mx) mx = s[i];
    }
    double* o = out + h * OKQ_D;
    for (int c = 0; c < OKQ_D; c++) o[c] = 0.0;
    for (int64_t i = 0; i < n; i++) {
      double p = exp(s[i] - mx);
      sum += p;
      for (int c = 0; c < OKQ_D; c++) o[c] += p * vh[i * OKQ_D + c];
    }
    for (int c = 0; c < OKQ_D; c++) o[c] = n > 0 ? o[c] / sum : 0.0;
  }
  free(kh); free(vh); free(s); free(H);
}

/*
 * Rotated-space path: the order the paper describes for its kernel.  The query is
 * rotated once per head (q' = H q), so that q . k_hat = norm * (q' . z_hat); the values
 * are accumulated as codebook levels in each modality's rotated basis and R_m^T is applied
 * once per head after the softmax-weighted sum.  By linearity this equals the definition
 * path; the tests require agreement to 1e-10.
 */
void okqo_attention_rot(const uint16_t* q, int G, int64_t n_packed, const uint8_t* k_codes,
                        const uint16_t* k_norm, const uint16_t* k_meta, const uint8_t* v_codes,
                        const uint16_t* v_norm, const uint8_t* modality, int n_tail,
                        const uint16_t* k_tail, const uint16_t* v_tail, const float* signs,
                        const float* R, double sm_scale, double* out) {
  const double cb[4] = {-(double)CB_B, -(double)CB_A, (double)CB_A, (double)CB_B};
  int64_t n = n_packed + n_tail;
  double* s = (double*)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
  for (int h = 0; h < G; h++) {
    double qd[OKQ_D], qr[OKQ_D];
    for (int c = 0; c < OKQ_D; c++) {
      qd[c] = (double)okqo_half_to_float(q[h * OKQ_D + c]);
      qr[c] = qd[c] * (double)signs[c];
    }
    /* q' = H q: Hadamard butterflies in double, then 1/sqrt(128) */
    for (int hh = 1; hh < OKQ_D; hh <<= 1)
      for (int j = 0; j < OKQ_D; j++)
        if ((j & hh) == 0) {
          double a = qr[j], b = qr[j + hh];
          qr[j] = a + b;
          qr[j + hh] = a - b;
        }
    for (int c = 0; c < OKQ_D; c++) qr[c] /= sqrt((double)OKQ_D);
    double mx = -INFINITY;
    for (int64_t g = 0; g < n_packed / OKQ_W; g++) {
      const uint16_t* meta = k_meta + g * OKQ_D * 2;
      double w[OKQ_D], bias = 0.0;
      for (int c = 0; c < OKQ_D; c++) {
        w[c] = qr[c] * (double)okqo_half_to_float(meta[2 * c + 1]);
        bias += qr[c] * (double)okqo_half_to_float(meta[2 * c]);
      }
      for (int i = 0; i < OKQ_W; i++) {
        int64_t tok = g * OKQ_W + i;
        double a = bias;
        for (int c = 0; c < OKQ_D; c++) a += w[c] * (double)get_code(k_codes + tok * 32, c);
        s[tok] = a * (double)okqo_half_to_float(k_norm[tok]) * sm_scale;
        if (s[tok] > mx) mx = s[tok];
      }
    }
    for (int i = 0; i < n_tail; i++) {
      double a = 0.0;
      for (int c = 0; c < OKQ_D; c++) a += qd[c] * (double)okqo_half_to_float(k_tail[i * OKQ_D + c]);
      s[n_packed + i] = a * sm_scale;
      if (s[n_packed + i] > mx) mx = s[n_packed + i];
    }
    double acc[3][OKQ_D], raw[OKQ_D], sum = 0.0;
    memset(acc, 0, sizeof(acc));
    memset(raw, 0, sizeof(raw));
    for (int64_t i = 0; i < n_packed; i++) {
      double p = exp(s[i] - mx);
      sum += p;
      double pv = p * (double)okqo_half_to_float(v_norm[i]);
      double* a = acc[modality[i]];
      for (int c = 0; c < OKQ_D; c++) a[c] += pv * cb[get_code(v_codes + i * 32, c)];
    }
    for (int i = 0; i < n_tail; i++) {
      double p = exp(s[n_packed + i] - mx);
      sum += p;
      for (int c = 0; c < OKQ_D; c++) raw[c] += p * (double)okqo_half_to_float(v_tail[i * OKQ_D + c]);
    }
    double* o = out + h * OKQ_D;
    for (int c = 0; c < OKQ_D; c++) {
      double t = raw[c];
      for (int m = 0; m < 3; m++) {
        const float* Rm = R + (size_t)m * OKQ_D * OKQ_D;
        double u = 0.0;
        for (int r = 0; r < OKQ_D; r++) u += (double)Rm[r * OKQ_D + c] * acc[m][r];
        t += u;
      }
      o[c] = n > 0 ? t / sum : 0.0;
    }
  }
  free(s);
}

/*
 * Many units at once (used for timing the oracle on the host cores and for larger parity
 * samples).  Unit u has its canonical arrays at index u of the [U][...] inputs, its
 * modality row at modality + unit_seq[u] * mod_stride, and its rotation set at
 * R + unit_rot[u] * 3*128*128 and signs at signs + unit_rot[u] * 128.
 * path: 0 = definition, 1 = rotated space.  Returns the number of threads used.
 */
int okqo_attention_batch(int path, int U, const uint16_t* q, int G, int64_t n_packed,
                         const uint8_t* k_codes, const uint16_t* k_norm, const uint16_t* k_meta,
                         const uint8_t* v_codes, const uint16_t* v_norm, const uint8_t* modality,
                         int64_t mod_stride, const int32_t* unit_seq, const int32_t* unit_rot,
                         int n_tail, const uint16_t* k_tail, const uint16_t* v_tail,
                         const float* signs, const float* R, double sm_scale, double* out) {
  int threads = 1;
#ifdef _OPENMP
  threads = omp_get_max_threads();
#pragma omp parallel for schedule(dynamic, 1)
#endif
  for (int u = 0; u < U; u++) {
    void (*fn)(const uint16_t*, int, int64_t, const uint8_t*, const uint16_t*, const uint16_t*,
               const uint8_t*, const uint16_t*, const uint8_t*, int, const uint16_t*,
               const uint16_t*, const float*, const float*, double, double*) =
        path == 0 ? okqo_attention_def : okqo_attention_rot;
    fn(q + (size_t)u * G * OKQ_D, G, n_packed, k_codes + (size_t)u * n_packed * 32,
       k_norm + (size_t)u * n_packed, k_meta + (size_t)u * (n_packed / OKQ_W) * OKQ_D * 2,
       v_codes + (size_t)u * n_packed * 32, v_norm + (size_t)u * n_packed,
       modality + (size_t)unit_seq[u] * mod_stride, n_tail,
       k_tail + (size_t)u * OKQ_W * OKQ_D, v_tail + (size_t)u * OKQ_W * OKQ_D,
       signs + (size_t)unit_rot[u] * OKQ_D, R + (size_t)unit_rot[u] * 3 * OKQ_D * OKQ_D, sm_scale,
       out + (size_t)u * G * OKQ_D);
  }
  return threads;
}

/* Quantise many units (keys and values) in parallel; inputs [U][n_tokens][128] fp16. */
int okqo_quantize_batch_fmt(int U, const uint16_t* k, const uint16_t* v, int64_t n_tokens,
                            const uint8_t* modality, int64_t mod_stride, const int32_t* unit_seq,
                            const int32_t* unit_rot, const float* signs, const float* R,
                            uint8_t* k_codes, uint16_t* k_norm, uint16_t* k_meta, uint8_t* v_codes,
                            uint16_t* v_norm, int meta_format, uint8_t* k_mx);

int okqo_quantize_batch(int U, const uint16_t* k, const uint16_t* v, int64_t n_tokens,
                        const uint8_t* modality, int64_t mod_stride, const int32_t* unit_seq,
                        const int32_t* unit_rot, const float* signs, const float* R,
                        uint8_t* k_codes, uint16_t* k_norm, uint16_t* k_meta, uint8_t* v_codes,
                        uint16_t* v_norm) {
  return okqo_quantize_batch_fmt(U, k, v, n_tokens, modality, mod_stride, unit_seq, unit_rot, signs, R, k_codes,
                                 k_norm, k_meta, v_codes, v_norm, 0, NULL);
}

/* meta_format 0: fp16 (m, s); 1: MXFP4 (k_meta receives the decoded pairs, k_mx [U][n_win][136] the stored bytes) */
int okqo_quantize_batch_fmt(int U, const uint16_t* k, const uint16_t* v, int64_t n_tokens,
                            const uint8_t* modality, int64_t mod_stride, const int32_t* unit_seq,
                            const int32_t* unit_rot, const float* signs, const float* R,
                            uint8_t* k_codes, uint16_t* k_norm, uint16_t* k_meta, uint8_t* v_codes,
                            uint16_t* v_norm, int meta_format, uint8_t* k_mx) {
  int threads = 1;
  int64_t np = (n_tokens / OKQ_W) * OKQ_W;
#ifdef _OPENMP
  threads = omp_get_max_threads();
#pragma omp parallel for schedule(dynamic, 1)
#endif
  for (int u = 0; u < U; u++) {
    if (meta_format == 1)
      okqo_quantize_keys_mx(k + (size_t)u * n_tokens * OKQ_D, n_tokens, signs + (size_t)unit_rot[u] * OKQ_D,
                            k_codes + (size_t)u * np * 32, k_norm + (size_t)u * np,
                            k_meta + (size_t)u * (np / OKQ_W) * OKQ_D * 2, k_mx + (size_t)u * (np / OKQ_W) * 136);
    else
      okqo_quantize_keys(k + (size_t)u * n_tokens * OKQ_D, n_tokens, signs + (size_t)unit_rot[u] * OKQ_D,
                         k_codes + (size_t)u * np * 32, k_norm + (size_t)u * np,
                         k_meta + (size_t)u * (np / OKQ_W) * OKQ_D * 2);
    okqo_quantize_values(v + (size_t)u * n_tokens * OKQ_D, n_tokens,
                         modality + (size_t)unit_seq[u] * mod_stride,
                         R + (size_t)unit_rot[u] * 3 * OKQ_D * OKQ_D, v_codes + (size_t)u * np * 32,
                         v_norm + (size_t)u * np);
  }
  return threads;
}
