/*
 * okq_ladder — OmniKVQuant at 3 and 4 bits per code (the K3V3 / K4V4 columns of the paper's
 * bit-width ladder table), next to the 2-bit hot path of okq.h.  Plain C ABI, device pointers,
 * a CUDA stream passed as void*; nothing is allocated.
 *
 * The arithmetic is the 2-bit path's with the number of levels changed:
 *   keys   (Eq. 2, Eq. 4)  fp16 norm, randomised Hadamard rotation, per 32-token window and channel a
 *          minimum m and a step s = (max - m') / (2^b - 1), both stored as fp16, code =
 *          clamp(rint((z - m') / s'), 0, 2^b - 1) against the stored pair;
 *   values (Eq. 6, Eq. 3)  fp16 norm, z = R_m v / norm as one fused-multiply-add chain per coordinate,
 *          code = index of the nearest of the 2^b Lloyd-Max levels of N(0, 1/128);
 *   decode (Eq. 1)         scores in the rotated space against one rotated query per head, online softmax,
 *          value sums in each modality's rotated basis, R_m^T once per head.
 * This is a plain CUDA-core implementation over a canonical cache (no fragment-order records, no tensor
 * cores: with eight or sixteen non-uniform value levels the bit-plane identity of the 2-bit decode kernel
 * does not apply, the levels come from a table); it exists for parity with the ladder and is not tuned.
 *
 * Cache layout (all buffers caller-owned, 16-byte aligned; n_tokens must be a multiple of 32: no raw tail):
 *   k_codes, v_codes  uint8 [batch][n_kv_heads][capacity][16 * bits]: per token a little-endian bit stream,
 *                     channel c in bits [bits * c, bits * c + bits)
 *   k_norm, v_norm    fp16  [batch][n_kv_heads][capacity]
 *   k_meta            fp16  [batch][n_kv_heads][capacity / 32][128][2] = (m, s)
 *   modality          uint8 [batch][capacity] (0 text, 1 audio, 2 video; larger ids count as text)
 */
#ifndef OKQ_LADDER_H
#define OKQ_LADDER_H

#include "okq.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct okq_ladder_cache {
  int32_t batch, n_kv_heads, n_q_heads, capacity;
  int32_t bits;      /* 2, 3 or 4 */
  int32_t reserved;  /* 0 */
  void* k_codes;
  void* k_norm;
  void* k_meta;
  void* v_codes;
  void* v_norm;
  uint8_t* modality;
} okq_ladder_cache;

/* The 2^bits levels and 2^bits - 1 decision thresholds (fp32, ascending) of the value codebook the kernels hold:
 * the minimum-MSE quantiser of N(0, 1/128) (Eq. 3).  `levels` and `thresholds` are HOST arrays of 16 and 15 floats;
 * returns the number of levels, 0 for an unsupported width. */
int32_t okq_ladder_codebook(int32_t bits, float* levels, float* thresholds);

/* Eq. 2 and Eq. 4 at `cache->bits` bits.  k_fp16: device fp16 [batch][n_kv_heads][n_tokens][128] with element
 * strides {batch, head, token} (channels contiguous); signs: device float [128] of +-1. */
okq_status okq_ladder_quantize_keys(const okq_ladder_cache* cache, const void* k_fp16, const int64_t strides[3],
                                    int32_t n_tokens, const float* signs, void* stream);

/* Eq. 6 and Eq. 3 at `cache->bits` bits; also stores `modality` ([batch][n_tokens]) into the cache.
 * R: device float [n_R][3][128][128], n_R = 1 or n_kv_heads. */
okq_status okq_ladder_quantize_values(const okq_ladder_cache* cache, const void* v_fp16, const int64_t strides[3],
                                      int32_t n_tokens, const uint8_t* modality, const float* R, int32_t n_R,
                                      void* stream);

/* Eq. 1 over the first n_tokens tokens of every sequence.  q: device fp16 [batch][n_q_heads][128];
 * out: device float [batch][n_q_heads][128]; one thread block per (sequence, KV head). */
okq_status okq_ladder_decode_attention(const okq_ladder_cache* cache, int32_t n_tokens, const void* q,
                                       float sm_scale, const float* signs, const float* R, int32_t n_R,
                                       float* out, void* stream);

/* TurboQuant baseline codec (the paper's Preliminaries, Eq. 2 and Eq. 3), for the synthetic error comparison against
 * OmniKVQuant at equal code width: per vector an fp16 norm, the randomised Hadamard rotation and the nearest level
 * of the same fixed codebook; no window statistics and no modality rotation, the same for keys and values.
 * x_fp16: device fp16 [n_vectors][128] contiguous; codes: device uint8 [n_vectors][16 * bits] (bit stream as above);
 * norms: device fp16 [n_vectors].  n_vectors = 0 is a no-op. */
okq_status okq_turboquant_encode(const void* x_fp16, int64_t n_vectors, int32_t bits, const float* signs, uint8_t* codes,
                                 void* norms, void* stream);

/* x_hat = |x| H^T level[code] as device float [n_vectors][128]. */
okq_status okq_turboquant_decode(const uint8_t* codes, const void* norms, int64_t n_vectors, int32_t bits,
                                 const float* signs, float* x_hat, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* OKQ_LADDER_H */
