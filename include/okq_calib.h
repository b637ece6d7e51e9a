/*
 * okq_calib.h - offline calibration of the per-modality value rotations R_m (the paper's
 * "Modality-aware value rotation": Eq. 5 and R_m = H U_m^T), C ABI.
 *
 * The decode / quantise path in okq.h takes R_m as an input; these calls produce it from calibration
 * activations of one (layer, KV head):
 *     w_j = sum_i alpha[i, j]^2                    okq_calib_attention_weights   (Eq. 5, left)
 *     C_m = sum_{j in m} w_j v_j^T v_j             okq_calib_moments             (Eq. 5, right)
 *     U_m = eigenvectors of C_m,  R_m = H U_m^T    okq_calib_rotation
 * Readings where the paper is silent: alpha is the causal softmax attention of the calibration sequence
 * (causal = 0 gives the full softmax), summed over the query heads that share the KV head; v_j is the raw
 * value; eigenvectors are ordered by descending eigenvalue, each with its largest-magnitude component
 * positive; H = Had_128 diag(signs) / sqrt(128), the key path's randomised Hadamard matrix.
 *
 * Conventions as in okq.h: every pointer is a DEVICE pointer unless it says host, owned by the caller,
 * 16-byte aligned; calls are asynchronous on `stream` (a cudaStream_t passed as void*); argument errors are
 * returned before anything is launched.  head_dim is 128.
 */
#ifndef OKQ_CALIB_H
#define OKQ_CALIB_H

#include "okq.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Bytes of device workspace the calls below need for a calibration sequence of n tokens and a GQA group
 * of `group` query heads (the maximum over the three calls; 0 on bad arguments). */
size_t okq_calib_workspace_bytes(int32_t group, int32_t n);

/*
 * w_j = sum over the group's heads g and queries i of alpha[g, i, j]^2, alpha = softmax_j(q_i . k_j * sm_scale)
 * over j <= i (causal != 0) or over all j.
 *   q_fp16  fp16 [group][n][128], k_fp16  fp16 [n][128], w_out  float [n]
 * Scores on the tensor cores (fp16 products, fp32 accumulation), two passes over the keys (row maximum and
 * normaliser, then the squared weights); the sums over queries are taken in a fixed order.
 * Errors: OKQ_ERR_INVALID_ARG (null, n <= 0, group <= 0), OKQ_ERR_ALIGNMENT, OKQ_ERR_WORKSPACE.
 */
okq_status okq_calib_attention_weights(const void* q_fp16, const void* k_fp16, int32_t group, int32_t n,
                                       float sm_scale, int32_t causal, void* workspace, size_t workspace_bytes,
                                       float* w_out, void* stream);

/*
 * C_m = sum_{j: modality_j = m} w_j v_j^T v_j for m = 0 (text), 1 (audio), 2 (video); ids > 2 count as text.
 *   v_fp16  fp16 [n][128], w  float [n] (>= 0), modality  uint8 [n], C_out  float [3][128][128]
 * A weighted 128 x 128 x n contraction per modality on the tensor cores: the values are one operand as they
 * are, w_j v_j split into two fp16 terms the other (weights first scaled by a power of two so that the
 * largest is at most 1), fp32 accumulation, partial sums over token ranges added in a fixed order.
 */
okq_status okq_calib_moments(const void* v_fp16, const float* w, const uint8_t* modality, int32_t n,
                             void* workspace, size_t workspace_bytes, float* C_out, void* stream);

/*
 * Eigen-decomposition of one symmetric 128 x 128 matrix (cyclic Jacobi in fp64, one thread block) and
 * R = H U^T with the ordering and sign convention stated above.
 *   C  float [128][128] (symmetric; only read), signs  float [128] (+-1)
 *   R_out  float [128][128] (row = rotated coordinate), lambda_out  float [128] (descending)
 *   workspace: 128 KB of the workspace (fp64 eigenvector matrix).
 * The device status convention of okq.h does not apply: the iteration has a fixed sweep limit (30), which
 * a symmetric matrix does not reach; `sweeps_out` (device int32, may be null) receives the sweeps used.
 */
okq_status okq_calib_rotation(const float* C, const float* signs, void* workspace, size_t workspace_bytes,
                              float* R_out, float* lambda_out, int32_t* sweeps_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* OKQ_CALIB_H */
