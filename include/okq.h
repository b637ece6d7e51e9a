/*
 * okq — 2-bit KV-cache quantisation and fused decode attention (OmniKVQuant hot path)
 * for NVIDIA B200 (sm_100a).  Plain C ABI: device pointers, sizes, a CUDA stream passed
 * as void*.  The library allocates no device memory, launches asynchronously on the given
 * stream and never aborts the process.  Its only state: the per-thread record of the last
 * CUDA error and of the profiling events (okq_profile_events), the process-wide choice of
 * the split-K kernel (okq_decode_select), and the fixed device array behind
 * okq_decode_attention_noalloc with the per-device cache of its address.
 *
 * Conventions
 *   - Every pointer inside okq_cache and every tensor argument is a DEVICE pointer owned
 *     by the caller, aligned to 16 bytes.  `const okq_cache*` itself and `strides` are
 *     HOST pointers, read before the call returns.
 *   - head_dim is 128, the key window is 32 tokens, codes are 2 bits; anything else is
 *     OKQ_ERR_UNSUPPORTED.  The GQA group n_q_heads / n_kv_heads must be an integer <= 8.
 *   - Modality ids: 0 text, 1 audio, 2 video (the paper's set {V, A, L}).
 *   - Errors that the host can see (null or misaligned pointers, bad shapes, workspace
 *     too small) are returned before anything is launched.  Errors only the device can
 *     see (a sequence would grow past `capacity`) set the cache's device status word to a
 *     non-zero okq_status and skip the write; the caller reads the word when it next
 *     synchronises.
 *
 * Storage format (fp16 metadata; 84 bytes per token per KV head = 2.625 bits/element,
 * the figure the paper's error-comparison table gives for FP16 (m, s) metadata):
 * the cache is an array of "window records", one per 32 consecutive tokens of one
 * (layer, sequence, KV head), OKQ_RECORD_BYTES each:
 *     [   0,  256)  key minimum m_gc, fp16 x 128 (channel order permuted, see below)
 *     [ 256,  512)  key step s_gc,    fp16 x 128 (same order)
 *     [ 512,  576)  key norms,   fp16 x 32 tokens
 *     [ 576,  640)  value norms, fp16 x 32 tokens
 *     [ 640, 1664)  key codes,   2 bits x 32 tokens x 128 channels
 *     [1664, 2688)  value codes, 2 bits x 32 tokens x 128 channels
 * With OKQ_META_MXFP4 (the paper's default metadata: 2.258 bits/element) the first 512 bytes shrink to
 * 136: m and s as 4-bit E2M1 elements with one power-of-two E8M0 scale per 32 consecutive channels
 * (converted as in the OCP microscaling format: block exponent floor(log2 max|x|) - 2, clamped to
 * [-23, 12] so that every decoded value is an fp16 number; elements rounded to the nearest grid value,
 * ties to even, saturating at 6 * 2^k), OKQ_RECORD_BYTES_MX = 2312 bytes per record, 72.25 per token per
 * KV head.  A key coordinate outside [m', m' + 3 s'] takes the end code.
 * Codes are computed against the decoded pair, exactly as with fp16 metadata.
 * Inside a record the channel / token order is the one the decode kernel's tensor-core
 * fragments want; okq_cache_export / okq_cache_import convert to and from the canonical
 * arrays (token-major codes with channel c of a token in byte c/4 at bits 2*(c%4);
 * metadata as [window][channel][m, s]).
 */
#ifndef OKQ_H
#define OKQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define OKQ_HEAD_DIM 128
#define OKQ_WINDOW 32
#define OKQ_RECORD_BYTES 2688    /* window record with fp16 (m, s) metadata */
#define OKQ_RECORD_BYTES_MX 2312 /* window record with MXFP4 (m, s) metadata */
#define OKQ_META_FP16 0
#define OKQ_META_MXFP4 1
#define OKQ_MAX_GROUP 8
#define OKQ_NOALLOC_SCRATCH_BYTES (64u << 20) /* fixed scratch of okq_decode_attention_noalloc */

typedef enum {
  OKQ_OK = 0,
  OKQ_ERR_INVALID_ARG = 1, /* null pointer, negative size, layer range out of bounds, ... */
  OKQ_ERR_UNSUPPORTED = 2, /* head_dim != 128, window != 32, GQA group > 8 or not integral */
  OKQ_ERR_ALIGNMENT = 3,   /* a device pointer is not 16-byte aligned */
  OKQ_ERR_CAPACITY = 4,    /* a sequence would exceed `capacity` (also the device status value) */
  OKQ_ERR_WORKSPACE = 5,   /* decode workspace smaller than okq_decode_workspace_bytes() */
  OKQ_ERR_CUDA = 6,        /* a CUDA runtime call failed; see okq_last_cuda_error() */
  OKQ_ERR_TIMEOUT = 7      /* device status value: a bounded device-side wait (an mbarrier of the tensor-core
                              pipelines) gave up; the kernel returned by itself, its results are invalid */
} okq_status;

/* Static, NUL-terminated description of a status value. */
const char* okq_status_string(okq_status s);
/* cudaError_t value behind the calling thread's most recent OKQ_ERR_CUDA (0 if none). */
int okq_last_cuda_error(void);

/* A 2-bit KV cache.  Plain data filled in by the caller. */
typedef struct okq_cache {
  int32_t n_layers, batch, n_kv_heads, n_q_heads;
  int32_t head_dim;  /* 128 */
  int32_t window;    /* 32 */
  int32_t capacity;  /* max tokens per sequence, multiple of 32 */
  int32_t meta_format; /* OKQ_META_FP16 (0) or OKQ_META_MXFP4 (1): how the key (m, s) pairs are stored */
  int32_t schedule;    /* OKQ_SCHEDULE_WINDOW (0) or OKQ_SCHEDULE_CAPTION (1): when raw tokens are packed, see below */
  int32_t reserved;    /* 0 */
  void* records;     /* [n_layers][batch][n_kv_heads][capacity/32][record bytes of the format]; 16-byte aligned */
  uint8_t* modality; /* [batch][capacity], shared by all layers and heads */
  void* k_tail;      /* [n_layers][batch][n_kv_heads][32 | 128][128] fp16: raw keys not packed yet (token t in slot t mod 32 | 128) */
  void* v_tail;      /* [n_layers][batch][n_kv_heads][32 | 160][128] fp16: raw values not packed yet (slot t mod 32 | 160) */
  int32_t* seq_len;  /* [n_layers][batch] tokens held; how many of them are packed follows from the schedule */
  int32_t* status;   /* [1] sticky first device-side error, 0 = none */
} okq_cache;

/*
 * Streaming schedules (the paper's "Implementation details").  With n tokens in a sequence:
 *   OKQ_SCHEDULE_WINDOW   keys and values are packed as soon as a 32-token window is complete: the first
 *                         32 * floor(n / 32) tokens of both are packed, at most 31 are raw fp16.
 *   OKQ_SCHEDULE_CAPTION  the paper's captioning schedule: keys are packed every 128 tokens, in four groups of
 *                         32 (the first 128 * floor(n / 128) keys are packed, at most 127 are raw), values stay
 *                         behind a sliding window of 128 raw fp16 tokens (the first 32 * floor((n - 128) / 32)
 *                         values are packed once n >= 128, 128 to 159 are raw).  A window's packed content is the
 *                         same under both schedules; only which recent tokens are still fp16 differs.
 *                         okq_decode_attention_simt returns OKQ_ERR_UNSUPPORTED for such a cache.
 */
#define OKQ_SCHEDULE_WINDOW 0
#define OKQ_SCHEDULE_CAPTION 1

/* Byte sizes of the six device buffers of a cache with the given shape fields (pointers
 * are ignored), in the order records, modality, k_tail, v_tail, seq_len, status.
 * Returns OKQ_OK or the shape error. */
okq_status okq_cache_sizes(const okq_cache* shape, size_t out_bytes[6]);

/* Bytes of scratch okq_decode_attention needs for `layer_count` layers with `num_splits`
 * (0 = let the library choose, the same choice the call makes).  0 on a shape error. */
size_t okq_decode_workspace_bytes(const okq_cache* cache, int32_t layer_count, int32_t num_splits);

/*
 * Key quantiser (paper Eq. 2 followed by Eq. 4): for every (sequence, KV head) of `layer`
 * quantise tokens [0, n_tokens) of k_fp16.  Per token: fp16 norm, z = H k/norm with
 * H = Had_128 diag(signs)/sqrt(128); per 32-token window and channel: m = min z,
 * s = (max - m)/3 as fp16, code = clamp(rint((z - m)/s), 0, 3).  The trailing
 * n_tokens % 32 tokens are copied raw to k_tail.  Sets seq_len[layer][*] = n_tokens.
 *   k_fp16   device, fp16, element (b, h, i, c) at k_fp16[b*strides[0] + h*strides[1] + i*strides[2] + c]
 *   strides  host, in elements; each a multiple of 8 so rows stay 16-byte aligned
 *   signs    device, float[128], each +1 or -1
 * Errors: OKQ_ERR_INVALID_ARG (n_tokens < 0, layer out of range, null), OKQ_ERR_CAPACITY
 * (n_tokens > capacity), OKQ_ERR_ALIGNMENT, OKQ_ERR_CUDA.
 */
okq_status okq_quantize_keys(const okq_cache* cache, int32_t layer, const void* k_fp16,
                             const int64_t strides[3], int32_t n_tokens, const float* signs,
                             void* stream);

/*
 * Value quantiser (paper Eq. 6 then Eq. 3): per token fp16 norm, z = R_m v/norm with the
 * matrix of the token's modality m, code = index of the nearest of the four fixed
 * Gaussian codebook levels.  Also stores `modality` into the cache and copies the
 * trailing n_tokens % 32 tokens raw to v_tail.  Sets seq_len[layer][*] = n_tokens.
 *   modality device, uint8 [batch][n_tokens]
 *   R        device, float [n_R][3][128][128] row-major, z = R[.][m] u; n_R is 1 (shared
 *            by the KV heads) or n_kv_heads
 * The rotation is evaluated as one fused-multiply-add chain per output coordinate over
 * the input index in ascending order, which makes the codes reproducible bit for bit.
 */
okq_status okq_quantize_values(const okq_cache* cache, int32_t layer, const void* v_fp16,
                               const int64_t strides[3], int32_t n_tokens, const uint8_t* modality,
                               const float* R, int32_t n_R, void* stream);

/*
 * Bulk (prefill) form of okq_quantize_values with the rotation z = R_m v on the tensor cores
 * (Eq. 6 as a dense [tokens x 128] x [128 x 128] product per modality; tcgen05.mma with R split
 * into two fp16 matrices and fp32 accumulation in tensor memory).  Same arguments, same stored
 * norms and the same stored codes, bit for bit: a coordinate that the tensor-core product leaves
 * within 2^-18 of a codebook threshold is recomputed with the fused-multiply-add chain of
 * okq_quantize_values before its code is taken.  If the tensor-core pipeline does not answer within a
 * bounded wait the device status word becomes OKQ_ERR_TIMEOUT and the remaining tiles are
 * skipped.
 */
okq_status okq_quantize_values_bulk(const okq_cache* cache, int32_t layer, const void* v_fp16,
                                    const int64_t strides[3], int32_t n_tokens,
                                    const uint8_t* modality, const float* R, int32_t n_R,
                                    void* stream);

/*
 * Testing aid for the bounded waits of okq_quantize_values_bulk (the paper has no counterpart): the same launch with
 * the first 128-token tile never delivered to the tensor-core pipeline and every wait limited to `limit_clocks` SM
 * clocks (a few milliseconds' worth is enough).  Every role's wait for that tile runs out, the kernel returns by
 * itself, the device status word becomes OKQ_ERR_TIMEOUT and the layer's value records are left incomplete: quantise
 * the layer again before using it.  Nothing faults and the context stays usable.
 */
okq_status okq_debug_bulk_timeout(const okq_cache* cache, int32_t layer, const void* v_fp16,
                                  const int64_t strides[3], int32_t n_tokens, const uint8_t* modality,
                                  const float* R, int32_t n_R, int64_t limit_clocks, void* stream);

/*
 * Streaming append (the paper's protocol keeps recent tokens in fp16 before they are
 * quantised): add one token per sequence to layers [layer, layer+layer_count).  The token
 * goes raw into the tail; when the tail reaches 32 tokens they are quantised as one window
 * exactly as the bulk calls would and the tail empties.  seq_len advances by one.
 *   k_new, v_new   device fp16 [layer_count][batch][n_kv_heads][128]
 *   modality_new   device uint8 [batch]
 *   signs          device float [layer_count][128]
 *   R              device float [layer_count][n_R][3][128][128]
 * A sequence already at `capacity` is left unchanged and the device status word becomes
 * OKQ_ERR_CAPACITY.  One kernel launch; while it runs, the top byte of the touched seq_len
 * entries holds a transient count (it is clear again when the kernel ends), which limits
 * the call to capacity < 2^24 and n_kv_heads <= 127 (OKQ_ERR_UNSUPPORTED otherwise).
 */
okq_status okq_append(const okq_cache* cache, int32_t layer, int32_t layer_count, const void* k_new,
                      const void* v_new, const uint8_t* modality_new, const float* signs,
                      const float* R, int32_t n_R, void* stream);

/*
 * Fused decode attention over the packed cache (paper Eq. 1 evaluated in the order the
 * paper describes for its kernel: the query is rotated once per head, scores are taken
 * against the codes in the rotated space, the softmax-weighted codebook levels are summed
 * per modality and R_m^T is applied once per head after aggregation).  One query token per
 * sequence, all cached tokens visible (packed windows and the raw tail), no mask.
 *   q          device fp16 [layer_count][batch][n_q_heads][128]
 *   sm_scale   softmax scale, normally 1/sqrt(128)
 *   signs, R   as for okq_append
 *   workspace  device scratch of at least okq_decode_workspace_bytes(cache, layer_count, num_splits)
 *   num_splits 0 = one persistent CTA per SM, each owning an equal slice of the flattened
 *              (layer, sequence, head, window) axis; n > 0 = n CTAs per (sequence, KV head)
 *              on average (at most 1024 in total)
 *   out        device float [layer_count][batch][n_q_heads][128]
 * A sequence with seq_len 0 yields zeros.
 */
okq_status okq_decode_attention(const okq_cache* cache, int32_t layer, int32_t layer_count,
                                const void* q, float sm_scale, const float* signs, const float* R,
                                int32_t n_R, void* workspace, size_t workspace_bytes,
                                int32_t num_splits, float* out, void* stream);

/*
 * okq_decode_attention for callers that have no scratch buffer to give and no way to get
 * one: code running where cudaMalloc is off limits (inside a serving loop whose memory was
 * carved up at start-up, under a caching allocator that must not be bypassed, in a plugin
 * that is only handed its inputs and outputs).  The paper has no counterpart; this is the
 * same kernel pair with its split-K partials kept in a fixed OKQ_NOALLOC_SCRATCH_BYTES
 * (64 MiB) array that is part of the library's device image, so every GPU that loads the
 * library carries those 64 MiB until the process exits.  The call allocates nothing: no
 * cudaMalloc, no cudaFree, no allocating library routine.
 *
 *   - Arguments are those of okq_decode_attention without workspace / workspace_bytes.
 *   - Limit: the tensor-core path's scratch of the largest launch (this is not okq_decode_workspace_bytes(),
 *     which also covers okq_decode_attention_simt and can be larger when num_splits is given), i.e.
 *     (layer_count * batch * n_kv_heads + number of CTAs) * 12736 bytes of per-CTA partials plus
 *     (layer_count * batch * n_kv_heads + 8 * number of CTAs) * 12832 bytes of per-warp-pair pieces,
 *     must fit in the scratch: about 1950 (sequence, KV head) pairs per launch with the automatic grid;
 *     anything larger returns OKQ_ERR_WORKSPACE and launches nothing (use
 *     okq_decode_attention with your own buffer).
 *   - The first call on each device looks up the scratch's device address (with that device
 *     current) and remembers it; make that first call outside any stream capture.
 *   - Every call on a device shares the one array.  Nothing in it has to be cleared: each
 *     launch overwrites the partials it later reads.  Two calls that overlap on the GPU
 *     (different streams, or different host threads) race on it and give wrong results;
 *     calls on one stream are ordered and safe.
 */
okq_status okq_decode_attention_noalloc(const okq_cache* cache, int32_t layer, int32_t layer_count,
                                        const void* q, float sm_scale, const float* signs,
                                        const float* R, int32_t n_R, int32_t num_splits, float* out,
                                        void* stream);

/*
 * The same computation on CUDA cores only (fp32 multiply-adds, dot products reduced with
 * warp shuffles): the straightforward form of the paper's kernel, kept as an independent
 * cross-check of the tensor-core path and as the measured arithmetic-bound baseline.
 * Arguments, workspace size and errors as for okq_decode_attention; num_splits is the
 * number of CTAs per (sequence, KV head).
 */
okq_status okq_decode_attention_simt(const okq_cache* cache, int32_t layer, int32_t layer_count,
                                     const void* q, float sm_scale, const float* signs,
                                     const float* R, int32_t n_R, void* workspace,
                                     size_t workspace_bytes, int32_t num_splits, float* out,
                                     void* stream);

/*
 * Profiling aid (the paper has no counterpart): until cleared with two nulls, every
 * okq_decode_attention call made by the calling thread records `before` on its stream
 * just ahead of the split-K kernel and `after` just behind it (ahead of the combine
 * kernel), so a benchmark can time the dominant kernel alone.  Both are cudaEvent_t
 * handles passed as void*, owned by the caller.
 */
void okq_profile_events(void* before, void* after);

/*
 * Choice of the split-K kernel behind okq_decode_attention (the paper has no counterpart; for cross-checks and
 * timing comparisons).  1 (default): the mma.sync warp-pair kernel; 0: the tcgen05 kernel with the unpacked codes
 * in tensor memory (fp16 metadata only; a cache with MXFP4 metadata always takes the warp-pair kernel).  Both fill
 * the same partial records for the same combine kernel.  Process-wide; not to be changed while a decode call is
 * being issued on another thread.  Returns the previous value; a value other than 0 or 1 changes nothing.
 */
int32_t okq_decode_select(int32_t impl);

/*
 * Canonical view of one layer (checkpointing and parity checks; the paper has no
 * counterpart, the arrays are simply Eq. 2-4 and Eq. 6 outputs in natural order).
 * All windows up to capacity are converted, whatever seq_len says.
 *   k_codes, v_codes  device uint8 [batch][n_kv_heads][capacity][32]
 *   k_norm, v_norm    device fp16  [batch][n_kv_heads][capacity]
 *   k_meta            device fp16  [batch][n_kv_heads][capacity/32][128][2]  (m, s)
 */
okq_status okq_cache_export(const okq_cache* cache, int32_t layer, uint8_t* k_codes, void* k_norm,
                            void* k_meta, uint8_t* v_codes, void* v_norm, void* stream);
okq_status okq_cache_import(const okq_cache* cache, int32_t layer, const uint8_t* k_codes,
                            const void* k_norm, const void* k_meta, const uint8_t* v_codes,
                            const void* v_norm, void* stream);
/*
 * With OKQ_META_MXFP4, okq_cache_export writes the DECODED (m, s) pairs into k_meta and
 * okq_cache_import returns OKQ_ERR_UNSUPPORTED (fp16 pairs need not lie on the MX grid).
 * okq_cache_export_mx (OKQ_META_MXFP4 caches only, else OKQ_ERR_UNSUPPORTED) also writes the
 * stored metadata bytes in natural channel order:
 *   k_mx   device uint8 [batch][n_kv_heads][capacity/32][136]:
 *          [0, 64) m elements, channel c in byte c/2 (even c in the low nibble; bit 3 = sign,
 *          bits 0-2 index {0, .5, 1, 1.5, 2, 3, 4, 6}); [64, 128) s elements likewise;
 *          [128, 132) m block exponents k + 127 for channels [32 j, 32 j + 32); [132, 136) s exponents.
 */
okq_status okq_cache_export_mx(const okq_cache* cache, int32_t layer, uint8_t* k_codes, void* k_norm,
                               void* k_meta, uint8_t* k_mx, uint8_t* v_codes, void* v_norm, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* OKQ_H */
