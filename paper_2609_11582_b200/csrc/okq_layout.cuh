// Physical layout of a window record and small helpers shared by the CUDA kernels.
//
// A record holds the 32 tokens of one window of one (layer, sequence, KV head).  The
// order of codes inside it follows the register fragments of mma.sync.m16n8k16, so that
// the decode kernel feeds the tensor cores with 16-byte shared-memory reads and a few
// mask/shift operations per 16 codes:
//
//  * Key codes are the B operand of  S^T[head][token] = W[head][channel] * C[channel][token].
//    Lane l = 4*g + t of a warp owns, for the tokens g, g+8, g+16, g+24 of the window, the
//    32 channels {16*kappa + 8*pair + 2*t + e}.  Those are two 32-bit words per token; in
//    a word, register r = 2*kappa + pair (r & 7 inside the word) sits at bit offset
//    8*((r>>2)&1) + 2*(r&3), its two channels e = 0/1 in the low/high 16 bits.
//  * Value codes are the A operand of  O^T[channel][head] = C[channel][token] * P[token][head].
//    Lane l = 4*g + t owns the channels {16*mu + 8*sh + g} (mu = 0..7, sh = 0/1) and the
//    tokens {16*kv + 8*pv + 2*t + e}: one word per mu, field index j = 2*kv + pv at bit
//    offset 8*sh + 2*j, token parity e in the low/high half.
//  * The 32 key norms (and value norms) are stored in the order norm_pos(i), which puts the
//    eight tokens whose scores a lane receives next to each other.
//  * (m, s) are stored as two planes of 128 fp16 in the order pi(c) that makes each
//    lane's 32 channels contiguous; the m plane is pre-multiplied by a power of four (meta_shift).
#pragma once
#include <cstdint>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

namespace okq {

constexpr int D = 128;
constexpr int W = 32;
constexpr int RECORD_BYTES = 2688;
constexpr int OFF_KM = 0;
constexpr int OFF_KS = 256;
constexpr int OFF_KNORM = 512;
constexpr int OFF_VNORM = 576;
constexpr int OFF_KCODE = 640;
constexpr int OFF_VCODE = 1664;

// position of channel c inside the m / s planes
__host__ __device__ inline int meta_pos(int c) {
  int kappa = c >> 4, slot = c & 15;
  int pair = slot >> 3, t = (slot & 7) >> 1, e = slot & 1;
  return t * 32 + kappa * 4 + pair * 2 + e;
}

// The m plane holds m_c * 4^j(c), j = (2*kappa + pair) & 3 (exact in fp16: |m| <= 1): 4^j is the position
// scale of the matching key-code field, which the decode kernel's query fragments are pre-divided by, so the
// stored value is the tensor-core operand of the bias sum as it is.  log4 of the factor, by channel / position:
__host__ __device__ inline int meta_shift(int c) { return (2 * (c >> 4) + ((c >> 3) & 1)) & 3; }
__host__ __device__ inline int meta_shift_pos(int p) { return (2 * ((p >> 2) & 7) + ((p >> 1) & 1)) & 3; }

// position of token i inside the key-norm / value-norm arrays: the four lanes of a quad each
// find the norms of "their" tokens {8*nu + 2*t + e} in 16 contiguous bytes
__host__ __device__ inline int norm_pos(int i) {
  int nu = i >> 3, t = (i & 7) >> 1, e = i & 1;
  return 8 * t + 2 * nu + e;
}

// The 64 16-byte pieces of a code block are stored in an order that lets both decode kernels read a staged copy
// without bank conflicts: the mma.sync kernel, whose lane l reads the "fragment" pieces l and 32 + l, and the tcgen05
// kernel, whose threads own one token (key codes) or one channel (value codes).  With the fragment piece index
// p = 32 a + 4 g + t (the order the mma.sync fragments above describe: piece p holds the words 4 p .. 4 p + 3) and
// g = 4 g2 + 2 g1 + g0, a piece sits at position 8 * row + column with
//   key codes:   row = 2 t + g2,  column = (t + 4 g0 + 2 g1 + a)  mod 8
//   value codes: row = 4 a + t,   column = (t + 4 g0 + 2 g1 + g2) mod 8
// Eight pieces read together always fall into the eight different 16-byte columns of the 128-byte bank line:
// the pieces (g0, t) of one quarter-warp of the mma.sync kernel; the pieces (a, g0, g1) that the 16 token-threads of
// a half-warp read for one t; the pieces g = 0..7 that a warp of channel-threads reads for one (a, t).
__host__ __device__ inline int kpiece_slot(int p) {
  const int t = p & 3, g = (p >> 2) & 7, a = p >> 5;
  return 8 * (2 * t + (g >> 2)) + ((t + 4 * (g & 1) + 2 * ((g >> 1) & 1) + a) & 7);
}
__host__ __device__ inline int vpiece_slot(int p) {
  const int t = p & 3, g = (p >> 2) & 7, a = p >> 5;
  return 8 * (4 * a + t) + ((t + 4 * (g & 1) + 2 * ((g >> 1) & 1) + (g >> 2)) & 7);
}
// stored position of fragment-order word w of the key / value code block
__host__ __device__ inline int kword_index(int w) { return 4 * kpiece_slot(w >> 2) + (w & 3); }
__host__ __device__ inline int vword_index(int w) { return 4 * vpiece_slot(w >> 2) + (w & 3); }

// key code of (token i in window, channel c): 32-bit word index in the key-code block and bit offset
__host__ __device__ inline void kcode_pos(int i, int c, int& word, int& bit) {
  int nu = i >> 3, g = i & 7;
  int kappa = c >> 4, slot = c & 15;
  int pair = slot >> 3, t = (slot & 7) >> 1, e = slot & 1;
  int r = 2 * kappa + pair;
  int ww = r >> 3, sh = (r >> 2) & 1, j = r & 3;
  word = kword_index((nu >> 1) * 128 + (4 * g + t) * 4 + (nu & 1) * 2 + ww);
  bit = 16 * e + 8 * sh + 2 * j;
}

// value code of (token i in window, channel c)
__host__ __device__ inline void vcode_pos(int i, int c, int& word, int& bit) {
  int mu = c >> 4, sh = (c >> 3) & 1, g = c & 7;
  int kv = i >> 4, pv = (i >> 3) & 1, t = (i & 7) >> 1, e = i & 1;
  int j = 2 * kv + pv;
  word = vword_index((mu >> 2) * 128 + (4 * g + t) * 4 + (mu & 3));
  bit = 16 * e + 8 * sh + 2 * j;
}

// A record = metadata (m, s) followed by a "body" [key norms 64 | value norms 64 | key codes 1024 |
// value codes 1024] whose layout is the same for both metadata formats.
//   Format 0 (fp16 (m, s)): 512 metadata bytes, records back to back (the offsets above).
//   Format 1 (MXFP4 (m, s), the paper's default): 136 metadata bytes [m nibbles 64 | s nibbles 64 |
//   m scales 4 | s scales 4], nibbles in meta_pos order (even position in the low nibble), one E8M0
//   scale per 32 consecutive channels.  2312 bytes per window; so that every body starts on a 16-byte
//   boundary, two consecutive windows share one 4624-byte block [meta 0 | meta 1 | body 0 | body 1].
constexpr int FMT_FP16 = 0, FMT_MXFP4 = 1;
constexpr int MX_META_BYTES = 136;
constexpr int META_BYTES_FP16 = 512;
constexpr int BODY_BYTES = 2176;
constexpr int B_KNORM = 0, B_VNORM = 64, B_KCODE = 128, B_VCODE = 1152;   // offsets inside a body
constexpr int MX_PAIR_BYTES = 2 * (MX_META_BYTES + BODY_BYTES);
static_assert(META_BYTES_FP16 + BODY_BYTES == RECORD_BYTES && OFF_KNORM == META_BYTES_FP16 + B_KNORM &&
              OFF_VCODE == META_BYTES_FP16 + B_VCODE, "record layout");

__host__ __device__ inline size_t mx_meta_off(size_t win) { return (win >> 1) * MX_PAIR_BYTES + (win & 1) * MX_META_BYTES; }
__host__ __device__ inline size_t mx_body_off(size_t win) {
  return (win >> 1) * MX_PAIR_BYTES + 2 * MX_META_BYTES + (win & 1) * BODY_BYTES;
}

constexpr int SCHED_WINDOW = 0, SCHED_CAPTION = 1;
constexpr int CAPTION_K_GROUP = 128;    // keys are packed every 128 tokens
constexpr int CAPTION_V_LAG = 128;      // values stay raw for 128 tokens
constexpr int CAPTION_V_SLOTS = CAPTION_V_LAG + W;   // ring of raw values: 128 .. 159 live tokens

struct CacheView {
  int n_layers, batch, n_kv_heads, n_q_heads, capacity;
  int fmt, sched;
  unsigned char* records;
  unsigned char* modality;
  __half* k_tail;
  __half* v_tail;
  int* seq_len;
  int* status;
  __host__ __device__ inline size_t n_windows() const { return (size_t)capacity / W; }
  // bytes of the records of one (layer, sequence, KV head)
  __host__ __device__ inline size_t unit_bytes() const {
    return fmt == FMT_MXFP4 ? ((n_windows() + 1) / 2) * (size_t)MX_PAIR_BYTES : n_windows() * (size_t)RECORD_BYTES;
  }
  __host__ __device__ inline unsigned char* unit(int layer, int b, int h) const {
    return records + (((size_t)layer * batch + b) * n_kv_heads + h) * unit_bytes();
  }
  __host__ __device__ inline unsigned char* meta(int layer, int b, int h, size_t win) const {
    return unit(layer, b, h) + (fmt == FMT_MXFP4 ? mx_meta_off(win) : win * RECORD_BYTES);
  }
  __host__ __device__ inline unsigned char* body(int layer, int b, int h, size_t win) const {
    return unit(layer, b, h) + (fmt == FMT_MXFP4 ? mx_body_off(win) : win * RECORD_BYTES + META_BYTES_FP16);
  }
  // raw-token slots per (layer, sequence, head), number of packed tokens of a sequence of n tokens, and
  // the slot of raw token t, for keys and for values
  __host__ __device__ inline int k_slots() const { return sched == SCHED_CAPTION ? CAPTION_K_GROUP : W; }
  __host__ __device__ inline int v_slots() const { return sched == SCHED_CAPTION ? CAPTION_V_SLOTS : W; }
  __host__ __device__ inline int k_packed(int n) const {
    return sched == SCHED_CAPTION ? n - n % CAPTION_K_GROUP : n - n % W;
  }
  __host__ __device__ inline int v_packed(int n) const {
    return sched == SCHED_CAPTION ? (n >= CAPTION_V_LAG ? (n - CAPTION_V_LAG) - (n - CAPTION_V_LAG) % W : 0) : n - n % W;
  }
  __host__ __device__ inline int k_slot(int t) const { return t % k_slots(); }
  __host__ __device__ inline int v_slot(int t) const { return t % v_slots(); }
  __host__ __device__ inline size_t k_tail_off(int layer, int b, int h) const {
    return (((size_t)layer * batch + b) * n_kv_heads + h) * (size_t)(k_slots() * D);
  }
  __host__ __device__ inline size_t v_tail_off(int layer, int b, int h) const {
    return (((size_t)layer * batch + b) * n_kv_heads + h) * (size_t)(v_slots() * D);
  }
};

// value codebook: Lloyd-Max levels of N(0, 1/128) and the decision threshold, fp32
constexpr float CB_INNER = 0x1.47d908p-5f;
constexpr float CB_OUTER = 0x1.116a3p-3f;
constexpr float CB_THRESH = 0x1.636072p-4f;
constexpr float RSQRT_D = 0x1.6a09e6p-4f;  // float(1/sqrt(128))

}  // namespace okq
