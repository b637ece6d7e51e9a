// Types shared by the two decode implementations (CUDA-core and tensor-core).
#pragma once
#include "okq_common.cuh"

namespace okq {

constexpr int GP = OKQ_MAX_GROUP;   // padded GQA group
constexpr int NACC = 4;             // 3 modality accumulators + 1 raw (tail) accumulator
constexpr int MAX_ENTRIES = 1024;   // (layer, sequence) pairs one launch can cover

// CUDA-core kernel: one per (sequence, head, split)
struct Partial {
  float m[GP];
  float l[GP];
  float acc[NACC][GP][D];
};

// tensor-core kernel: one per (CTA, (sequence, head)) overlap; accumulators stay in
// mma fragment order [modality][register][lane]
struct PartialF {
  float m[GP];          // running maximum per head (log2 domain)
  float l[GP];          // sum of exp2(score - m)
  float Sp[3][32];      // per modality: sum of p * vnorm, four lane-partials per head
  float frag[3][32][32];
};

// tensor-core kernel: what one warp pair accumulated over its part of one (sequence, head); the CTA
// merges its pairs' pieces into the PartialF records at the end of the launch
constexpr int MMA_PAIRS = 8;        // warp pairs per CTA
constexpr int PAIR_REGS = 33;       // 32 accumulator registers + the running weight sum, per lane
struct PairPartial {
  float frag[3][PAIR_REGS][32];   // [modality][register][lane]
  float sm[3][GP];                // running maximum the modality's accumulators refer to (-inf: none)
  float wm[GP], wl[GP];           // running maximum and sum of exp2(score - maximum) per head
};

struct DecodeParams {
  CacheView cv;
  int layer0, layer_count, n_splits, group;
  const __half* q;     // [layer_count][batch][n_q_heads][128]
  const float* signs;  // [layer_count][128]
  const float* R;      // [layer_count][n_R][3][128][128]
  int n_R;
  float sm_scale;
  Partial* partials;   // CUDA-core path: [layer_count*batch*n_kv_heads][n_splits]
  PartialF* partials_f;  // tensor-core path: [n_units + n_cta]
  PairPartial* pair_parts;  // tensor-core path: [n_units + 8 * n_cta]
  float* out;          // [layer_count][batch][n_q_heads][128]
};

// prefix[e] = number of windows (all KV heads) of the (layer, sequence) entries before e,
// entries ordered layer-major; returns the total.  Called by every thread of the block.
__device__ inline int block_prefix(const CacheView& cv, int layer0, int n_entries, int* prefix) {
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    const int chunk = (n_entries + 31) / 32;
    const int e0 = min(n_entries, lane * chunk), e1 = min(n_entries, e0 + chunk);
    int sum = 0;
    for (int e = e0; e < e1; e++) sum += (cv.v_packed(cv.seq_len[(size_t)layer0 * cv.batch + e]) / W) * cv.n_kv_heads;
    int incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int v = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += v;
    }
    int run = incl - sum;
    for (int e = e0; e < e1; e++) {
      prefix[e] = run;
      run += (cv.v_packed(cv.seq_len[(size_t)layer0 * cv.batch + e]) / W) * cv.n_kv_heads;
    }
    if (lane == 31) prefix[n_entries] = incl;
  }
  __syncthreads();
  return prefix[n_entries];
}

// tcgen05 split-K kernel (fp16 metadata): fills partials_f exactly where launch_decode_mma's own split kernel would
okq_status launch_decode_tc(const DecodeParams& P, int n_cta, cudaStream_t s);
// which split-K kernel launch_decode_mma uses: 0 = the tcgen05 kernel (fp16 metadata), 1 = the mma.sync warp-pair kernel
extern int g_decode_impl;

// launches the tensor-core split kernel (bracketed by the optional events) and its combine kernel
okq_status launch_decode_mma(const DecodeParams& P, int n_cta, cudaStream_t s, cudaEvent_t before, cudaEvent_t after);

}  // namespace okq
