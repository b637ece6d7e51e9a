// Fused decode attention, tensor-core version (the production path of okq_decode_attention).
//
// The GQA group's scores and value sums are dense contractions over the cached tokens
//     S^T[head][token]   = W[head][channel] * C_k[channel][token]        (per 32-token window)
//     O^T[channel][head] = C_v[channel][token] * P[token][head]
// and run on mma.sync.m16n8k16 with the 2-bit codes unpacked in registers:
//   * a code field masked out of its 32-bit word *is* an fp16 subnormal (code * 4^j * 2^-24,
//     j the field's position), so unpacking is one AND per two codes; the factor 4^j is folded
//     into the other operand (the query weights, or the softmax numerators);
//   * W = q'_c * s_gc is split into an fp16 high and low part, which fill the 16 rows of the
//     m16 tile (8 heads x {hi, lo}), so the split costs no extra tensor work; the per-window
//     bias sum_c q'_c m_gc goes through the same pipe against a constant operand;
//   * the value codebook {-b,-a,a,b} is affine in the two code bits:
//     cb[c] = (b-a)*c + (3a-b)*bit1(c) - b, so two bit-plane products plus the running sum
//     of the weights reproduce it exactly.
// A CTA runs 8 warp pairs.  The "score" warp of a pair computes the scores and the online
// softmax (FlashAttention order) and hands the fp16 numerators to its "value" warp through
// shared memory; the value warp accumulates the codebook sums of the previous window meanwhile
// and streams the window records through a cp.async ring, two windows ahead of the score warp
// (with MXFP4 metadata it also expands them into the fp16 planes).  One named barrier per pair
// and iteration keeps the two in step (no spin-waits anywhere).  Windows whose tokens all belong
// to the modality the registers hold take a straight-line path.  Values accumulate in the rotated
// basis of the current modality, in registers for at most 32 windows at a time; each modality's
// running sums live in shared memory.
// The grid is persistent: CTA i owns an equal slice of the flattened (layer, sequence, head,
// window) axis, each of its pairs an eighth of that slice, which the pair walks without any
// block-wide step; at the end the block merges its pairs' pieces into one partial per
// (sequence, head) it touched.  The combine kernel merges the partials, adds the raw fp16 tail
// tokens, applies R_m^T once per head and normalises.
#include <type_traits>
#include "okq_common.cuh"
#include "okq_device.cuh"
#include "okq_decode_shared.cuh"
#include "okq_decode_frag.cuh"

namespace okq {

namespace {

constexpr int NPAIR = MMA_PAIRS;                // warp pairs per CTA
constexpr int NTHREADS = NPAIR * 64;
constexpr int NSTAGE = 4;                       // record ring per pair
constexpr int PREFETCH = 2;                     // windows in flight ahead of the score warp
// staged window image: the fp16-metadata record, the window's 32 modality bytes and, with MXFP4
// metadata, the 136 stored metadata bytes (decoded into the first 512 bytes by the score warp)
constexpr int STAGE_MOD = RECORD_BYTES, STAGE_MX = RECORD_BYTES + 32;
template <int FMT> constexpr int stage_bytes() { return FMT == FMT_MXFP4 ? STAGE_MX + 144 : STAGE_MX; }
constexpr float RESCALE_LOG2 = 3.0f;            // numerators stay below 2^3 * 2^6 * vnorm in fp16
constexpr int FLUSH = 32;                       // windows a value warp accumulates in registers at most
constexpr int SPILL_STRIDE = 36;                // floats per lane in the deposited sums: 33 used, 144-byte rows

struct Handoff {
  uint4 pb[32];         // per lane: numerators p * vnorm * 2^6 / 4^nu of its 8 tokens, fp16 pairs (nu = x,y,z,w)
  float m[GP];          // running maximum per head after this window (log2 domain)
  float alpha[GP];      // factor the value accumulators must be multiplied by before this window
  int rescale;          // non-zero if any alpha != 1
  int pad[15];
};

template <int FMT>
struct MmaSmem {
  __align__(16) unsigned char stage[NPAIR][NSTAGE][stage_bytes<FMT>()];
  __align__(16) Handoff hand[NPAIR][2];
  __align__(16) float spill[NPAIR][3][32][SPILL_STRIDE];   // [pair][modality][lane]: the lane's 33 sums, 128-bit rows
  float spill_m[NPAIR][3][GP];
  float fin_w[NPAIR][2][GP];   // running maximum and weight sum a pair's score warp ended its last range with
  int prefix[MAX_ENTRIES + 1];
};

constexpr int MB_SEG = 32;                      // (sequence, head) units merged per batch at the end of the launch
struct MergeSmem {
  int pa[MB_SEG], pb[MB_SEG];                   // first and last warp pair that worked on the unit (pb < pa: none)
  int last_kept[MB_SEG];                        // whether pair pb's piece is in shared memory (all before it are)
  float meta[MB_SEG + NPAIR][5 * GP];           // per piece: sm[3][GP], wm[GP], wl[GP]; index = unit + pair - pa[0]
  float M[MB_SEG][GP];                          // merged running maximum
  float fac[MB_SEG + NPAIR][3][GP];             // per piece, modality and head: exp2(sm - M), 0 where the piece holds nothing
};

struct Segment {
  const unsigned char* rec0;   // first record of the (layer, sequence, head)
  const unsigned char* mod0;   // modality row of the sequence
  int w0, n_my;                // this pair's windows of that (layer, sequence, head): first window, count
  const __half* q;             // query rows of the KV head's group: [group][128]
  const float* signs;          // Hadamard signs of the layer
  PairPartial* piece;          // where the pair leaves what it accumulated ...
  bool keep;                   // ... unless this is the last unit of the pair's range: then it stays in shared memory
};

// Scores of one packed window against the group's queries, by one warp, from a staged image of the window's key
// part ((m, s) planes, key norms, key codes at their record offsets): the split-K kernel's score step.
// sc[nu][e] = log2-domain score of head g = lane >> 2 against token 8 nu + 2 (lane & 3) + e.
__device__ __forceinline__ void window_scores_mma(const unsigned char* st, const uint2 (&qreg)[16], float fsc, int lane,
                                                  float (&sc)[4][2]) {
  const int t = lane & 3;
  const uint4* mp = reinterpret_cast<const uint4*>(st + OFF_KM + 64 * t);
  const uint4* sp = reinterpret_cast<const uint4*>(st + OFF_KS + 64 * t);
  float dbA[4] = {0.f, 0.f, 0.f, 0.f}, dbB[4] = {0.f, 0.f, 0.f, 0.f};
  float d[4][4];
#pragma unroll
  for (int nu = 0; nu < 4; nu++)
#pragma unroll
    for (int i = 0; i < 4; i++) d[nu][i] = 0.f;
  const uint4 kc0 = *reinterpret_cast<const uint4*>(st + OFF_KCODE + 16 * kpiece_slot(lane));
  const uint4 kc1 = *reinterpret_cast<const uint4*>(st + OFF_KCODE + 16 * kpiece_slot(32 + lane));
  const uint32_t kw[4][2] = {{kc0.x, kc0.y}, {kc0.z, kc0.w}, {kc1.x, kc1.y}, {kc1.z, kc1.w}};
#pragma unroll
  for (int kq = 0; kq < 4; kq++) {
    const uint4 m4 = mp[kq], s4 = sp[kq];
#pragma unroll
    for (int half = 0; half < 2; half++) {
      const int kappa = 2 * kq + half;
      const uint2 q0 = qreg[2 * kappa], q1 = qreg[2 * kappa + 1];
      uint32_t a0, a1, a2, a3;
      if (half) mma16816(dbB, q0.x, q0.y, q1.x, q1.y, m4.z, m4.w);
      else mma16816(dbA, q0.x, q0.y, q1.x, q1.y, m4.x, m4.y);
      split_product(u2h(q0.x), u2h(q0.y), u2h(half ? s4.z : s4.x), a0, a1);
      split_product(u2h(q1.x), u2h(q1.y), u2h(half ? s4.w : s4.y), a2, a3);
      const int ww = kappa >> 2, sh = (kappa >> 1) & 1;
      const uint32_t mk0 = half ? 0x00300030u : 0x00030003u;
      const uint32_t mk1 = half ? 0x00c000c0u : 0x000c000cu;
#pragma unroll
      for (int nu = 0; nu < 4; nu++) {
        uint32_t src = sh ? (kw[nu][ww] >> 8) : kw[nu][ww];
        mma16816(d[nu], a0, a1, a2, a3, src & mk0, src & mk1);
      }
    }
  }
  const uint4 kn4 = *reinterpret_cast<const uint4*>(st + OFF_KNORM + 16 * t);
  const uint32_t knu[4] = {kn4.x, kn4.y, kn4.z, kn4.w};
  const float bias0 = ((dbA[0] + dbB[0]) + (dbA[2] + dbB[2])) * 0x1p-24f;   // the code sums carry 2^-24, the bias does not
#pragma unroll
  for (int nu = 0; nu < 4; nu++) {
    const float2 kn = __half22float2(u2h(knu[nu]));
    sc[nu][0] = ((d[nu][0] + d[nu][2]) + bias0) * (kn.x * fsc);
    sc[nu][1] = ((d[nu][1] + d[nu][3]) + bias0) * (kn.y * fsc);
  }
}

// ---------------------------------------------------------------- score warp
template <int FMT>
__device__ __forceinline__ void score_warp(MmaSmem<FMT>& sm, const Segment& sg, int G, float sm_scale, int pair,
                                           int lane) {
  const int g = lane >> 2, t = lane & 3;
  float run_m = -INFINITY, run_l = 0.f;

  uint2 qreg[16];
  float fsc;
  query_fragments(sg.q, sg.signs, G, sm_scale, lane, qreg, fsc);   // while the first windows are on their way
  pair_barrier(pair);   // the value warp has the first window in place

  for (int k = 0; k <= sg.n_my; k++) {
    if (k < sg.n_my) {
      // copied (and, with MXFP4 metadata, expanded into the fp16 planes) by the value warp, complete before the last barrier
      unsigned char* st = sm.stage[pair][k % NSTAGE];
      const uint4* mp = reinterpret_cast<const uint4*>(st + OFF_KM + 64 * t);
      const uint4* sp = reinterpret_cast<const uint4*>(st + OFF_KS + 64 * t);
      // bias sum_c q'_c m_c (two independent chains)
      // and scores sum_c q'_c s_c code_c, one k-step (16 channels) at a time
      float dbA[4] = {0.f, 0.f, 0.f, 0.f}, dbB[4] = {0.f, 0.f, 0.f, 0.f};
      float d[4][4];
#pragma unroll
      for (int nu = 0; nu < 4; nu++)
#pragma unroll
        for (int i = 0; i < 4; i++) d[nu][i] = 0.f;
      const uint4 kc0 = *reinterpret_cast<const uint4*>(st + OFF_KCODE + 16 * kpiece_slot(lane));
      const uint4 kc1 = *reinterpret_cast<const uint4*>(st + OFF_KCODE + 16 * kpiece_slot(32 + lane));
      const uint32_t kw[4][2] = {{kc0.x, kc0.y}, {kc0.z, kc0.w}, {kc1.x, kc1.y}, {kc1.z, kc1.w}};
#pragma unroll
      for (int kq = 0; kq < 4; kq++) {
        const uint4 m4 = mp[kq], s4 = sp[kq];
#pragma unroll
        for (int half = 0; half < 2; half++) {
          const int kappa = 2 * kq + half;
          const uint2 q0 = qreg[2 * kappa], q1 = qreg[2 * kappa + 1];
          uint32_t a0, a1, a2, a3;
          // bias: the stored m * 4^j is the B operand as it is (every column the same), the query fragments
          // (hi rows, lo rows) the A operand
          if (half) mma16816(dbB, q0.x, q0.y, q1.x, q1.y, m4.z, m4.w);
          else mma16816(dbA, q0.x, q0.y, q1.x, q1.y, m4.x, m4.y);
          split_product(u2h(q0.x), u2h(q0.y), u2h(half ? s4.z : s4.x), a0, a1);
          split_product(u2h(q1.x), u2h(q1.y), u2h(half ? s4.w : s4.y), a2, a3);
          const int ww = kappa >> 2, sh = (kappa >> 1) & 1;
          const uint32_t mk0 = half ? 0x00300030u : 0x00030003u;
          const uint32_t mk1 = half ? 0x00c000c0u : 0x000c000cu;
#pragma unroll
          for (int nu = 0; nu < 4; nu++) {
            uint32_t src = sh ? (kw[nu][ww] >> 8) : kw[nu][ww];
            mma16816(d[nu], a0, a1, a2, a3, src & mk0, src & mk1);
          }
        }
      }
      // online softmax (log2 domain); this lane: head g, tokens 8*nu + 2*t + e
      const uint4 kn4 = *reinterpret_cast<const uint4*>(st + OFF_KNORM + 16 * t);
      const uint4 vn4 = *reinterpret_cast<const uint4*>(st + OFF_VNORM + 16 * t);
      const uint32_t knu[4] = {kn4.x, kn4.y, kn4.z, kn4.w}, vnu[4] = {vn4.x, vn4.y, vn4.z, vn4.w};
      // the code sums carry 2^-24 (subnormal code operands), the bias sum does not
      const float bias0 = ((dbA[0] + dbB[0]) + (dbA[2] + dbB[2])) * 0x1p-24f, bias1 = bias0;
      // sc = score / fsc: the head's scale fsc > 0 (query scaling, 1/sqrt(d), log2 e) enters the exponent below in
      // one multiply-add and the maximum once
      float sc[4][2];
      float mx = -INFINITY;
#pragma unroll
      for (int nu = 0; nu < 4; nu++) {
        float2 kn = __half22float2(u2h(knu[nu]));
        sc[nu][0] = ((d[nu][0] + d[nu][2]) + bias0) * kn.x;
        sc[nu][1] = ((d[nu][1] + d[nu][3]) + bias1) * kn.y;
        mx = fmaxf(mx, fmaxf(sc[nu][0], sc[nu][1]));
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      mx *= fsc;
      // the reference maximum only moves when it is exceeded by more than 2^RESCALE_LOG2, so the
      // value accumulators are rescaled a few times per range instead of at every new maximum
      const float m_new = mx > run_m + RESCALE_LOG2 ? mx : run_m;
      const float alpha = ex2(run_m - m_new);  // 0 on the first window
      const int changed = __any_sync(0xffffffffu, m_new > run_m);
      run_l *= alpha;
      run_m = m_new;
      Handoff& ho = sm.hand[pair][k & 1];
      uint32_t pb[4];
#pragma unroll
      for (int nu = 0; nu < 4; nu++) {
        float2 vn = __half22float2(u2h(vnu[nu]));
        const float off = (float)(6 - 2 * nu) - run_m;
        const float cinv = (float)(1 << (2 * nu)) * (1.0f / 64.0f);
        float p0 = ex2(fmaf(sc[nu][0], fsc, off)), p1 = ex2(fmaf(sc[nu][1], fsc, off));
        run_l = fmaf(p0 + p1, cinv, run_l);
        pb[nu] = pack_sat(p0 * vn.x, p1 * vn.y);
      }
      ho.pb[lane] = make_uint4(pb[0], pb[1], pb[2], pb[3]);
      if (t == 0) { ho.m[g] = run_m; ho.alpha[g] = alpha; }
      if (lane == 0) ho.rescale = changed;
    }
    pair_barrier(pair);
  }
  run_l += __shfl_xor_sync(0xffffffffu, run_l, 1);
  run_l += __shfl_xor_sync(0xffffffffu, run_l, 2);
  if (t == 0) {
    if (sg.keep) { sm.fin_w[pair][0][g] = run_m; sm.fin_w[pair][1][g] = run_l; }
    else { sg.piece->wm[g] = run_m; sg.piece->wl[g] = run_l; }
  }
}

// ---------------------------------------------------------------- value warp
template <int FMT>
__device__ __forceinline__ void value_warp(MmaSmem<FMT>& sm, const Segment& sg, int pair, int lane) {
  const int g = lane >> 2, t = lane & 3;
  float acc[8][4];
#pragma unroll
  for (int mu = 0; mu < 8; mu++)
#pragma unroll
    for (int i = 0; i < 4; i++) acc[mu][i] = 0.f;
  float run_S = 0.f;
  int cur_mod = -1;
  int since = 0;             // windows accumulated in registers since the last deposit
  // nothing deposited yet (the deposited registers themselves are only read where a maximum says so)
  if (lane < 3 * GP) (&sm.spill_m[pair][0][0])[lane] = -INFINITY;
  __syncwarp();
  // The value warp also streams the records: it has registers to spare and the copies of window k + 2 are issued
  // while it works on window k - 1; a window is complete (cp.async.wait_group) before the barrier after which the
  // score warp reads it.
  auto issue = [&](int k) {
    if (k < sg.n_my) {
      const int win = sg.w0 + k;
      unsigned char* dst = sm.stage[pair][k % NSTAGE];
      if (FMT == FMT_FP16) {
        const unsigned char* src = sg.rec0 + (size_t)win * RECORD_BYTES;
#pragma unroll
        for (int i = 0; i < 6; i++) {
          int c16 = lane + 32 * i;
          if (c16 < RECORD_BYTES / 16) cp_async16(dst + 16 * c16, src + 16 * c16);
        }
      } else {
        // body (16-byte aligned) behind the 512 bytes the decoded (m, s) will occupy; the 136
        // metadata bytes are only 8-byte aligned
        // two windows share one block [meta 0 | meta 1 | body 0 | body 1]: offsets in 32 bits
        const uint32_t odd = (uint32_t)win & 1u, blk = ((uint32_t)win >> 1) * (uint32_t)MX_PAIR_BYTES;
        const unsigned char* body = sg.rec0 + (blk + 2u * MX_META_BYTES + odd * (uint32_t)BODY_BYTES);
        const unsigned char* meta = sg.rec0 + (blk + odd * (uint32_t)MX_META_BYTES);
#pragma unroll
        for (int i = 0; i < 5; i++) {
          int c16 = lane + 32 * i;
          if (c16 < BODY_BYTES / 16) cp_async16(dst + META_BYTES_FP16 + 16 * c16, body + 16 * c16);
        }
        if (lane < MX_META_BYTES / 8) cp_async8(dst + STAGE_MX + 8 * lane, meta + 8 * lane);
      }
      if (lane < 2) cp_async16(dst + STAGE_MOD + 16 * lane, sg.mod0 + (size_t)win * W + 16 * lane);
    }
    cp_async_commit();
  };
#pragma unroll
  for (int k = 0; k < PREFETCH; k++) issue(k);
  // with MXFP4 metadata: the stored (m, s) of a window that has landed, expanded into the fp16 planes of its staged image
  auto expand_meta = [&](int k) {
    if (FMT == FMT_MXFP4 && k < sg.n_my) {
      __syncwarp();   // the other lanes' copies have landed too
      unsigned char* st = sm.stage[pair][k % NSTAGE];
      uint2 m4, s4;
      mx_decode_lane(st + STAGE_MX, lane, m4, s4);
      *reinterpret_cast<uint2*>(st + OFF_KM + 8 * lane) = m4;
      *reinterpret_cast<uint2*>(st + OFF_KS + 8 * lane) = s4;
    }
  };
  cp_async_wait<PREFETCH - 1>();
  expand_meta(0);
  pair_barrier(pair);   // window 0 is in place

  // Adds the live accumulators (which refer to the running maxima ho.m) to the current modality's sums in
  // shared memory and clears them.  Apart from modality changes this happens every FLUSH windows: the
  // tensor cores' fp32 accumulation does not round to nearest, so a long chain of MMAs into one register
  // drifts, and the difference against the exactly rounded weight sum run_S is amplified by the codebook's
  // cancellation (code plane minus b times the weight sum); short chains summed with FFMA do not drift.
  auto deposit = [&](const Handoff& ho) {
    float4* dst = reinterpret_cast<float4*>(&sm.spill[pair][cur_mod][lane][0]);
    float* dm = &sm.spill_m[pair][cur_mod][0];
    const float s_lo = dm[2 * t], s_hi = dm[2 * t + 1], s_g = dm[g];
    if (s_g == -INFINITY) {   // first deposit of this modality (the same for every head)
#pragma unroll
      for (int mu = 0; mu < 8; mu++) dst[mu] = make_float4(acc[mu][0], acc[mu][1], acc[mu][2], acc[mu][3]);
      reinterpret_cast<float*>(dst)[32] = run_S;
    } else {
      const float f_lo = ex2(s_lo - ho.m[2 * t]), f_hi = ex2(s_hi - ho.m[2 * t + 1]), f_g = ex2(s_g - ho.m[g]);
#pragma unroll
      for (int mu = 0; mu < 8; mu++) {
        float4 v = dst[mu];
        v.x = fmaf(v.x, f_lo, acc[mu][0]); v.y = fmaf(v.y, f_hi, acc[mu][1]);
        v.z = fmaf(v.z, f_lo, acc[mu][2]); v.w = fmaf(v.w, f_hi, acc[mu][3]);
        dst[mu] = v;
      }
      float* dS = reinterpret_cast<float*>(dst) + 32;
      *dS = fmaf(*dS, f_g, run_S);
    }
    __syncwarp();
    if (t == 0) dm[g] = ho.m[g];
    __syncwarp();
#pragma unroll
    for (int mu = 0; mu < 8; mu++)
#pragma unroll
      for (int i = 0; i < 4; i++) acc[mu][i] = 0.f;
    run_S = 0.f;
    since = 0;
  };

  for (int k = 0; k <= sg.n_my; k++) {
    issue(k + PREFETCH);
    if (k >= 1) {
      const unsigned char* st = sm.stage[pair][(k - 1) % NSTAGE];
      const Handoff& ho = sm.hand[pair][(k - 1) & 1];
      if (ho.rescale) {
        const float a_lo = ho.alpha[2 * t], a_hi = ho.alpha[2 * t + 1];
#pragma unroll
        for (int mu = 0; mu < 8; mu++) {
          acc[mu][0] *= a_lo; acc[mu][1] *= a_hi; acc[mu][2] *= a_lo; acc[mu][3] *= a_hi;
        }
        run_S *= ho.alpha[g];
      }
      const unsigned char* wmod = st + STAGE_MOD;
      const int mymod = wmod[lane];
      const int first = __shfl_sync(0xffffffffu, mymod, 0);
      const bool uniform = __all_sync(0xffffffffu, mymod == first);
      const uint4 vc0 = *reinterpret_cast<const uint4*>(st + OFF_VCODE + 16 * vpiece_slot(lane));
      const uint4 vc1 = *reinterpret_cast<const uint4*>(st + OFF_VCODE + 16 * vpiece_slot(32 + lane));
      const uint32_t vw[8] = {vc0.x, vc0.y, vc0.z, vc0.w, vc1.x, vc1.y, vc1.z, vc1.w};
      const uint4 pb4 = ho.pb[lane];
      const uint32_t pb[4] = {pb4.x, pb4.y, pb4.z, pb4.w};
      // (3a - b) / (2 (b - a)): weight of the bit-1 plane relative to the code plane
      constexpr float DELTA_REL = (3.0f * CB_INNER - CB_OUTER) / (2.0f * (CB_OUTER - CB_INNER));
      const __half2 drel = __float2half2_rn(DELTA_REL);
      // the two bit-plane products of the numerators b0 (zero where a token is not of the current modality) over
      // the 16-token halves named by halfmask, and the weight sum
      auto half_products = [&](const uint32_t (&b0)[4], const uint32_t (&b1)[4], auto kv_c) {
        constexpr int kv = decltype(kv_c)::value;
        constexpr uint32_t mA = 0x00030003u << (4 * kv), mB = 0x000c000cu << (4 * kv);
        constexpr uint32_t nA = 0x00020002u << (4 * kv), nB = 0x00080008u << (4 * kv);
        const uint32_t p0 = b0[2 * kv], p1 = b0[2 * kv + 1], q0 = b1[2 * kv], q1 = b1[2 * kv + 1];
        // the two bit-plane products of one m-tile hit the same accumulator: keep them four
        // MMAs apart so the second never waits for the first
#pragma unroll
        for (int mq = 0; mq < 8; mq += 4) {
          uint32_t w8[4];
#pragma unroll
          for (int i = 0; i < 4; i++) {
            const uint32_t w = vw[mq + i];
            w8[i] = w >> 8;
            mma16816(acc[mq + i], w & mA, w8[i] & mA, w & mB, w8[i] & mB, p0, p1);
          }
#pragma unroll
          for (int i = 0; i < 4; i++) {
            const uint32_t w = vw[mq + i];
            mma16816(acc[mq + i], w & nA, w8[i] & nA, w & nB, w8[i] & nB, q0, q1);
          }
        }
      };
      auto products = [&](const uint32_t (&b0)[4], unsigned halfmask, auto whole) {
        uint32_t b1[4];
#pragma unroll
        for (int nu = 0; nu < 4; nu++) {
          b1[nu] = h2u(__hmul2(u2h(b0[nu]), drel));
          float2 pf = __half22float2(u2h(b0[nu]));   // weight sum from the rounded numerators
          run_S = fmaf(pf.x + pf.y, (float)(1 << (2 * nu)) * (1.0f / 64.0f), run_S);
        }
        if constexpr (decltype(whole)::value) {   // both halves, straight-line, compile-time masks
          half_products(b0, b1, std::integral_constant<int, 0>{});
          half_products(b0, b1, std::integral_constant<int, 1>{});
        } else {
#pragma unroll 1   // rolled on purpose: unrolling both halves makes ptxas spill the accumulators
          for (int kv = 0; kv < 2; kv++) {
            if (!((halfmask >> kv) & 1)) continue;
            const uint32_t mA = 0x00030003u << (4 * kv), mB = 0x000c000cu << (4 * kv);
            const uint32_t nA = 0x00020002u << (4 * kv), nB = 0x00080008u << (4 * kv);
            const uint32_t p0 = kv ? b0[2] : b0[0], p1 = kv ? b0[3] : b0[1];
            const uint32_t q0 = kv ? b1[2] : b1[0], q1 = kv ? b1[3] : b1[1];
#pragma unroll
            for (int mq = 0; mq < 8; mq += 4) {
              uint32_t w8[4];
#pragma unroll
              for (int i = 0; i < 4; i++) {
                const uint32_t w = vw[mq + i];
                w8[i] = w >> 8;
                mma16816(acc[mq + i], w & mA, w8[i] & mA, w & mB, w8[i] & mB, p0, p1);
              }
#pragma unroll
              for (int i = 0; i < 4; i++) {
                const uint32_t w = vw[mq + i];
                mma16816(acc[mq + i], w & nA, w8[i] & nA, w & nB, w8[i] & nB, q0, q1);
              }
            }
          }
        }
      };
      if (uniform && first == cur_mod) {
        // the common case: every token of the window belongs to the modality the registers hold
        products(pb, 3u, std::true_type{});
      } else {
        unsigned present = uniform ? (1u << first)
                                   : ((__any_sync(0xffffffffu, mymod == 0) ? 1u : 0u) |
                                      (__any_sync(0xffffffffu, mymod == 1) ? 2u : 0u) |
                                      (__any_sync(0xffffffffu, mymod == 2) ? 4u : 0u));
        for (int pass = 0; pass < 3 && present; pass++) {
          int m = (cur_mod >= 0 && (present >> cur_mod) & 1) ? cur_mod : (__ffs(present) - 1);
          present &= ~(1u << m);
          if (m != cur_mod) {
            if (cur_mod >= 0) deposit(ho);
            cur_mod = m;
          }
          uint32_t b0[4];
          unsigned halfmask = 3u;  // which 16-token halves hold a token of modality m
          if (uniform) {
#pragma unroll
            for (int nu = 0; nu < 4; nu++) b0[nu] = pb[nu];
          } else {
            bool any_lo = false, any_hi = false;
#pragma unroll
            for (int nu = 0; nu < 4; nu++) {
              const bool k0 = wmod[8 * nu + 2 * t] == m, k1 = wmod[8 * nu + 2 * t + 1] == m;
              b0[nu] = pb[nu] & ((k0 ? 0x0000ffffu : 0u) | (k1 ? 0xffff0000u : 0u));
              if (nu < 2) any_lo |= (k0 | k1); else any_hi |= (k0 | k1);
            }
            halfmask = (__any_sync(0xffffffffu, any_lo) ? 1u : 0u) | (__any_sync(0xffffffffu, any_hi) ? 2u : 0u);
          }
          products(b0, halfmask, std::false_type{});
        }
      }
      // before the barrier: the score warp may overwrite this hand-off record right after it
      if (k == sg.n_my || ++since >= FLUSH) deposit(ho);
    }
    cp_async_wait<1>();   // all but the copies just issued: window k + 1 is complete
    expand_meta(k + 1);
    pair_barrier(pair);
  }
  cp_async_wait<0>();
  // leave the three modalities' accumulators (each lane its own column) and their maxima in the pair's piece
  if (sg.keep) return;   // the block's merge reads this pair's sums where they are
#pragma unroll 1
  for (int m = 0; m < 3; m++) {
    const float mm = sm.spill_m[pair][m][g];
    if (t == 0) sg.piece->sm[m][g] = mm;
    if (mm != -INFINITY) {
      const float4* src = reinterpret_cast<const float4*>(&sm.spill[pair][m][lane][0]);
      float* dst = &sg.piece->frag[m][0][lane];
#pragma unroll
      for (int mu = 0; mu < 8; mu++) {
        const float4 v = src[mu];
        dst[(4 * mu) * 32] = v.x; dst[(4 * mu + 1) * 32] = v.y; dst[(4 * mu + 2) * 32] = v.z; dst[(4 * mu + 3) * 32] = v.w;
      }
      dst[32 * 32] = reinterpret_cast<const float*>(src)[32];
    }
  }
  __syncwarp();
}

}  // namespace

// grid = n_cta (persistent), 512 threads
//
// CTA i owns the windows [i * per, (i + 1) * per) of the flattened (layer, sequence, head, window) axis and
// cuts them into eight contiguous ranges, one per warp pair.  A pair walks its range on its own, with no
// block-wide step in between: where the range crosses into another (sequence, head) the score warp sets up
// that head group's query fragments, the value warp leaves what it accumulated in a PairPartial piece and
// starts afresh.  At the end of the launch the block merges, per (sequence, head) it touched, the pieces of
// the pairs that worked on it into one PartialF.
template <int FMT>
__global__ void __launch_bounds__(NTHREADS, 1) k_decode_mma(DecodeParams P) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  MmaSmem<FMT>& sm = *reinterpret_cast<MmaSmem<FMT>*>(smem_raw);
  const CacheView& cv = P.cv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int pair = warp & (NPAIR - 1);
  const bool is_score = warp < NPAIR;
  const int G = P.group, Hkv = cv.n_kv_heads;
  const int n_entries = P.layer_count * cv.batch;

  // ---- partition of the flattened window axis
  const int total = block_prefix(cv, P.layer0, n_entries, sm.prefix);
  const int per = (total + gridDim.x - 1) / gridDim.x;
  const int pos0 = min(total, (int)blockIdx.x * per), pos1 = min(total, pos0 + per);
  const int cnt = (pos1 - pos0 + NPAIR - 1) / NPAIR;

  struct Where { int e, h, w0, nwin; };
  auto locate = [&](int pos) {   // (entry, head, window) of a flattened position; largest e with prefix[e] <= pos
    int lo = 0, hi = n_entries;
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (sm.prefix[mid] <= pos) lo = mid; else hi = mid;
    }
    Where wh;
    wh.e = lo;
    wh.nwin = (sm.prefix[lo + 1] - sm.prefix[lo]) / Hkv;
    const int off = pos - sm.prefix[lo];
    wh.h = off / wh.nwin;
    wh.w0 = off % wh.nwin;
    return wh;
  };

  {
    int pos = min(pos1, pos0 + pair * cnt);
    const int pos_end = min(pos1, pos + cnt);
    while (pos < pos_end) {
      const Where wh = locate(pos);
      const int li = wh.e / cv.batch, b = wh.e % cv.batch;
      Segment sg;
      sg.rec0 = cv.unit(P.layer0 + li, b, wh.h);
      sg.mod0 = cv.modality + (size_t)b * cv.capacity;
      sg.w0 = wh.w0;
      sg.n_my = min(pos_end - pos, wh.nwin - wh.w0);
      sg.q = P.q + (((size_t)li * cv.batch + b) * cv.n_q_heads + (size_t)wh.h * G) * D;
      sg.signs = P.signs + (size_t)li * D;
      sg.piece = P.pair_parts + (size_t)(wh.e * Hkv + wh.h) + ((size_t)blockIdx.x * NPAIR + pair);
      sg.keep = pos + sg.n_my == pos_end;
      if (is_score) score_warp<FMT>(sm, sg, G, P.sm_scale, pair, lane);
      else value_warp<FMT>(sm, sg, pair, lane);
      pos += sg.n_my;
    }
  }
  __syncthreads();   // the pieces were written by this block's own warps: visible to the block from here on

  // ---- merge the pairs' pieces into one partial per (sequence, head) of the block's range, MB_SEG
  // (sequence, head) units at a time so that the loads of many units are in flight together.  The tables
  // take the place of the record ring, which is idle by now.
  if (pos0 >= pos1) return;
  MergeSmem& mg = *reinterpret_cast<MergeSmem*>(smem_raw);
  const Where wf = locate(pos0), wl = locate(pos1 - 1);
  const int u_first = wf.e * Hkv + wf.h, u_last = wl.e * Hkv + wl.h;
  for (int ub = u_first; ub <= u_last; ub += MB_SEG) {
    const int n_u = min(MB_SEG, u_last - ub + 1);
    // (a) the units' window ranges inside the block's slice and the pairs that worked on them
    if (tid < n_u) {
      const int u = ub + tid, e = u / Hkv, h = u % Hkv;
      const int nwin = (sm.prefix[e + 1] - sm.prefix[e]) / Hkv;
      const int a0 = max(pos0, sm.prefix[e] + h * nwin), a1 = min(pos1, sm.prefix[e] + (h + 1) * nwin);
      mg.pa[tid] = a1 > a0 ? (a0 - pos0) / cnt : 0;
      const int pb = a1 > a0 ? (a1 - 1 - pos0) / cnt : -1;   // empty: a (sequence, head) with no packed window
      mg.pb[tid] = pb;
      // pairs before the last end their range inside this unit, so their sums are still in shared memory; the
      // last one's are too unless its range goes on into the next unit
      mg.last_kept[tid] = pb >= 0 && min(pos1, pos0 + (pb + 1) * cnt) <= a1;
    }
    __syncthreads();
    // (b) the pieces' maxima and weight sums: one warp per (unit, pair)
    for (int j = warp; j < n_u * NPAIR; j += NTHREADS / 32) {
      const int su = j / NPAIR, p = j % NPAIR;
      if (p < mg.pa[su] || p > mg.pb[su]) continue;
      float* dst = mg.meta[su + p - mg.pa[0]];
      if (p < mg.pb[su] || mg.last_kept[su]) {
        dst[lane] = lane < 3 * GP ? (&sm.spill_m[p][0][0])[lane] : sm.fin_w[p][0][lane - 3 * GP];
        if (lane < GP) dst[32 + lane] = sm.fin_w[p][1][lane];
      } else {
        const PairPartial& pp = P.pair_parts[(size_t)(ub + su) + (size_t)blockIdx.x * NPAIR + p];
        dst[lane] = (&pp.sm[0][0])[lane];                         // sm[3][GP], then wm[GP]
        if (lane < GP) dst[32 + lane] = pp.wl[lane];
      }
    }
    __syncthreads();
    // (c) merged maximum and weight sum per (unit, head)
    if (tid < n_u * GP) {
      const int su = tid / GP, j = tid % GP;
      if (mg.pb[su] >= mg.pa[su]) {
        float mj = -INFINITY, L = 0.f;
        for (int p = mg.pa[su]; p <= mg.pb[su]; p++) mj = fmaxf(mj, mg.meta[su + p - mg.pa[0]][3 * GP + j]);
        for (int p = mg.pa[su]; p <= mg.pb[su]; p++) {
          const float* me = mg.meta[su + p - mg.pa[0]];
          L += me[4 * GP + j] * exp2f(me[3 * GP + j] - mj);
        }
        mg.M[su][j] = mj;
        PartialF* out = P.partials_f + (size_t)(ub + su) + blockIdx.x;
        out->m[j] = mj;
        out->l[j] = L;
      }
    }
    __syncthreads();
    // (d) the accumulators: one item = four lanes' worth of one (unit, modality, register) row
    // rescale factors, once per (piece, modality, head)
    for (int j = tid; j < n_u * NPAIR * 3 * GP; j += NTHREADS) {
      const int su = j / (NPAIR * 3 * GP), p = (j / (3 * GP)) % NPAIR, k = j % (3 * GP);
      if (p < mg.pa[su] || p > mg.pb[su]) continue;
      const float smv = mg.meta[su + p - mg.pa[0]][k];
      (&mg.fac[su + p - mg.pa[0]][0][0])[k] = smv == -INFINITY ? 0.f : exp2f(smv - mg.M[su][k % GP]);
    }
    __syncthreads();
    // (d) the accumulators: one item = four consecutive registers of one lane of one (unit, modality), or that
    // lane's weight sum.  A lane's registers are one 128-bit row read where the piece is still in shared memory;
    // registers r and r + 2 belong to head 2 (lane & 3), r + 1 and r + 3 to the next head.
    constexpr int RG = 9, UNIT_ITEMS = 3 * RG * 32;
    for (int it = tid; it < n_u * UNIT_ITEMS; it += NTHREADS) {
      const int su = it / UNIT_ITEMS, idx = it % UNIT_ITEMS;
      const int L = idx & 31, rg = (idx >> 5) % RG, m = idx / (RG * 32);
      const int pa = mg.pa[su], np = mg.pb[su] - pa + 1;
      if (np <= 0) continue;
      const int inc0 = su + pa - mg.pa[0];
      const bool last_kept = mg.last_kept[su] != 0;
      const int hsel = rg < 8 ? 2 * (L & 3) : (L >> 2);
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int q = 0; q < NPAIR; q++) {
        if (q >= np || mg.meta[inc0 + q][m * GP] == -INFINITY) continue;   // no such pair / no token of this modality
        const float* fc = mg.fac[inc0 + q][m];
        const float fe = fc[hsel], fo = rg < 8 ? fc[hsel + 1] : fe;
        float4 x;
        if (q < np - 1 || last_kept) {
          const float* sp = &sm.spill[pa + q][m][L][0];
          x = rg < 8 ? *reinterpret_cast<const float4*>(sp + 4 * rg) : make_float4(sp[32], 0.f, 0.f, 0.f);
        } else {
          const float* gp = &P.pair_parts[(size_t)(ub + su) + (size_t)blockIdx.x * NPAIR + pa + q].frag[m][0][L];
          x = rg < 8 ? make_float4(gp[(4 * rg) * 32], gp[(4 * rg + 1) * 32], gp[(4 * rg + 2) * 32], gp[(4 * rg + 3) * 32])
                     : make_float4(gp[32 * 32], 0.f, 0.f, 0.f);
        }
        v.x = fmaf(x.x, fe, v.x); v.y = fmaf(x.y, fo, v.y); v.z = fmaf(x.z, fe, v.z); v.w = fmaf(x.w, fo, v.w);
      }
      PartialF* out = P.partials_f + (size_t)(ub + su) + blockIdx.x;
      if (rg < 8) {
        out->frag[m][4 * rg][L] = v.x; out->frag[m][4 * rg + 1][L] = v.y;
        out->frag[m][4 * rg + 2][L] = v.z; out->frag[m][4 * rg + 3][L] = v.w;
      } else {
        out->Sp[m][L] = v.x;
      }
    }
    __syncthreads();
  }
}

constexpr int PARTIAL_HDR_FLOATS = 2 * GP + 3 * 32;   // m[GP], l[GP], Sp[3][32] at the start of a PartialF
constexpr int CB_SEQ_MAX = 4;             // most sequences per combine CTA (one 128-thread group each)

constexpr int MRG_MAX = 8;                // partials per (sequence, head) whose factors are precomputed
constexpr int CB_CHUNK = 16;              // rows of a rotation matrix staged per step
constexpr int CB_NBUF = 4;                // staged slices in flight (three ahead of the one in use)

// CAPTION: the captioning schedule keeps up to 159 raw values (and up to 127 raw keys) per sequence, and
// the keys of the raw values' tokens may already be packed
// SEQ: sequences per CTA (4 for full grids: the matrices are streamed once per four sequences; 1 when the
// grid would otherwise leave most SMs idle, e.g. a single-layer call)
template <bool CAPTION, int SEQ>
struct CombineSmem {
  static constexpr int CB_SEQ = SEQ, CB_ROWS = SEQ * GP;
  static constexpr int TAIL = CAPTION ? CAPTION_V_SLOTS : W;   // most raw-value tokens of a sequence
  // ring of 16-row slices of the rotation matrices; with one sequence per block it is large enough for a quarter
  // of the columns of all three matrices, which the four-slice configuration fetches whole at the start
  static constexpr int RBUF_FLOATS = SEQ == 1 ? 3 * D * (D / 4) : CB_NBUF * CB_CHUNK * D;
  __align__(16) float Rbuf[RBUF_FLOATS];
  // per partial and head: rescale factor, weight sums of the modalities (one-sequence blocks have room for the
  // partials of a long single sequence, which is spread over many CTAs of the split-K kernel)
  static constexpr int MRG_TAB = SEQ == 1 ? 64 : MRG_MAX;
  __align__(16) float mrg[CB_SEQ][MRG_TAB][GP][4];
  __align__(16) float vec[3][CB_ROWS][D];     // merged rotated-basis sums, [modality][row][rotated channel]
  __align__(16) float rawv[CB_ROWS][D];       // raw-tail contribution, [row][channel]
  // tail scores (log2 domain), then softmax numerators, [sequence][token][head]: blocks of several sequences keep
  // them in the matrix ring, which is idle until the rotated sums are complete
  static constexpr bool TSC_IN_RING = SEQ != 1;
  static_assert(!TSC_IN_RING || CB_SEQ * TAIL * GP <= RBUF_FLOATS, "tail scores must fit the matrix ring");
  __align__(16) float tsc_own[TSC_IN_RING ? 4 : CB_SEQ * TAIL * GP];
  float Ms[CB_SEQ][GP], Ls[CB_SEQ][GP];
  float red[CB_SEQ][4][GP];   // per warp of a sequence: partial maxima / sums of the softmax bookkeeping
  // one-sequence blocks: the headers (m, l, weight sums) of the sequence's first MRG_TAB partials, fetched early
  __align__(16) float hdr[SEQ == 1 ? MRG_TAB * PARTIAL_HDR_FLOATS : 4];
  __align__(16) __half vsm[SEQ == 1 ? TAIL * D : 8];   // one-sequence blocks: the raw value rows, fetched early
  int prefix[MAX_ENTRIES + 1];
};

// (stored m, s) at position p of a window's (m, s) planes, from its metadata in either format; the fp16 format's
// m carries its position scale, the MXFP4 format decodes to the plain value
__device__ __forceinline__ float2 window_meta_pos(const unsigned char* meta, int fmt, int p) {
  if (fmt == FMT_FP16)
    return make_float2(__half2float(reinterpret_cast<const __half*>(meta + OFF_KM)[p]),
                       __half2float(reinterpret_cast<const __half*>(meta + OFF_KS)[p]));
  const unsigned mn = (meta[p >> 1] >> (4 * (p & 1))) & 15u, sn = (meta[64 + (p >> 1)] >> (4 * (p & 1))) & 15u;
  const int blk = (p >> 3) & 3;
  return make_float2(mx_decode(mn, (int)meta[128 + blk] - 127), mx_decode(sn, (int)meta[132 + blk] - 127));
}

// NS: CTAs that share one (head, sequence group): each computes D / NS output columns (used when the grid
// would otherwise leave most SMs idle; the merge is repeated by every slice, the matrix streaming is split)
template <bool CAPTION, int NS, int SEQ>
__global__ void __launch_bounds__(SEQ * 128, SEQ == CB_SEQ_MAX ? 2 : 1) k_combine_mma(DecodeParams P, int n_cta) {
  constexpr int CB_SEQ = SEQ, CB_ROWS = SEQ * GP;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  CombineSmem<CAPTION, SEQ>& sm = *reinterpret_cast<CombineSmem<CAPTION, SEQ>*>(smem_raw);
  float* const tsc_base = sm.TSC_IN_RING ? &sm.Rbuf[0] : &sm.tsc_own[0];
  auto tsc = [&](int b_, int i_) -> float* { return tsc_base + ((size_t)b_ * sm.TAIL + i_) * GP; };   // one token's eight heads
  const CacheView& cv = P.cv;
  const int h = blockIdx.x / NS, sl = blockIdx.x % NS, li = blockIdx.z, layer = P.layer0 + li;
  const int bs = threadIdx.x >> 7, c = threadIdx.x & 127;
  const int b = blockIdx.y * CB_SEQ + bs;
  const bool live = b < cv.batch;
  const int bb = live ? b : 0;
  const int G = P.group, Hkv = cv.n_kv_heads;
  const int n_entries = P.layer_count * cv.batch;
  const int seq = live ? cv.seq_len[layer * cv.batch + bb] : 0;
  // tokens [0, v_pk) have packed values (and keys): they are in the split-K partials; tokens [v_pk, seq) have raw
  // values; of those, [v_pk, k_pk) have packed keys (captioning schedule only), the rest raw keys
  const int v_pk = cv.v_packed(seq), k_pk = cv.k_packed(seq);
  const int nwin = v_pk / W, n_tail = seq - v_pk;
  const __half* qbase = P.q + (((size_t)li * cv.batch + bb) * cv.n_q_heads + h * G) * D;
  const __half* kt = cv.k_tail + cv.k_tail_off(layer, bb, h);
  const __half* vt = cv.v_tail + cv.v_tail_off(layer, bb, h);
  // Scratch inside the rotated-sum array (written much later), per sequence: the raw key rows of a chunk of the
  // tail (272-byte rows: 16-byte reads of 32 different rows hit different banks) or, under the captioning
  // schedule, the key parts of the up to four packed windows among the raw-value tokens; then the group's query
  // rows.  Everything is fetched with cp.async so that all the loads are in flight together.
  constexpr int KROW = D + 8;                              // halfs per staged key row
  constexpr int KSM_FLOATS = W * KROW / 2, QSM_FLOATS = GP * D / 2;
  constexpr int KIMG = OFF_VCODE + 144;                    // key part of a window record (+ its MXFP4 metadata bytes)
  static_assert(CB_SEQ * (KSM_FLOATS + QSM_FLOATS) <= 3 * CB_ROWS * D && 4 * KIMG <= KSM_FLOATS * 4, "tail scratch must fit");
  __half* ksm = reinterpret_cast<__half*>(&sm.vec[0][0][0] + bs * (KSM_FLOATS + QSM_FLOATS));
  __half* qsm = ksm + W * KROW;
  unsigned char* kimg = reinterpret_cast<unsigned char*>(ksm);
  const int npc = CAPTION ? (k_pk - v_pk) / W : 0;   // packed windows among the raw-value tokens: the first chunks
  // a chunk of the tail is one 32-token window: its keys are either all packed or all raw
  auto stage_tail = [&](int chunk) {
    if (chunk == 0 && c < G * (D / 8)) cp_async16(qsm + 8 * c, qbase + 8 * c);
    if (chunk >= npc)
      for (int idx = c; idx < W * (D / 8); idx += 128) {
        const int r = idx / (D / 8), c8 = idx % (D / 8);
        if (chunk * W + r < n_tail)
          cp_async16(ksm + r * KROW + 8 * c8, kt + cv.k_slot(v_pk + chunk * W + r) * D + 8 * c8);
      }
    cp_async_commit();
  };
  if (SEQ == 1)   // the raw value rows go the same way (used after the softmax numerators are known)
    for (int idx = c; idx < n_tail * (D / 8); idx += 128) {
      const int r = idx / (D / 8), c8 = idx % (D / 8);
      cp_async16(&sm.vsm[r * D + 8 * c8], vt + cv.v_slot(v_pk + r) * D + 8 * c8);
    }
  for (int ch = 0; ch < npc; ch++) {   // key parts of the packed windows whose values are still raw
    const int win = v_pk / W + ch;
    unsigned char* img = kimg + ch * KIMG;
    if (cv.fmt == FMT_FP16) {
      const unsigned char* rec = cv.meta(layer, bb, h, win);   // the record starts with its (m, s) planes
      if (c < OFF_VCODE / 16) cp_async16(img + 16 * c, rec + 16 * c);
    } else {
      const unsigned char* body = cv.body(layer, bb, h, win);
      const unsigned char* meta = cv.meta(layer, bb, h, win);
      if (c < 4) cp_async16(img + OFF_KNORM + 16 * c, body + B_KNORM + 16 * c);
      else if (c < 4 + 64) cp_async16(img + OFF_KCODE + 16 * (c - 4), body + B_KCODE + 16 * (c - 4));
      else if (c < 4 + 64 + MX_META_BYTES / 8) cp_async8(img + OFF_VCODE + 8 * (c - 68), meta + 8 * (c - 68));
    }
  }
  if (n_tail > 0) stage_tail(0);   // on its way while the prefix is computed
  const int total = block_prefix(cv, P.layer0, n_entries, sm.prefix);
  const int per = total > 0 ? (total + n_cta - 1) / n_cta : 1;
  constexpr float ACC_SCALE = (CB_OUTER - CB_INNER) * 262144.0f;  // (b - a) * 2^18
  constexpr float LOG2E = 1.4426950408889634f;
  // Coefficient of the weight sum S: -b from the codebook identity, plus the mean of what the bit-1
  // plane loses because its relative weight (3a-b)/(2(b-a)) enters the MMA rounded to fp16 (bit 1 is
  // set for half of the codes on average); the zero-mean remainder is at the 1e-5 level.
  constexpr float DELTA_REL = (3.0f * CB_INNER - CB_OUTER) / (2.0f * (CB_OUTER - CB_INNER));
  const float S_COEF = -CB_OUTER + (CB_OUTER - CB_INNER) * (DELTA_REL - __half2float(__float2half_rn(DELTA_REL)));

  const int e = li * cv.batch + bb;
  const int unit = e * Hkv + h;
  const int start = sm.prefix[e] + h * nwin, end = start + nwin;
  const int cta_lo = nwin > 0 ? start / per : 0, cta_hi = nwin > 0 ? (end - 1) / per : -1;
  const int n_hdr = SEQ == 1 ? max(0, min(cta_hi - cta_lo + 1, sm.MRG_TAB)) : 0;   // partials whose headers are staged
  if (SEQ == 1) {
    for (int idx = c; idx < n_hdr * (PARTIAL_HDR_FLOATS / 4); idx += 128) {
      const int ci = idx / (PARTIAL_HDR_FLOATS / 4), q4 = idx % (PARTIAL_HDR_FLOATS / 4);
      cp_async16(&sm.hdr[ci * PARTIAL_HDR_FLOATS + 4 * q4],
                 reinterpret_cast<const float*>(&P.partials_f[(size_t)unit + cta_lo + ci]) + 4 * q4);
    }
    cp_async_commit();
  }
  if (CAPTION) {   // scores of the packed windows among the raw-value tokens: one warp per window, on the tensor cores
    cp_async_wait<0>();
    __syncthreads();
    const int wv = c >> 5, lane = c & 31;
    if (wv < npc) {
      Segment sq;
      sq.q = qbase;
      sq.signs = P.signs + (size_t)li * D;
      uint2 qreg[16];
      float fsc;
      query_fragments(sq.q, sq.signs, G, P.sm_scale, lane, qreg, fsc);
      unsigned char* st = kimg + wv * KIMG;
      if (cv.fmt == FMT_MXFP4) {   // decode the stored (m, s) into the fp16 planes of the staged image
        uint2 m4, s4;
        mx_decode_lane(st + OFF_VCODE, lane, m4, s4);
        *reinterpret_cast<uint2*>(st + OFF_KM + 8 * lane) = m4;
        *reinterpret_cast<uint2*>(st + OFF_KS + 8 * lane) = s4;
        __syncwarp();
      }
      float sc[4][2];
      window_scores_mma(st, qreg, fsc, lane, sc);
      const int g = lane >> 2, t = lane & 3;
#pragma unroll
      for (int nu = 0; nu < 4; nu++)
#pragma unroll
        for (int e2 = 0; e2 < 2; e2++)
          tsc(bs, wv * W + 8 * nu + 2 * t + e2)[g] = g < G ? sc[nu][e2] : -INFINITY;
    }
    __syncthreads();   // the images are done with: the scratch takes raw key rows next
  }
  // tail scores: thread -> (token = c & 31 of a 32-token chunk, heads (c >> 5) * 2 + {0, 1})
  for (int chunk = npc; chunk * W < n_tail; chunk++) {   // chunks of raw keys
    const int tok = chunk * W + (c & 31);
    float s2[2] = {-INFINITY, -INFINITY};
    const int j0 = (c >> 5) * 2;
    if (chunk > 0) stage_tail(chunk);
    cp_async_wait<0>();
    asm volatile("bar.sync %0, 128;\n" ::"r"(bs + 1) : "memory");   // the sequence's 128 threads
    if (tok < n_tail && j0 < G) {
      float a2[2] = {0.f, 0.f};
      {
        const __half* krow = ksm + (c & 31) * KROW;
#pragma unroll 4
        for (int k = 0; k < D; k += 8) {
          const uint4 kv = *reinterpret_cast<const uint4*>(krow + k);
          const __half2* k2 = reinterpret_cast<const __half2*>(&kv);
#pragma unroll
          for (int hh = 0; hh < 2; hh++) {
            if (j0 + hh >= G) continue;
            const uint4 qv = *reinterpret_cast<const uint4*>(qsm + (j0 + hh) * D + k);
            const __half2* q2 = reinterpret_cast<const __half2*>(&qv);
#pragma unroll
            for (int u = 0; u < 4; u++) {
              const float2 qf = __half22float2(q2[u]), kf = __half22float2(k2[u]);
              a2[hh] = fmaf(qf.x, kf.x, a2[hh]);
              a2[hh] = fmaf(qf.y, kf.y, a2[hh]);
            }
          }
        }
      }
      s2[0] = a2[0] * P.sm_scale * LOG2E;
      if (j0 + 1 < G) s2[1] = a2[1] * P.sm_scale * LOG2E;
    }
    if (tok < sm.TAIL) { tsc(bs, tok)[j0] = s2[0]; tsc(bs, tok)[j0 + 1] = s2[1]; }
    if ((chunk + 1) * W < n_tail)
      asm volatile("bar.sync %0, 128;\n" ::"r"(bs + 1) : "memory");   // before the next chunk's rows land
  }
  // Blocks of several sequences have no room to hold all raw value rows: they pass through the key-row scratch 32
  // rows at a time, the first 32 on their way from here on (used once the softmax numerators are known).
  __half* vrows = ksm;
  auto stage_values = [&](int r0) {
    for (int idx = c; idx < min(W, n_tail - r0) * (D / 8); idx += 128) {
      const int r = idx / (D / 8), c8 = idx % (D / 8);
      cp_async16(vrows + r * D + 8 * c8, vt + cv.v_slot(v_pk + r0 + r) * D + 8 * c8);
    }
    cp_async_commit();
  };
  if (SEQ != 1 && n_tail > 0) {
    asm volatile("bar.sync %0, 128;\n" ::"r"(bs + 1) : "memory");   // the last chunk's key rows have been read
    stage_values(0);
  }
  // four column slices per (head, sequence): this block's 32 columns of the three matrices (48 KB) start their way
  // into shared memory now (behind the tail's own cp.async groups, which had to be waited for) and are used at the
  // very end, after the merge
  constexpr bool PRELOAD = NS == 4;
  static_assert(!PRELOAD || SEQ == 1, "the whole-slice preload needs the one-sequence buffer");
  if (PRELOAD) {
    const float* Rsl = P.R + ((size_t)li * P.n_R + (P.n_R == 1 ? 0 : h)) * 3 * D * D + sl * (D / NS);
    for (int i = threadIdx.x; i < 3 * D * (D / NS) / 4; i += SEQ * 128) {
      const int row = i / (D / NS / 4), c4 = i % (D / NS / 4);
      cp_async16(&sm.Rbuf[row * (D / NS) + 4 * c4], Rsl + (size_t)row * D + 4 * c4);
    }
    cp_async_commit();
  }
  // the staged headers must have landed (a sequence without tail tokens has not waited yet); the matrix preload,
  // the newest group, may stay in flight
  if (SEQ == 1) { if (PRELOAD) cp_async_wait<1>(); else cp_async_wait<0>(); }
  __syncthreads();
  {
    // Softmax bookkeeping by all 128 threads of the sequence: thread = (head j, stripe); a stripe takes every 16th
    // partial and every 16th tail token (the captioning schedule has up to 159 of them); stripes are joined by two
    // shuffles inside a warp and a four-entry table across the warps.
    const int j = c & (GP - 1), stripe = c >> 3, wv = c >> 5, lane = c & 31;
    const int n_part = cta_hi - cta_lo + 1;
    auto part_m = [&](int ci) {
      return ci < n_hdr ? sm.hdr[ci * PARTIAL_HDR_FLOATS + j] : P.partials_f[(size_t)unit + cta_lo + ci].m[j];
    };
    auto part_l = [&](int ci) {
      return ci < n_hdr ? sm.hdr[ci * PARTIAL_HDR_FLOATS + GP + j] : P.partials_f[(size_t)unit + cta_lo + ci].l[j];
    };
    float M = -INFINITY;
    for (int ci = stripe; ci < n_part; ci += 16) M = fmaxf(M, part_m(ci));
    for (int i = stripe; i < n_tail; i += 16) M = fmaxf(M, tsc(bs, i)[j]);
    M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 8));
    M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 16));
    if (lane < GP) sm.red[bs][wv][j] = M;
    asm volatile("bar.sync %0, 128;\n" ::"r"(bs + 1) : "memory");
    M = fmaxf(fmaxf(sm.red[bs][0][j], sm.red[bs][1][j]), fmaxf(sm.red[bs][2][j], sm.red[bs][3][j]));
    asm volatile("bar.sync %0, 128;\n" ::"r"(bs + 1) : "memory");   // the table is reused for the sums
    float L = 0.f;
    for (int ci = stripe; ci < n_part; ci += 16) {
      const float pm = part_m(ci);
      if (pm != -INFINITY) L += part_l(ci) * exp2f(pm - M);
    }
    for (int i = stripe; i < n_tail; i += 16) {   // softmax numerators in place of the scores
      const float pnum = exp2f(tsc(bs, i)[j] - M);   // 0 for the heads beyond the group (-inf scores)
      tsc(bs, i)[j] = pnum;
      L += pnum;
    }
    L += __shfl_xor_sync(0xffffffffu, L, 8);
    L += __shfl_xor_sync(0xffffffffu, L, 16);
    if (lane < GP) sm.red[bs][wv][j] = L;
    asm volatile("bar.sync %0, 128;\n" ::"r"(bs + 1) : "memory");
    if (c < GP) {
      sm.Ms[bs][c] = M;
      sm.Ls[bs][c] = (sm.red[bs][0][c] + sm.red[bs][1][c]) + (sm.red[bs][2][c] + sm.red[bs][3][c]);
    }
  }
  __syncthreads();
  // per partial and head: the rescale factor exp2(m - M) and the weight sums S_m (the four lanes of a quad hold
  // partial sums), so that the merge below only reads accumulator fragments
  for (int idx = c; idx < min(cta_hi - cta_lo + 1, sm.MRG_TAB) * GP; idx += 128) {
    const int ci = idx / GP, j = idx % GP;
    // the partial's header: staged in shared memory (one-sequence blocks) or in global memory
    const float* ph = ci < n_hdr ? &sm.hdr[ci * PARTIAL_HDR_FLOATS]
                                 : reinterpret_cast<const float*>(&P.partials_f[(size_t)unit + cta_lo + ci]);
    const float pm = ph[j];
    float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
    if (pm != -INFINITY) {
      const float4 s0 = *reinterpret_cast<const float4*>(ph + 2 * GP + 4 * j);
      const float4 s1 = *reinterpret_cast<const float4*>(ph + 2 * GP + 32 + 4 * j);
      const float4 s2 = *reinterpret_cast<const float4*>(ph + 2 * GP + 64 + 4 * j);
      f.x = exp2f(pm - sm.Ms[bs][j]);
      f.y = s0.x + s0.y + s0.z + s0.w;
      f.z = s1.x + s1.y + s1.z + s1.w;
      f.w = s2.x + s2.y + s2.z + s2.w;
    }
    *reinterpret_cast<float4*>(sm.mrg[bs][ci][j]) = f;
  }
  __syncthreads();
  // raw-value tokens: every value row is read once for all heads
  float araw[GP];
#pragma unroll
  for (int j = 0; j < GP; j++) araw[j] = 0.f;
  constexpr int TAIL_ALL = 1 << 20;   // one-sequence blocks hold all their raw value rows: a single pass
  for (int r0 = 0; r0 < n_tail; r0 += (SEQ == 1 ? TAIL_ALL : W)) {
    const __half* rows = SEQ == 1 ? sm.vsm : vrows;
    if (SEQ != 1) {
      if (r0 > 0) {
        asm volatile("bar.sync %0, 128;\n" ::"r"(bs + 1) : "memory");   // everyone is done with the previous rows
        stage_values(r0);
      }
      cp_async_wait<0>();
      asm volatile("bar.sync %0, 128;\n" ::"r"(bs + 1) : "memory");
    }
    const int nr = SEQ == 1 ? n_tail : min(W, n_tail - r0);
#pragma unroll 8
    for (int i = 0; i < nr; i++) {
      const float x = __half2float(rows[i * D + c]);
      const float4 w0 = *reinterpret_cast<const float4*>(tsc(bs, r0 + i));
      const float4 w1 = *reinterpret_cast<const float4*>(tsc(bs, r0 + i) + 4);
      araw[0] = fmaf(w0.x, x, araw[0]); araw[1] = fmaf(w0.y, x, araw[1]);
      araw[2] = fmaf(w0.z, x, araw[2]); araw[3] = fmaf(w0.w, x, araw[3]);
      araw[4] = fmaf(w1.x, x, araw[4]); araw[5] = fmaf(w1.y, x, araw[5]);
      araw[6] = fmaf(w1.z, x, araw[6]); araw[7] = fmaf(w1.w, x, araw[7]);
    }
  }
  // (the value rows passed through scratch inside the rotated-sum array, which the merge below fills: a sequence
  // group must not start writing it while another still reads its rows)
  if (SEQ != 1) __syncthreads();
  // merge of the split-K partials, four heads at a time: per partial the twelve accumulator fragments of this
  // thread's channel are fetched together (independent loads), then scaled by the table's factors
#pragma unroll
  for (int jg = 0; jg < GP; jg += 4) {
    float vacc[4][3];
#pragma unroll
    for (int jj = 0; jj < 4; jj++) vacc[jj][0] = vacc[jj][1] = vacc[jj][2] = 0.f;
    if (jg < G) {
      // one-sequence blocks have registers to spare: the fragments of four partials are fetched together (a long
      // single sequence has dozens of partials per head)
      constexpr int MU4 = SEQ == 1 ? 4 : 1;
      for (int ct0 = cta_lo; ct0 <= cta_hi; ct0 += MU4) {
        float fr[MU4][4][3];
#pragma unroll
        for (int u = 0; u < MU4; u++) {
          const PartialF& pp = P.partials_f[(size_t)unit + min(ct0 + u, cta_hi)];
#pragma unroll
          for (int jj = 0; jj < 4; jj++) {
            const int j = jg + jj;
            const int r = 4 * (c >> 4) + 2 * ((c >> 3) & 1) + (j & 1), l32 = 4 * (c & 7) + (j >> 1);
#pragma unroll
            for (int m = 0; m < 3; m++) fr[u][jj][m] = pp.frag[m][r][l32];
          }
        }
#pragma unroll
        for (int u = 0; u < MU4; u++) {
          const int ct = ct0 + u;
          if (ct > cta_hi) continue;
          const PartialF& pp = P.partials_f[(size_t)unit + ct];
#pragma unroll
          for (int jj = 0; jj < 4; jj++) {
            const int j = jg + jj;
            float ef, S[3];
            if (ct - cta_lo < sm.MRG_TAB) {
              const float4 f = *reinterpret_cast<const float4*>(sm.mrg[bs][ct - cta_lo][j]);
              ef = f.x; S[0] = f.y; S[1] = f.z; S[2] = f.w;
            } else {   // more partials than the table holds (few heads over many CTAs): compute in place
              const float pm = pp.m[j];
              ef = pm == -INFINITY ? 0.f : exp2f(pm - sm.Ms[bs][j]);
#pragma unroll
              for (int m = 0; m < 3; m++) S[m] = pp.Sp[m][4 * j] + pp.Sp[m][4 * j + 1] + pp.Sp[m][4 * j + 2] + pp.Sp[m][4 * j + 3];
            }
            if (j < G && ef != 0.f) {
#pragma unroll
              for (int m = 0; m < 3; m++) vacc[jj][m] = fmaf(fmaf(ACC_SCALE, fr[u][jj][m], S_COEF * S[m]), ef, vacc[jj][m]);
            }
          }
        }
      }
    }
#pragma unroll
    for (int jj = 0; jj < 4; jj++) {
      sm.vec[0][bs * GP + jg + jj][c] = vacc[jj][0];
      sm.vec[1][bs * GP + jg + jj][c] = vacc[jj][1];
      sm.vec[2][bs * GP + jg + jj][c] = vacc[jj][2];
      sm.rawv[bs * GP + jg + jj][c] = araw[jg + jj];
    }
  }

  // out[row][c] = raw[row][c] + sum_m sum_r R_m[r][c] * vec[m][row][r].  The first half of the threads compute
  // a 4-row x 4-column tile each; the second half stream the matrices through shared memory in 16-row
  // slices, three slices ahead.
  // (with the matrices preloaded there is nothing to stream: both halves compute, each every other 16-row slice)
  constexpr bool PRE = NS == 4;
  const int khalf = PRE ? threadIdx.x / (CB_SEQ * 64) : 0;
  const bool comp = PRE || threadIdx.x < CB_SEQ * 64;
  constexpr int CW = 4 / NS;          // output columns per compute thread
  constexpr int SW = D / NS;          // output columns of this CTA = floats per staged matrix row
  static_assert(NS == 1 || NS == 4, "column slices");
  const int rw = ((threadIdx.x % (CB_SEQ * 64)) >> 5) * 4, cl = (threadIdx.x & 31) * CW;   // first row / column (inside the slice) of the tile
  const float* Rset = P.R + ((size_t)li * P.n_R + (P.n_R == 1 ? 0 : h)) * 3 * D * D + sl * SW;
  constexpr int N_CHUNK = 3 * D / CB_CHUNK;
  float* rbuf = &sm.Rbuf[0];          // ring of CB_NBUF slices of CB_CHUNK x SW floats (or, preloaded, all rows)
  auto stage = [&](int chunk) {   // rows [16*chunk, 16*chunk+16) of the three stacked matrices, this CTA's columns
    const float* src = Rset + (size_t)chunk * CB_CHUNK * D;
    float* dst = rbuf + (chunk % CB_NBUF) * CB_CHUNK * SW;
    if (chunk < N_CHUNK)
      for (int i = threadIdx.x - CB_SEQ * 64; i < CB_CHUNK * SW / 4; i += CB_SEQ * 64) {
        const int row = i / (SW / 4), c4 = i % (SW / 4);
        cp_async16(dst + row * SW + 4 * c4, src + (size_t)row * D + 4 * c4);
      }
    cp_async_commit();
  };
  float o[4][CW];
#pragma unroll
  for (int i = 0; i < 4; i++)
#pragma unroll
    for (int k = 0; k < CW; k++) o[i][k] = 0.f;
  if (PRELOAD) {
    cp_async_wait<0>();
    __syncthreads();   // the matrices have landed and vec is complete
  } else {
    if (sm.TSC_IN_RING) __syncthreads();   // everyone has read its softmax numerators: the ring takes matrices now
    if (!comp)
      for (int pre = 0; pre < CB_NBUF - 1; pre++) stage(pre);
  }
  for (int chunk = 0; chunk < N_CHUNK; chunk++) {
    if (!PRELOAD) {
      if (!comp) cp_async_wait<CB_NBUF - 2>();
      __syncthreads();   // slice `chunk` has landed; everyone is done with slice chunk-1 (and, first time, vec is complete)
    }
    if (!comp) {
      if (!PRELOAD) stage(chunk + CB_NBUF - 1);   // into the buffer of slice chunk-1
    } else if (!PRE || (chunk & 1) == khalf) {
      const int m = chunk / (D / CB_CHUNK), r0 = (chunk % (D / CB_CHUNK)) * CB_CHUNK;
      const float* rb = rbuf + (PRELOAD ? chunk : chunk % CB_NBUF) * CB_CHUNK * SW;
#pragma unroll 2
      for (int r = 0; r < CB_CHUNK; r += 4) {
        float4 x[4];
#pragma unroll
        for (int i = 0; i < 4; i++) x[i] = *reinterpret_cast<const float4*>(&sm.vec[m][rw + i][r0 + r]);
        if (NS == 1) {
          float4 rr[4];
#pragma unroll
          for (int k = 0; k < 4; k++) rr[k] = *reinterpret_cast<const float4*>(&rb[(r + k) * SW + cl]);
#pragma unroll
          for (int i = 0; i < 4; i++) {
            o[i][0] = fmaf(rr[0].x, x[i].x, o[i][0]); o[i][1 % CW] = fmaf(rr[0].y, x[i].x, o[i][1 % CW]);
            o[i][2 % CW] = fmaf(rr[0].z, x[i].x, o[i][2 % CW]); o[i][3 % CW] = fmaf(rr[0].w, x[i].x, o[i][3 % CW]);
            o[i][0] = fmaf(rr[1].x, x[i].y, o[i][0]); o[i][1 % CW] = fmaf(rr[1].y, x[i].y, o[i][1 % CW]);
            o[i][2 % CW] = fmaf(rr[1].z, x[i].y, o[i][2 % CW]); o[i][3 % CW] = fmaf(rr[1].w, x[i].y, o[i][3 % CW]);
            o[i][0] = fmaf(rr[2].x, x[i].z, o[i][0]); o[i][1 % CW] = fmaf(rr[2].y, x[i].z, o[i][1 % CW]);
            o[i][2 % CW] = fmaf(rr[2].z, x[i].z, o[i][2 % CW]); o[i][3 % CW] = fmaf(rr[2].w, x[i].z, o[i][3 % CW]);
            o[i][0] = fmaf(rr[3].x, x[i].w, o[i][0]); o[i][1 % CW] = fmaf(rr[3].y, x[i].w, o[i][1 % CW]);
            o[i][2 % CW] = fmaf(rr[3].z, x[i].w, o[i][2 % CW]); o[i][3 % CW] = fmaf(rr[3].w, x[i].w, o[i][3 % CW]);
          }
        } else {   // one column per thread
          const float r0v = rb[(r + 0) * SW + cl], r1v = rb[(r + 1) * SW + cl], r2v = rb[(r + 2) * SW + cl], r3v = rb[(r + 3) * SW + cl];
#pragma unroll
          for (int i = 0; i < 4; i++)
            o[i][0] = fmaf(r3v, x[i].w, fmaf(r2v, x[i].z, fmaf(r1v, x[i].y, fmaf(r0v, x[i].x, o[i][0]))));
        }
      }
    }
  }
  if (PRE) {   // the second half's sums reach the first through the tail-score array, idle by now
    float* red = &sm.tsc_own[0] + (threadIdx.x % (CB_SEQ * 64)) * 4 * CW;
    static_assert(!PRE || CB_SEQ * 64 * 4 * CW <= CB_SEQ * W * GP, "reduction scratch");
    if (khalf) {
#pragma unroll
      for (int i = 0; i < 4; i++)
#pragma unroll
        for (int k = 0; k < CW; k++) red[i * CW + k] = o[i][k];
    }
    __syncthreads();
    if (!khalf) {
#pragma unroll
      for (int i = 0; i < 4; i++)
#pragma unroll
        for (int k = 0; k < CW; k++) o[i][k] += red[i * CW + k];
    }
  }
  if (comp && !khalf) {
#pragma unroll
    for (int i = 0; i < 4; i++) {
      const int row = rw + i, ob = blockIdx.y * CB_SEQ + row / GP, j = row % GP;
      if (ob >= cv.batch || j >= G) continue;
      const float L = sm.Ls[row / GP][j];
      const float inv = L > 0.f ? 1.0f / L : 0.f;
      float* dst = &P.out[(((size_t)li * cv.batch + ob) * cv.n_q_heads + h * G + j) * D + sl * SW + cl];
      if (NS == 1) {
        const float4 rv = *reinterpret_cast<const float4*>(&sm.rawv[row][cl]);
        *reinterpret_cast<float4*>(dst) = make_float4((o[i][0] + rv.x) * inv, (o[i][1 % CW] + rv.y) * inv,
                                                      (o[i][2 % CW] + rv.z) * inv, (o[i][3 % CW] + rv.w) * inv);
      } else {
        dst[0] = (o[i][0] + sm.rawv[row][sl * SW + cl]) * inv;
      }
    }
  }
}

template <bool CAPTION, int NS, int SEQ>
static cudaError_t combine_attr() {
  return cudaFuncSetAttribute(k_combine_mma<CAPTION, NS, SEQ>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)sizeof(CombineSmem<CAPTION, SEQ>));
}

template <bool CAPTION, int NS, int SEQ>
static void combine_launch(const DecodeParams& P, int n_cta, cudaStream_t s) {
  const dim3 grid(P.cv.n_kv_heads * NS, (P.cv.batch + SEQ - 1) / SEQ, P.layer_count);
  k_combine_mma<CAPTION, NS, SEQ><<<grid, SEQ * 128, sizeof(CombineSmem<CAPTION, SEQ>), s>>>(P, n_cta);
}

template <bool CAPTION>
static void combine_dispatch(const DecodeParams& P, int n_cta, cudaStream_t s) {
  // full grids: four sequences per block, so that a layer's matrices are streamed once per four sequences;
  // fewer such blocks than SMs: one sequence per block; a handful (e.g. a single-layer call): one sequence
  // and a quarter of the output columns per block
  const int n_blocks = P.cv.n_kv_heads * ((P.cv.batch + CB_SEQ_MAX - 1) / CB_SEQ_MAX) * P.layer_count;
  if (4 * n_blocks <= n_cta) combine_launch<CAPTION, 4, 1>(P, n_cta, s);
  else if (n_blocks <= n_cta) combine_launch<CAPTION, 1, 1>(P, n_cta, s);
  else combine_launch<CAPTION, 1, CB_SEQ_MAX>(P, n_cta, s);
}

int g_decode_impl = 1;

okq_status launch_decode_mma(const DecodeParams& P, int n_cta, cudaStream_t s, cudaEvent_t before, cudaEvent_t after) {
  static thread_local unsigned long long attr_mask = 0;
  int attr_dev = 0;
  if (attr_needed(attr_mask, attr_dev)) {
    cudaError_t e = cudaFuncSetAttribute(k_decode_mma<FMT_FP16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)sizeof(MmaSmem<FMT_FP16>));
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(k_decode_mma<FMT_MXFP4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)sizeof(MmaSmem<FMT_MXFP4>));
    if (e == cudaSuccess) e = combine_attr<false, 4, 1>();
    if (e == cudaSuccess) e = combine_attr<false, 1, 1>();
    if (e == cudaSuccess) e = combine_attr<false, 1, CB_SEQ_MAX>();
    if (e == cudaSuccess) e = combine_attr<true, 4, 1>();
    if (e == cudaSuccess) e = combine_attr<true, 1, 1>();
    if (e == cudaSuccess) e = combine_attr<true, 1, CB_SEQ_MAX>();
    if (e != cudaSuccess) { set_last_cuda_error((int)e); return OKQ_ERR_CUDA; }
    attr_done(attr_mask, attr_dev);
  }
  if (before) cudaEventRecord(before, s);
  if (P.cv.fmt == FMT_FP16 && g_decode_impl == 0) {
    const okq_status st = launch_decode_tc(P, n_cta, s);
    if (st != OKQ_OK) return st;
  } else if (P.cv.fmt == FMT_MXFP4) k_decode_mma<FMT_MXFP4><<<n_cta, NTHREADS, sizeof(MmaSmem<FMT_MXFP4>), s>>>(P);
  else k_decode_mma<FMT_FP16><<<n_cta, NTHREADS, sizeof(MmaSmem<FMT_FP16>), s>>>(P);
  if (after) cudaEventRecord(after, s);
  if (P.cv.sched == SCHED_CAPTION) combine_dispatch<true>(P, n_cta, s);
  else combine_dispatch<false>(P, n_cta, s);
  return OKQ_OK;
}

}  // namespace okq
