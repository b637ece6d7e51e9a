// Fused decode attention over the packed cache, split-K kernel on the 5th-generation tensor cores
// (tcgen05.mma with the unpacked codes as the A operand in tensor memory).
//
// Per (sequence, KV head) the scores and the value sums of the GQA group are the contractions
//     S[token][head]     = C_k[token][channel] * W[channel][head]        (per 32-token window, Eq. 4 in the rotated space)
//     O[channel][head]  += C_v[channel][token] * P[token][head]          (Eq. 1, values in their modality's rotated basis)
// The kernel works on "super-windows" of four consecutive windows (128 tokens = the 128 lanes of tensor memory):
//   * key codes:   a thread owns one token, masks the 2-bit fields out of its eight code words (a masked field is the
//                  fp16 subnormal code * 4^j * 2^-24, so unpacking is one AND per two codes) and writes them to tensor
//                  memory with tcgen05.st: A = [128 tokens x 128 channels];
//   * weights:     W = q'_c * s_gc (rotated query times the window's step, split into an fp16 high and low part, the
//                  4^j of the matching code field divided out) goes to shared memory as the B operand
//                  [64 = 4 windows x 2 head halves x (4 heads hi, 4 heads lo)] x [128 channels]; eight tcgen05.mma
//                  (M 128, N 64, K 16) give every token its scores against the four windows' weights, of which it reads
//                  its own window's; the bias sum_c q'_c m_gc comes from eight mma.sync per window in the same warp;
//   * softmax:     a thread owns one token and four heads (tcgen05.ld of its 8 score columns), keeps a reference maximum
//                  per head that only moves at flush points, and writes the fp16 numerators p * |v| * 2 / 4^j as the B
//                  operand [32 tokens x 16] of the value product, one tile per modality present in the window;
//   * value codes: a thread owns one channel, masks its 32 tokens' fields (code plane and bit-1 plane: the codebook
//                  {-b,-a,a,b} is affine in (code, bit 1)) into tensor memory: A = [128 channels x 32 tokens] x 2 planes;
//                  four tcgen05.mma (M 128, N 16, K 16) per window and modality add into the modality's accumulators,
//                  which stay in tensor memory;
//   * flush:       every eight super-windows (the tensor cores' fp32 accumulation does not round to nearest; short
//                  chains summed with FFMA keep the drift out), when a score exceeds the reference by more than 2^8,
//                  and at the end of a (sequence, head), the accumulators are added to running sums in shared memory
//                  under the then-current reference; at the end of a (sequence, head) the sums leave as one PartialF.
// Roles (warps): 0-3 key codes, 4-7 weights, 8-15 softmax (window q = warp & 3, heads 4 (warp >> 2 & 1) ..), 16-23 value
// codes (even / odd windows), 24-27 flush, 28 loader (one bulk copy of a super-window's records; the stored order of the
// 16-byte pieces of the code blocks makes the unpacking reads free of bank conflicts), 29 score MMA issue, 30 value MMA issue.  They meet only at
// mbarriers; every wait is bounded and ends in OKQ_ERR_TIMEOUT.
// The grid is persistent: CTA i owns an equal slice of the flattened (layer, sequence, head, window) axis, the same
// partition the combine kernel assumes (one PartialF per (CTA, (sequence, head)) overlap, slot = unit + CTA index).
#include "okq_common.cuh"
#include "okq_device.cuh"
#include "okq_decode_shared.cuh"
#include "okq_decode_frag.cuh"

namespace okq {

namespace {

constexpr int TC_WARPS = 31, TC_THREADS = TC_WARPS * 32;
constexpr int WARP_K = 0, WARP_W = 4, WARP_SM = 8, WARP_V = 16, WARP_FL = 24, WARP_LD = 28, WARP_MMA_S = 29, WARP_MMA_V = 30;
constexpr int SWW = 4;                          // windows per super-window
constexpr int NST = 6;                          // staged super-windows
constexpr int STG_WIN = RECORD_BYTES;           // staged window: the record as it is stored
constexpr int STG_MOD = SWW * STG_WIN;          // the super-window's modality bytes
constexpr int STG_BYTES = STG_MOD + SWW * W;
constexpr int BW_LBO = 160;                     // bytes between 8-channel chunks of the weight operand (128 + 32: the
                                                // weight warps' 16-byte stores then hit eight different bank groups)
constexpr int BW_SBO = 16 * BW_LBO;             // bytes between 8-row groups
constexpr int BW_BYTES = 8 * BW_SBO;            // N = 64 rows
constexpr int NBIAS = 4;                        // ring of bias / scale records (super-windows)
constexpr int NAV = 6;                          // value-code / numerator ring (windows)
constexpr int BP_TILE = 1024;                   // numerators of one window and modality: [4 token blocks][2 head blocks][128 B]
constexpr int NREQ = 8;                         // flush requests in flight
constexpr int FLUSH_SWS = 8;                    // super-windows accumulated in tensor memory at most
constexpr float T_LOG2 = 8.0f;                  // a score may exceed the reference maximum by this much (log2)
constexpr int C_LOG2 = 1;                       // numerators carry 2^C_LOG2: p <= 2^8, |v| < 128 stay below the fp16 maximum
// tensor-memory columns: key codes (two buffers), scores, value codes (NAV windows x two planes), accumulators
constexpr uint32_t AK_COL = 0, S_COL = 128, AV_COL = 192, ACC_COL = 384;
static_assert(AV_COL + 32 * NAV <= ACC_COL && ACC_COL + 96 <= 512, "tensor memory columns");
constexpr long long WAIT_LIMIT_CLOCKS = 4000000000ll;   // about two seconds of SM clocks

#ifdef OKQ_TC_TIMELINE
__device__ long long g_tl[8 * 64 * 8];
#define TL(role, sw, ev) do { if (blockIdx.x == 0 && lane == 0 && (sw) < 64) g_tl[((role) * 64 + (sw)) * 8 + (ev)] = clock64(); } while (0)
#else
#define TL(role, sw, ev) do { } while (0)
#endif

struct FlushReq {
  float m_period[GP];   // reference maximum the accumulators in tensor memory refer to
  float l[GP];          // end of a (sequence, head): sum of exp2(score - m_period)
  float S[3][GP];       // end of a (sequence, head): per modality sum of p * |v|
  int touched;          // modalities accumulated since the last flush (bit m)
  int seg_end;          // non-zero: write the PartialF record `pidx` and start afresh
  int pidx, pad;
};

struct TcSmem {
  __align__(128) unsigned char stage[NST][STG_BYTES];
  __align__(128) unsigned char bw[2][BW_BYTES];
  __align__(128) unsigned char bp[NAV][3][BP_TILE];
  __align__(16) float sums[3][GP][D];           // running sums [modality][head][channel] of plane0 + drel * plane1
  __align__(16) float bias[NBIAS][SWW][GP];
  __align__(16) float fsc[NBIAS][GP];
  __align__(16) float wmax[2][SWW][GP];
  __align__(16) float mold[2][GP];
  __align__(16) float lred[SWW][GP];
  __align__(16) float Sred[SWW][3][GP];
  __align__(16) FlushReq req[NREQ];
  __align__(16) int ovf[2][2 * SWW];
  __align__(16) int touched_w[2][SWW];
  int bp_present[NAV], bp_flush[NAV];
  __align__(8) unsigned long long stage_full[NST], stage_free[NST], ak_full[2], bw_full[2], ab_free[2], s_full, s_free;
  __align__(8) unsigned long long av_full[NAV], bp_full[NAV], v_done[NAV], req_full[NREQ];
  __align__(8) unsigned long long flush_ready, acc_free, sm_sync;
  uint32_t tmem_slot;
  volatile int abort;
  int prefix[MAX_ENTRIES + 1];
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t mbar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
               : "=r"(ok) : "r"(mbar), "r"(parity) : "memory");
  return ok != 0;
}
// Up to 64 tries in a loop of two instructions (a try suspends the thread until the phase completes or a short,
// system-chosen time has passed): a waiting warp must not take issue slots and ALU cycles from the working ones.
__device__ __forceinline__ bool mbar_try64(uint32_t mbar, uint32_t parity) {
  bool ok = false;
#pragma unroll 1
  for (int i = 0; i < 64 && !ok; i++) {
    ok = mbar_try(mbar, parity);
#ifdef OKQ_TC_SLEEP
    if (!ok) __nanosleep(OKQ_TC_SLEEP);
#endif
  }
  return ok;
}
// Bounded wait of a whole warp for one phase of an mbarrier; gives up after about two seconds or soon after another
// role has given up, and raises the abort flag.  The clock and the flag are looked at every 64th try only.
__device__ __noinline__ bool mbar_wait_slow(TcSmem& sm, uint32_t mbar, uint32_t parity) {
  const long long t0 = clock64();
  bool done = false;
  while (!done) {
    done = mbar_try64(mbar, parity);
    if (!done && (sm.abort || clock64() - t0 > WAIT_LIMIT_CLOCKS)) break;
  }
  if (!done) sm.abort = 1;
  return __all_sync(0xffffffffu, done);
}
__device__ __forceinline__ bool mbar_wait(TcSmem& sm, unsigned long long* bar, uint32_t parity) {
  const uint32_t mbar = smem_u32(bar);
  if (__all_sync(0xffffffffu, mbar_try(mbar, parity))) return true;
  return mbar_wait_slow(sm, mbar, parity);
}

__device__ __forceinline__ void fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }

__device__ __forceinline__ bool elect_one() {
  uint32_t pred = 0;
  asm volatile("{\n\t.reg .b32 rx;\n\t.reg .pred px;\n\telect.sync rx|px, 0xffffffff;\n\tselp.u32 %0, 1, 0, px;\n\t}\n" : "=r"(pred));
  return pred != 0;
}

// shared-memory matrix descriptor, no swizzle: `lbo` bytes between 8-element chunks along K (K-major operand) or
// between 8-row blocks along K (MN-major operand), `sbo` bytes between 8-row groups along M/N
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((saddr >> 4) & 0x3fff) | ((uint64_t)((lbo >> 4) & 0x3fff) << 16) |
         ((uint64_t)((sbo >> 4) & 0x3fff) << 32) | ((uint64_t)1 << 46);
}
// D[tmem] = A[tmem] * B[smem] (ACC false) or D += A * B (ACC true), fp16 operands, fp32 accumulation
template <bool ACC>
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a, uint64_t bdesc, uint32_t idesc) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}\n"
               ::"r"(d), "r"(a), "l"(bdesc), "r"(idesc), "n"(ACC ? 1 : 0) : "memory");
}
__device__ __forceinline__ void mma_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
                 "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
                 "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]),
                 "r"(r[30]), "r"(r[31]) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr) : "memory");
}

// A CTA's walk over its slice of the flattened window axis: consecutive pieces ("segments"), each inside one
// (layer, sequence, head) unit.  Every role walks the same sequence.
struct Seg {
  int e, h, w0, n_my, unit;
};
struct SegWalk {
  const int* prefix;
  int n_entries, Hkv, pos, pos_end;
  __device__ __forceinline__ bool next(Seg& s) {
    if (pos >= pos_end) return false;
    int lo = 0, hi = n_entries;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (prefix[mid] <= pos) lo = mid; else hi = mid;
    }
    const int nwin = (prefix[lo + 1] - prefix[lo]) / Hkv;
    const int off = pos - prefix[lo];
    s.e = lo;
    s.h = off / nwin;
    s.w0 = off % nwin;
    s.n_my = min(pos_end - pos, nwin - s.w0);
    s.unit = lo * Hkv + s.h;
    pos += s.n_my;
    return true;
  }
};

}  // namespace

// grid = n_cta (persistent), TC_THREADS threads
__global__ void __launch_bounds__(TC_THREADS, 1) k_decode_tc(DecodeParams P) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  TcSmem& sm = *reinterpret_cast<TcSmem*>(smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u));
  const CacheView& cv = P.cv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = P.group, Hkv = cv.n_kv_heads;
  const int n_entries = P.layer_count * cv.batch;

  // ---- set-up: barriers, tensor memory, the zero halves of the numerator tiles, the partition
  if (tid == 0) {
    for (int i = 0; i < NST; i++) { mbar_init(&sm.stage_full[i], 1); mbar_init(&sm.stage_free[i], 24); }
    for (int i = 0; i < 2; i++) { mbar_init(&sm.ak_full[i], 4); mbar_init(&sm.bw_full[i], 4); mbar_init(&sm.ab_free[i], 1); }
    mbar_init(&sm.s_full, 1); mbar_init(&sm.s_free, 8);
    for (int i = 0; i < NAV; i++) { mbar_init(&sm.av_full[i], 4); mbar_init(&sm.bp_full[i], 2); mbar_init(&sm.v_done[i], 1); }
    for (int i = 0; i < NREQ; i++) mbar_init(&sm.req_full[i], 1);
    mbar_init(&sm.flush_ready, 1); mbar_init(&sm.acc_free, 4); mbar_init(&sm.sm_sync, 8);
    sm.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;\n" ::"r"(smem_u32(&sm.tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  for (int i = tid; i < NAV * 3 * BP_TILE / 16; i += TC_THREADS) reinterpret_cast<uint4*>(&sm.bp[0][0][0])[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_async_smem();
  const int total = block_prefix(cv, P.layer0, n_entries, sm.prefix);   // ends in __syncthreads
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = sm.tmem_slot;
  const int per = (total + gridDim.x - 1) / gridDim.x;
  const int pos0 = min(total, (int)blockIdx.x * per), pos1 = min(total, pos0 + per);
  auto walker = [&]() {
    SegWalk w;
    w.prefix = sm.prefix; w.n_entries = n_entries; w.Hkv = Hkv; w.pos = pos0; w.pos_end = pos1;
    return w;
  };

  if (warp == WARP_LD) {
    // ------------------------------------------------------------------ loader
    SegWalk walk = walker();
    Seg sg;
    int n = 0;
    bool alive = true;
    while (alive && walk.next(sg)) {
      const int li = sg.e / cv.batch, b = sg.e % cv.batch;
      const unsigned char* rec0 = cv.unit(P.layer0 + li, b, sg.h);
      const unsigned char* mod0 = cv.modality + (size_t)b * cv.capacity;
      const int nsw = (sg.n_my + SWW - 1) / SWW;
      for (int i = 0; i < nsw; i++, n++) {
        const int st = n % NST, use = n / NST;
        if (use >= 1 && !mbar_wait(sm, &sm.stage_free[st], (uint32_t)(use - 1) & 1u)) { alive = false; break; }
        TL(0, n, 0);
        const int n_w = min(SWW, sg.n_my - SWW * i), win0 = sg.w0 + SWW * i;
        if (lane == 0) {
          // two bulk copies: the super-window's records (contiguous) and its modality bytes
          const uint32_t bar = smem_u32(&sm.stage_full[st]), dst = smem_u32(sm.stage[st]);
          const uint32_t nrec = (uint32_t)(n_w * RECORD_BYTES), nmod = (uint32_t)(n_w * W);
          asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(nrec + nmod) : "memory");
          asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                       ::"r"(dst), "l"(rec0 + (size_t)win0 * RECORD_BYTES), "r"(nrec), "r"(bar) : "memory");
          asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                       ::"r"(dst + (uint32_t)STG_MOD), "l"(mod0 + (size_t)win0 * W), "r"(nmod), "r"(bar) : "memory");
        }
        __syncwarp();
        TL(0, n, 1);
      }
    }
  } else if (warp < WARP_W) {
    // ------------------------------------------------------------------ key codes -> tensor memory
    // lane L holds the token with norm position L (i = 8 nu + 2 t' + e', L = 8 t' + 2 nu + e'); its eight code words
    // are the 8-byte halves (nu & 1) of the pieces (a = nu >> 1, g = i & 7, t), t = 0..3
    const int q = warp - WARP_K;
    const int tp = lane >> 3, nu = (lane >> 1) & 3, ep = lane & 1;
    const int g = 2 * tp + ep;
    uint32_t koff[4];   // the lane's 8-byte half of its piece (a = nu >> 1, g, t), t = 0..3
#pragma unroll
    for (int t = 0; t < 4; t++) koff[t] = OFF_KCODE + 16 * kpiece_slot(32 * (nu >> 1) + 4 * g + t) + 8 * (nu & 1);
    SegWalk walk = walker();
    Seg sg;
    int n = 0;
    bool alive = true;
    while (alive && walk.next(sg)) {
      const int nsw = (sg.n_my + SWW - 1) / SWW;
      for (int i = 0; i < nsw; i++, n++) {
        const int st = n % NST, buf = n & 1;
        const int n_w = min(SWW, sg.n_my - SWW * i);
        if (!mbar_wait(sm, &sm.stage_full[st], (uint32_t)(n / NST) & 1u)) { alive = false; break; }
        if (q == 0) TL(1, n, 0);
        uint2 w[4];
        if (q < n_w) {
          const unsigned char* base = sm.stage[st] + q * STG_WIN;
#pragma unroll
          for (int t = 0; t < 4; t++) w[t] = *reinterpret_cast<const uint2*>(base + koff[t]);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.stage_free[st]);   // the code words are in registers
        if (n >= 2 && !mbar_wait(sm, &sm.ab_free[buf], (uint32_t)((n >> 1) - 1) & 1u)) { alive = false; break; }
        fence_after();
        if (q == 0) TL(1, n, 1);
        if (q < n_w) {
#pragma unroll
          for (int ww = 0; ww < 2; ww++) {
            // register r = 8 ww + 4 sh + j of word t: channels at K index 8 t + 32 (2 ww + sh) + 2 j + {0, 1}
            uint32_t r[32];
#pragma unroll
            for (int t = 0; t < 4; t++) {
              const uint32_t lo = ww ? w[t].y : w[t].x, hi = lo >> 8;
#pragma unroll
              for (int j = 0; j < 4; j++) {
                r[4 * t + j] = lo & (0x00030003u << (2 * j));
                r[16 + 4 * t + j] = hi & (0x00030003u << (2 * j));
              }
            }
            tmem_st32(tmem + ((uint32_t)(32 * q) << 16) + AK_COL + 64u * buf + 32u * ww, r);
          }
          if (q == 0) TL(1, n, 2);
          tmem_wait_st();
        }
        fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.ak_full[buf]);
        if (q == 0) TL(1, n, 3);
      }
    }
  } else if (warp < WARP_SM) {
    // ------------------------------------------------------------------ weights W = q' s (hi, lo) and the bias
    // lane (g, t): head g, K chunks t + 4 i (positions 32 t + 8 i .. + 7 of the (m, s) planes); row of the operand:
    // 16 window + 8 (g >> 2) + (g & 3) for the high part, + 4 for the low part
    const int wq = warp - WARP_W;
    const int g = lane >> 2, t = lane & 3;
    SegWalk walk = walker();
    Seg sg;
    int n = 0;
    bool alive = true;
    while (alive && walk.next(sg)) {
      const int li = sg.e / cv.batch, b = sg.e % cv.batch;
      uint2 qreg[16];
      float fsc;
      query_fragments(P.q + (((size_t)li * cv.batch + b) * cv.n_q_heads + (size_t)sg.h * G) * D, P.signs + (size_t)li * D, G,
                      P.sm_scale, lane, qreg, fsc);
      const int nsw = (sg.n_my + SWW - 1) / SWW;
      for (int i = 0; i < nsw; i++, n++) {
        const int st = n % NST, buf = n & 1, nb = n % NBIAS;
        const int n_w = min(SWW, sg.n_my - SWW * i);
        if (!mbar_wait(sm, &sm.stage_full[st], (uint32_t)(n / NST) & 1u)) { alive = false; break; }
        // the buffer's previous weights have been consumed (their products are complete)
        if (n >= 2 && !mbar_wait(sm, &sm.ab_free[buf], (uint32_t)((n >> 1) - 1) & 1u)) { alive = false; break; }
        if (wq == 0) TL(2, n, 0);
        if (wq < n_w) {
          const unsigned char* swin = sm.stage[st] + wq * STG_WIN;
          const uint4* sp = reinterpret_cast<const uint4*>(swin + OFF_KS + 64 * t);
          const uint4* mp = reinterpret_cast<const uint4*>(swin + OFF_KM + 64 * t);
          unsigned char* bhi = sm.bw[buf] + (2 * wq + (g >> 2)) * BW_SBO + t * BW_LBO + (g & 3) * 16;
          float dbA[4] = {0.f, 0.f, 0.f, 0.f}, dbB[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int i4 = 0; i4 < 4; i4++) {
            const uint4 s4 = sp[i4], m4 = mp[i4];
            const uint2 q0 = qreg[4 * i4], q1 = qreg[4 * i4 + 1], q2 = qreg[4 * i4 + 2], q3 = qreg[4 * i4 + 3];
            mma16816(dbA, q0.x, q0.y, q1.x, q1.y, m4.x, m4.y);
            mma16816(dbB, q2.x, q2.y, q3.x, q3.y, m4.z, m4.w);
            uint4 hi, lo;
            split_product(u2h(q0.x), u2h(q0.y), u2h(s4.x), hi.x, lo.x);
            split_product(u2h(q1.x), u2h(q1.y), u2h(s4.y), hi.y, lo.y);
            split_product(u2h(q2.x), u2h(q2.y), u2h(s4.z), hi.z, lo.z);
            split_product(u2h(q3.x), u2h(q3.y), u2h(s4.w), hi.w, lo.w);
            *reinterpret_cast<uint4*>(bhi + 4 * i4 * BW_LBO) = hi;
            *reinterpret_cast<uint4*>(bhi + 4 * i4 * BW_LBO + 64) = lo;
          }
          // the code sums carry 2^-24 (subnormal code operands), the bias sum does not
          if (t == 0) sm.bias[nb][wq][g] = ((dbA[0] + dbB[0]) + (dbA[2] + dbB[2])) * 0x1p-24f;
          if (wq == 0 && t == 0) sm.fsc[nb][g] = fsc;
        }
        if (wq == 0) TL(2, n, 2);
        fence_async_smem();
        if (wq == 0) TL(2, n, 3);
        __syncwarp();
        if (lane == 0) { mbar_arrive(&sm.bw_full[buf]); mbar_arrive(&sm.stage_free[st]); }
        if (wq == 0) TL(2, n, 1);
      }
    }
  } else if (warp == WARP_MMA_S) {
    // ------------------------------------------------------------------ score MMAs
    constexpr uint32_t idesc = (1u << 4) | ((64u >> 3) << 17) | ((128u >> 4) << 24);   // D fp32, A/B fp16, B K-major, N 64, M 128
    const uint64_t bdb0 = make_desc(smem_u32(sm.bw[0]), BW_LBO, BW_SBO), bdb1 = make_desc(smem_u32(sm.bw[1]), BW_LBO, BW_SBO);
    const uint32_t tmem_u = __reduce_or_sync(0xffffffffu, tmem);
    SegWalk walk = walker();
    Seg sg;
    int n = 0;
    bool alive = true;
    while (alive && walk.next(sg)) {
      const int nsw = (sg.n_my + SWW - 1) / SWW;
      for (int i = 0; i < nsw; i++, n++) {
        const int buf = n & 1;
        const uint32_t par = (uint32_t)(n >> 1) & 1u;
        if (!mbar_wait(sm, &sm.ak_full[buf], par) || !mbar_wait(sm, &sm.bw_full[buf], par)) { alive = false; break; }
        if (n >= 1 && !mbar_wait(sm, &sm.s_free, (uint32_t)(n - 1) & 1u)) { alive = false; break; }
        fence_after();
        TL(3, n, 0);
        if (elect_one()) {
          if (buf == 0) {
            mma_ts<false>(tmem_u + S_COL, tmem_u + AK_COL, bdb0, idesc);
#pragma unroll
            for (int ks = 1; ks < 8; ks++) mma_ts<true>(tmem_u + S_COL, tmem_u + AK_COL + 8u * ks, bdb0 + (uint64_t)((2 * ks * BW_LBO) >> 4), idesc);
            mma_commit(&sm.s_full);
            mma_commit(&sm.ab_free[0]);
          } else {
            mma_ts<false>(tmem_u + S_COL, tmem_u + AK_COL + 64u, bdb1, idesc);
#pragma unroll
            for (int ks = 1; ks < 8; ks++) mma_ts<true>(tmem_u + S_COL, tmem_u + AK_COL + 64u + 8u * ks, bdb1 + (uint64_t)((2 * ks * BW_LBO) >> 4), idesc);
            mma_commit(&sm.s_full);
            mma_commit(&sm.ab_free[1]);
          }
        }
        __syncwarp();
        TL(3, n, 1);
      }
    }
  } else if (warp < WARP_V) {
    // ------------------------------------------------------------------ softmax
    // warp (window wq, head half hh): lane = token row, heads 4 hh .. 4 hh + 3
    const int wq = (warp - WARP_SM) & 3, hh = (warp - WARP_SM) >> 2;
    const int tok = 8 * ((lane >> 1) & 3) + 2 * (lane >> 3) + (lane & 1);   // token of the window this lane owns
    const int jpos = (lane >> 1) & 3;                                      // its field index in the value-code words
    const float pscale = exp2f((float)(C_LOG2 - 2 * jpos)), sinv = exp2f((float)(2 * jpos - C_LOG2));
    constexpr int HH = GP / 2;
    float m_ref[HH], l[HH], Sm[3][HH];
    SegWalk walk = walker();
    Seg sg;
    int n = 0, x0 = 0, gs = 0, nreq = 0, seg_idx = 0;
    bool alive = true;
    auto group_sync = [&]() -> bool {   // the eight softmax warps meet; data written before is visible after
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.sm_sync);
      const bool ok = mbar_wait(sm, &sm.sm_sync, (uint32_t)gs & 1u);
      gs++;
      return ok;
    };
    while (alive && walk.next(sg)) {
#pragma unroll
      for (int h = 0; h < HH; h++) { m_ref[h] = -INFINITY; l[h] = 0.f; Sm[0][h] = Sm[1][h] = Sm[2][h] = 0.f; }
      int touched = 0, period = 0;
      const int nsw = (sg.n_my + SWW - 1) / SWW;
      for (int i = 0; i < nsw && alive; i++, n++) {
        const int st = n % NST, nb = n % NBIAS;
        const int n_w = min(SWW, sg.n_my - SWW * i);
        const bool valid = wq < n_w;
        if (wq == 0 && hh == 0) TL(4, n, 0);
        if (!mbar_wait(sm, &sm.s_full, (uint32_t)n & 1u)) { alive = false; break; }
        fence_after();
        if (wq == 0 && hh == 0) TL(4, n, 1);
        float x[HH];
        uint32_t r[8];
        if (valid) {
          tmem_ld8(tmem + ((uint32_t)(32 * wq) << 16) + S_COL + 16u * wq + 8u * hh, r);
          tmem_wait_ld();
        }
        fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.s_free);   // the scores are in registers
        const unsigned char* swin = sm.stage[st] + wq * STG_WIN;
        bool ovl = false;
        if (valid) {
          if (!mbar_wait(sm, &sm.stage_full[st], (uint32_t)(n / NST) & 1u)) { alive = false; break; }
          const float kn = __half2float(reinterpret_cast<const __half*>(swin + OFF_KNORM)[lane]);
          const float4 b4 = *reinterpret_cast<const float4*>(&sm.bias[nb][wq][HH * hh]);
          const float4 f4 = *reinterpret_cast<const float4*>(&sm.fsc[nb][HH * hh]);
          const float bs[HH] = {b4.x, b4.y, b4.z, b4.w}, fs[HH] = {f4.x, f4.y, f4.z, f4.w};
#pragma unroll
          for (int h = 0; h < HH; h++) {
            x[h] = ((__uint_as_float(r[h]) + __uint_as_float(r[HH + h])) + bs[h]) * (kn * fs[h]);
            ovl |= x[h] > m_ref[h] + T_LOG2;
          }
        }
        // do the eight warps agree to keep the reference maximum?
        const bool force = i == 0 || period >= FLUSH_SWS;
        const int wovl = __any_sync(0xffffffffu, ovl);
        int par = gs & 1;
        if (lane == 0) { sm.ovf[par][4 * hh + wq] = wovl; if (hh == 0) sm.touched_w[par][wq] = touched; }
        if (wq == 0 && hh == 0) TL(4, n, 2);
        if (!group_sync()) { alive = false; break; }
        if (wq == 0 && hh == 0) TL(4, n, 3);
        const int4 o0 = *reinterpret_cast<const int4*>(&sm.ovf[par][0]), o1 = *reinterpret_cast<const int4*>(&sm.ovf[par][4]);
        const int4 tw = *reinterpret_cast<const int4*>(&sm.touched_w[par][0]);
        const bool need = force || (o0.x | o0.y | o0.z | o0.w | o1.x | o1.y | o1.z | o1.w) != 0;
        bool flag = false;
        if (need) {
          // new reference: the maximum seen so far, this super-window included
          float wm[HH];
#pragma unroll
          for (int h = 0; h < HH; h++) wm[h] = valid ? x[h] : -INFINITY;
#pragma unroll
          for (int d = 1; d < 32; d <<= 1)
#pragma unroll
            for (int h = 0; h < HH; h++) wm[h] = fmaxf(wm[h], __shfl_xor_sync(0xffffffffu, wm[h], d));
          par = gs & 1;
          if (lane < HH) {
            float v = wm[0], mo = m_ref[0];
#pragma unroll
            for (int h = 1; h < HH; h++) { v = lane == h ? wm[h] : v; mo = lane == h ? m_ref[h] : mo; }
            sm.wmax[par][wq][HH * hh + lane] = v;
            if (wq == 0) sm.mold[par][HH * hh + lane] = mo;
          }
          if (!group_sync()) { alive = false; break; }
          if (i > 0) {   // what tensor memory holds refers to the old reference: have it flushed before this super-window
            if (wq == 0 && hh == 0 && lane == 0) {
              FlushReq& rq = sm.req[nreq % NREQ];
              *reinterpret_cast<float4*>(&rq.m_period[0]) = *reinterpret_cast<const float4*>(&sm.mold[par][0]);
              *reinterpret_cast<float4*>(&rq.m_period[4]) = *reinterpret_cast<const float4*>(&sm.mold[par][4]);
              rq.touched = tw.x | tw.y | tw.z | tw.w; rq.seg_end = 0; rq.pidx = 0;
              __threadfence_block();
              mbar_arrive(&sm.req_full[nreq % NREQ]);
            }
            nreq++;
            flag = true;
          }
#pragma unroll
          for (int h = 0; h < HH; h++) {
            const int hg = HH * hh + h;
            const float mn = fmaxf(fmaxf(m_ref[h], fmaxf(sm.wmax[par][0][hg], sm.wmax[par][1][hg])), fmaxf(sm.wmax[par][2][hg], sm.wmax[par][3][hg]));
            const float al = ex2(m_ref[h] - mn);   // 0 for the first super-window of a unit
            l[h] *= al; Sm[0][h] *= al; Sm[1][h] *= al; Sm[2][h] *= al;
            m_ref[h] = mn;
          }
          touched = 0;
          period = 0;
        }
        period++;
        if (i == 0 && seg_idx > 0) flag = true;   // the previous unit's last request is served before this window's products
        if (valid) {
          const int xw = x0 + wq, slot = xw % NAV, use = xw / NAV;
          if (wq == 0 && hh == 0) TL(4, n, 4);
#ifndef OKQ_TC_ABLATE_VALUES
          if (use >= 1 && !mbar_wait(sm, &sm.v_done[slot], (uint32_t)(use - 1) & 1u)) { alive = false; break; }
#endif
          if (wq == 0 && hh == 0) TL(4, n, 5);
          const float vn = __half2float(reinterpret_cast<const __half*>(swin + OFF_VNORM)[lane]);
          int mod = sm.stage[st][STG_MOD + W * wq + tok];
          mod = mod > 2 ? 0 : mod;
          const float vs = vn * pscale;
          uint32_t pb[2];
#pragma unroll
          for (int h2 = 0; h2 < 2; h2++) {
            const float p0 = ex2(x[2 * h2] - m_ref[2 * h2]), p1 = ex2(x[2 * h2 + 1] - m_ref[2 * h2 + 1]);
            l[2 * h2] += p0; l[2 * h2 + 1] += p1;
            pb[h2] = pack_sat(p0 * vs, p1 * vs);
          }
          float pt[HH];   // the rounded numerators, as the tensor cores will see them
#pragma unroll
          for (int h2 = 0; h2 < 2; h2++) {
            const float2 f = __half22float2(u2h(pb[h2]));
            pt[2 * h2] = f.x * sinv; pt[2 * h2 + 1] = f.y * sinv;
          }
          const int first = __shfl_sync(0xffffffffu, mod, 0);
          const bool uniform = __all_sync(0xffffffffu, mod == first);
          unsigned char* tile = sm.bp[slot][0] + (lane >> 3) * 256 + (lane & 7) * 16 + 8 * hh;
          unsigned present;
          if (uniform) {
            present = 1u << first;
            *reinterpret_cast<uint2*>(tile) = make_uint2(pb[0], pb[1]);
            if (first == 0) {
#pragma unroll
              for (int h = 0; h < HH; h++) Sm[0][h] += pt[h];
            } else if (first == 1) {
#pragma unroll
              for (int h = 0; h < HH; h++) Sm[1][h] += pt[h];
            } else {
#pragma unroll
              for (int h = 0; h < HH; h++) Sm[2][h] += pt[h];
            }
          } else {
            present = (__any_sync(0xffffffffu, mod == 0) ? 1u : 0u) | (__any_sync(0xffffffffu, mod == 1) ? 2u : 0u) |
                      (__any_sync(0xffffffffu, mod == 2) ? 4u : 0u);
            int ti = 0;
#pragma unroll
            for (int m = 0; m < 3; m++) {
              if (!((present >> m) & 1u)) continue;
              const bool mine = mod == m;
              *reinterpret_cast<uint2*>(tile + ti * BP_TILE) = mine ? make_uint2(pb[0], pb[1]) : make_uint2(0u, 0u);
#pragma unroll
              for (int h = 0; h < HH; h++) Sm[m][h] += mine ? pt[h] : 0.f;
              ti++;
            }
          }
          touched |= (int)present;
          if (hh == 0 && lane == 0) { sm.bp_present[slot] = (int)present; sm.bp_flush[slot] = (wq == 0 && flag) ? 1 : 0; }
          if (wq == 0 && hh == 0) TL(4, n, 7);
          fence_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.bp_full[slot]);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.stage_free[st]);
        if (wq == 0 && hh == 0) TL(4, n, 6);
        x0 += n_w;
      }
      if (!alive) break;
      // end of the (sequence, head) piece: totals for the partial's header, and its last flush request
#pragma unroll
      for (int d = 1; d < 32; d <<= 1)
#pragma unroll
        for (int h = 0; h < HH; h++) {
          l[h] += __shfl_xor_sync(0xffffffffu, l[h], d);
          Sm[0][h] += __shfl_xor_sync(0xffffffffu, Sm[0][h], d);
          Sm[1][h] += __shfl_xor_sync(0xffffffffu, Sm[1][h], d);
          Sm[2][h] += __shfl_xor_sync(0xffffffffu, Sm[2][h], d);
        }
      const int par = gs & 1;
      if (lane == 0) {
#pragma unroll
        for (int h = 0; h < HH; h++) {
          const int hg = HH * hh + h;
          sm.lred[wq][hg] = l[h];
          sm.Sred[wq][0][hg] = Sm[0][h]; sm.Sred[wq][1][hg] = Sm[1][h]; sm.Sred[wq][2][hg] = Sm[2][h];
          if (wq == 0) sm.mold[par][hg] = m_ref[h];
        }
        if (hh == 0) sm.touched_w[par][wq] = touched;
      }
      if (!group_sync()) { alive = false; break; }
      if (wq == 0 && hh == 0 && lane == 0) {
        FlushReq& rq = sm.req[nreq % NREQ];
#pragma unroll
        for (int h = 0; h < GP; h++) {
          rq.m_period[h] = sm.mold[par][h];
          rq.l[h] = (sm.lred[0][h] + sm.lred[1][h]) + (sm.lred[2][h] + sm.lred[3][h]);
#pragma unroll
          for (int m = 0; m < 3; m++) rq.S[m][h] = (sm.Sred[0][m][h] + sm.Sred[1][m][h]) + (sm.Sred[2][m][h] + sm.Sred[3][m][h]);
        }
        rq.touched = sm.touched_w[par][0] | sm.touched_w[par][1] | sm.touched_w[par][2] | sm.touched_w[par][3];
        rq.seg_end = 1;
        rq.pidx = sg.unit + (int)blockIdx.x;
        __threadfence_block();
        mbar_arrive(&sm.req_full[nreq % NREQ]);
      }
      nreq++;
      seg_idx++;
    }
  } else if (warp < WARP_FL) {
    // ------------------------------------------------------------------ value codes -> tensor memory
    // two groups of four warps take the even and the odd windows; lane = channel c = 16 mu + 8 sh + g of the warp's
    // 32; its words are word (mu & 3) of the pieces (A = mu >> 2, g, t)
    const int vq = (warp - WARP_V) & 3, vpar = (warp - WARP_V) >> 2;
    const int sh = (lane >> 3) & 1, g = lane & 7;
    uint32_t voff[4];   // word (mu & 3) of the lane's piece (A = vq >> 1, g, t), t = 0..3
#pragma unroll
    for (int t = 0; t < 4; t++) voff[t] = OFF_VCODE + 16 * vpiece_slot(32 * (vq >> 1) + 4 * g + t) + 4 * (2 * (vq & 1) + (lane >> 4));
    SegWalk walk = walker();
    Seg sg;
    int n = 0, xw = 0;
    int pending = -1;   // slot whose tcgen05.st has been issued but not yet announced
    bool alive = true;
    while (alive && walk.next(sg)) {
      const int nsw = (sg.n_my + SWW - 1) / SWW;
      for (int i = 0; i < nsw && alive; i++, n++) {
        const int st = n % NST;
        const int n_w = min(SWW, sg.n_my - SWW * i);
        if (!mbar_wait(sm, &sm.stage_full[st], (uint32_t)(n / NST) & 1u)) { alive = false; break; }
        if (vq == 0 && vpar == 0) TL(5, n, 0);
        for (int j = 0; j < n_w; j++, xw++) {
#ifdef OKQ_TC_ABLATE_VALUES
          continue;
#endif
          if ((xw & 1) != vpar) continue;
          const int slot = xw % NAV, use = xw / NAV;
          const unsigned char* base = sm.stage[st] + j * STG_WIN;
          uint32_t wd[4];
#pragma unroll
          for (int t = 0; t < 4; t++) wd[t] = *reinterpret_cast<const uint32_t*>(base + voff[t]) >> (8 * sh);
          // word t, field jj: tokens with K index 8 t + 2 jj + {0, 1}; columns 4 t + jj (code plane), 16 + 4 t + jj (bit 1)
          uint32_t r[32];
#pragma unroll
          for (int t = 0; t < 4; t++)
#pragma unroll
            for (int jj = 0; jj < 4; jj++) {
              r[4 * t + jj] = wd[t] & (0x00030003u << (2 * jj));
              r[16 + 4 * t + jj] = wd[t] & (0x00020002u << (2 * jj));
            }
          if (pending >= 0) {   // the previous window's store had the time of this window's unpacking
            tmem_wait_st();
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.av_full[pending]);
          }
          if (use >= 1 && !mbar_wait(sm, &sm.v_done[slot], (uint32_t)(use - 1) & 1u)) { alive = false; break; }
          fence_after();
          tmem_st32(tmem + ((uint32_t)(32 * vq) << 16) + AV_COL + 32u * slot, r);
          pending = slot;
          if (vq == 0 && vpar == 0) TL(5, n, 1 + (j >> 1));
        }
        if (pending >= 0) {
          tmem_wait_st();
          fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.av_full[pending]);
          pending = -1;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.stage_free[st]);
      }
    }
  } else if (warp == WARP_MMA_V) {
    // ------------------------------------------------------------------ value MMAs
    constexpr uint32_t idesc = (1u << 4) | (1u << 16) | ((16u >> 3) << 17) | ((128u >> 4) << 24);   // B MN-major, N 16, M 128
    const uint64_t bp0 = make_desc(smem_u32(sm.bp[0][0]), 256, 128);
    const uint32_t tmem_u = __reduce_or_sync(0xffffffffu, tmem);
    SegWalk walk = walker();
    Seg sg;
    int xw = 0, f = 0;
    unsigned acc_valid = 0;
    bool alive = true;
#ifdef OKQ_TC_ABLATE_VALUES
    alive = false;
#endif
    while (alive && walk.next(sg)) {
      for (int j = 0; j < sg.n_my; j++, xw++) {
        const int slot = xw % NAV;
        const uint32_t par = (uint32_t)(xw / NAV) & 1u;
        if ((xw & 3) == 0) TL(6, xw >> 2, 0);
        if (!mbar_wait(sm, &sm.av_full[slot], par)) { alive = false; break; }
        if ((xw & 3) == 0) TL(6, xw >> 2, 1);
        if (!mbar_wait(sm, &sm.bp_full[slot], par)) { alive = false; break; }
        if ((xw & 3) == 0) TL(6, xw >> 2, 2);
        fence_after();
        // warp-wide reductions of values every lane holds alike: the compiler then knows them to be uniform and the
        // issuing thread works from uniform registers
        const unsigned present = __reduce_or_sync(0xffffffffu, (unsigned)sm.bp_present[slot]);
        if (__reduce_or_sync(0xffffffffu, (unsigned)sm.bp_flush[slot])) {
          if (elect_one()) mma_commit(&sm.flush_ready);
          __syncwarp();
          if (!mbar_wait(sm, &sm.acc_free, (uint32_t)f & 1u)) { alive = false; break; }
          fence_after();
          f++;
          acc_valid = 0;
        }
        if ((xw & 3) == 0) TL(6, xw >> 2, 5);
        if (elect_one()) {
          const uint32_t av = tmem_u + AV_COL + 32u * (uint32_t)slot;
          uint64_t bd = bp0 + (uint64_t)((slot * 3 * BP_TILE) >> 4);
#pragma unroll
          for (int m = 0; m < 3; m++) {
            if (!((present >> m) & 1u)) continue;
            const uint32_t d = tmem_u + ACC_COL + 32u * m;
            if ((acc_valid >> m) & 1u) {
              mma_ts<true>(d, av, bd, idesc); mma_ts<true>(d, av + 8u, bd + 32u, idesc);
              mma_ts<true>(d + 16u, av + 16u, bd, idesc); mma_ts<true>(d + 16u, av + 24u, bd + 32u, idesc);
            } else {
              mma_ts<false>(d, av, bd, idesc); mma_ts<true>(d, av + 8u, bd + 32u, idesc);
              mma_ts<false>(d + 16u, av + 16u, bd, idesc); mma_ts<true>(d + 16u, av + 24u, bd + 32u, idesc);
            }
            bd += (uint64_t)(BP_TILE >> 4);
          }
#ifdef OKQ_TC_TIMELINE
          if (blockIdx.x == 0 && (xw & 3) == 0 && (xw >> 2) < 64) g_tl[(6 * 64 + (xw >> 2)) * 8 + 6] = clock64();
#endif
          mma_commit(&sm.v_done[slot]);
#ifdef OKQ_TC_TIMELINE
          if (blockIdx.x == 0 && (xw & 3) == 0 && (xw >> 2) < 64) g_tl[(6 * 64 + (xw >> 2)) * 8 + 7] = clock64();
#endif
        }
        __syncwarp();
        if ((xw & 3) == 0) TL(6, xw >> 2, 3);
        if ((xw & 3) == 3) TL(6, xw >> 2, 4);
        acc_valid |= present;
      }
    }
    if (alive && xw > 0) {
      if (elect_one()) mma_commit(&sm.flush_ready);
      __syncwarp();
    }
  } else if (warp < WARP_LD) {
    // ------------------------------------------------------------------ flush: tensor memory -> running sums -> partial
    const int fq = warp - WARP_FL;
    const int c = 32 * fq + lane;
    constexpr float DELTA_REL = (3.0f * CB_INNER - CB_OUTER) / (2.0f * (CB_OUTER - CB_INNER));
    const float drel_h = __half2float(__float2half_rn(DELTA_REL));   // the combine kernel assumes this rounding
    constexpr float OUT_SCALE = (float)(1 << (6 - C_LOG2));          // PartialF fragments carry 2^-18, the accumulators 2^(C_LOG2-24)
    float sm_ref[3][GP];
#pragma unroll
    for (int m = 0; m < 3; m++)
#pragma unroll
      for (int h = 0; h < GP; h++) sm_ref[m][h] = -INFINITY;
    int n_seg = 0;
    {
      SegWalk walk = walker();
      Seg sg;
      while (walk.next(sg)) n_seg++;
    }
    int k = 0, seg_done = 0;
#ifdef OKQ_TC_ABLATE_VALUES
    n_seg = 0;
#endif
    while (seg_done < n_seg) {
      if (!mbar_wait(sm, &sm.req_full[k % NREQ], (uint32_t)(k / NREQ) & 1u) || !mbar_wait(sm, &sm.flush_ready, (uint32_t)k & 1u)) break;
      fence_after();
      const FlushReq& rq = sm.req[k % NREQ];
      const int touched = rq.touched;
#pragma unroll
      for (int m = 0; m < 3; m++) {
        if (!((touched >> m) & 1)) continue;
        uint32_t a0[8], a1[8];
        tmem_ld8(tmem + ((uint32_t)(32 * fq) << 16) + ACC_COL + (uint32_t)(2 * m) * 16u, a0);
        tmem_ld8(tmem + ((uint32_t)(32 * fq) << 16) + ACC_COL + (uint32_t)(2 * m + 1) * 16u, a1);
        tmem_wait_ld();
#pragma unroll
        for (int h = 0; h < GP; h++) {
          const float v = fmaf(drel_h, __uint_as_float(a1[h]), __uint_as_float(a0[h]));
          float* sp = &sm.sums[m][h][c];
          *sp = sm_ref[m][h] == -INFINITY ? v : fmaf(*sp, ex2(sm_ref[m][h] - rq.m_period[h]), v);
          sm_ref[m][h] = rq.m_period[h];
        }
      }
      fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.acc_free);
      if (rq.seg_end) {
        PartialF* out = P.partials_f + rq.pidx;
        const int r0 = 4 * (c >> 4) + 2 * ((c >> 3) & 1), l32 = 4 * (c & 7);
#pragma unroll
        for (int m = 0; m < 3; m++) {
          float v[GP];
#pragma unroll
          for (int h = 0; h < GP; h++)
            v[h] = sm_ref[m][h] == -INFINITY ? 0.f : sm.sums[m][h][c] * (ex2(sm_ref[m][h] - rq.m_period[h]) * OUT_SCALE);
          *reinterpret_cast<float4*>(&out->frag[m][r0][l32]) = make_float4(v[0], v[2], v[4], v[6]);
          *reinterpret_cast<float4*>(&out->frag[m][r0 + 1][l32]) = make_float4(v[1], v[3], v[5], v[7]);
#pragma unroll
          for (int h = 0; h < GP; h++) sm_ref[m][h] = -INFINITY;
        }
        if (fq == 0) {
          if (lane < GP) { out->m[lane] = rq.m_period[lane]; out->l[lane] = rq.l[lane]; }
        } else {
          out->Sp[fq - 1][lane] = (lane & 3) == 0 ? rq.S[fq - 1][lane >> 2] : 0.f;
        }
        seg_done++;
      }
      k++;
    }
  }

  fence_before();
  __syncthreads();
  if (tid == 0 && sm.abort) atomicCAS(cv.status, 0, (int)OKQ_ERR_TIMEOUT);
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;\n" ::"r"(tmem) : "memory");
}

#ifdef OKQ_TC_TIMELINE
extern "C" int okq_debug_timeline(long long* host_out) {
  return (int)cudaMemcpyFromSymbol(host_out, g_tl, sizeof(g_tl));
}
#endif

okq_status launch_decode_tc(const DecodeParams& P, int n_cta, cudaStream_t s) {
  static thread_local unsigned long long attr_mask = 0;
  int attr_dev = 0;
  if (attr_needed(attr_mask, attr_dev)) {
    cudaError_t e = cudaFuncSetAttribute(k_decode_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TcSmem) + 128);
    if (e != cudaSuccess) { set_last_cuda_error((int)e); return OKQ_ERR_CUDA; }
    attr_done(attr_mask, attr_dev);
  }
  k_decode_tc<<<n_cta, TC_THREADS, sizeof(TcSmem) + 128, s>>>(P);
  return OKQ_OK;
}

}  // namespace okq
