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
// Online softmax runs per warp in FlashAttention order; each warp streams its own windows
// through a cp.async ring in shared memory.  Values accumulate in the rotated basis of the
// current modality; the other modalities' accumulators wait in shared memory.  The grid is
// persistent: CTA i owns an equal slice of the flattened (layer, sequence, head, window)
// axis and writes one partial per (sequence, head) it touches; the combine kernel merges
// them, adds the raw fp16 tail tokens, applies R_m^T once per head and normalises.
#include "okq_common.cuh"
#include "okq_device.cuh"
#include "okq_decode_shared.cuh"

namespace okq {

namespace {

constexpr int NWARP = 8;
constexpr int NSTAGE = 3;
constexpr int STAGE_BYTES = RECORD_BYTES + 32;  // record + the window's 32 modality bytes
constexpr int SPILL_REGS = 33;                  // 32 accumulator registers + the running weight sum

struct MmaSmem {
  __align__(16) unsigned char stage[NWARP][NSTAGE][STAGE_BYTES];
  float spill[NWARP][3][SPILL_REGS][32];
  float spill_m[NWARP][3][GP];
  float qs[GP][D];       // q' * 2^kh, natural channel order
  float fscale[GP];      // 2^(24-kh) * sm_scale * log2(e)
  float wm[NWARP][GP], wl[NWARP][GP];
  int prefix[MAX_ENTRIES + 1];
};

__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ uint32_t h2u(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ __half2 u2h(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }

// fp16 pair (lo half = a, hi half = b), saturating instead of overflowing to infinity
__device__ __forceinline__ uint32_t pack_sat(float a, float b) {
  uint32_t r;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;\n" : "=r"(r) : "f"(b), "f"(a));
  return r;
}

// hi/lo split of the product q * x (q = qh + ql, x an exact fp16 pair): hi = rn(qh*x),
// lo = rn(ql*x + (qh*x - hi)); the inner fma recovers the rounding error of hi exactly.
__device__ __forceinline__ void split_product(__half2 qh, __half2 ql, __half2 x, uint32_t& hi, uint32_t& lo) {
  __half2 h = __hmul2(qh, x);
  __half2 e = __hfma2(qh, x, __hneg2(h));
  hi = h2u(h);
  lo = h2u(__hfma2(ql, x, e));
}

}  // namespace

// grid = n_cta (persistent), 256 threads
__global__ void __launch_bounds__(NWARP * 32, 1) k_decode_mma(DecodeParams P) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  MmaSmem& sm = *reinterpret_cast<MmaSmem*>(smem_raw);
  const CacheView& cv = P.cv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int G = P.group, Hkv = cv.n_kv_heads;
  const int n_entries = P.layer_count * cv.batch;

  // ---- partition of the flattened window axis
  const int total = block_prefix(cv, P.layer0, n_entries, sm.prefix);
  const int per = (total + gridDim.x - 1) / gridDim.x;
  int pos = min(total, (int)blockIdx.x * per);
  const int pos_end = min(total, pos + per);

  while (pos < pos_end) {
    // locate (entry, head, first window) of this segment
    int lo = 0, hi = n_entries;  // largest e with prefix[e] <= pos
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (sm.prefix[mid] <= pos) lo = mid; else hi = mid;
    }
    const int e = lo, li = e / cv.batch, b = e % cv.batch, layer = P.layer0 + li;
    const int nwin = (sm.prefix[e + 1] - sm.prefix[e]) / Hkv;
    const int off = pos - sm.prefix[e];
    const int h = off / nwin, w0 = off % nwin;
    const int seg = min(pos_end - pos, nwin - w0);
    const int unit = e * Hkv + h;

    // ---- per-segment setup: q' for the group's heads, scaled to the fp16 range
    {
      const int hh = warp;  // one head per warp (GP == NWARP)
      float4 qr = make_float4(0, 0, 0, 0);
      if (hh < G) {
        const __half* qrow = P.q + (((size_t)li * cv.batch + b) * cv.n_q_heads + h * G + hh) * D;
        float4 x = load_row4(qrow, lane);
        const float4 sg = *reinterpret_cast<const float4*>(P.signs + (size_t)li * D + 4 * lane);
        qr = warp_fwht(make_float4(x.x * sg.x, x.y * sg.y, x.z * sg.z, x.w * sg.w), lane);
      }
      float v[4] = {qr.x * RSQRT_D, qr.y * RSQRT_D, qr.z * RSQRT_D, qr.w * RSQRT_D};
      float mx = fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3])));
#pragma unroll
      for (int d = 16; d; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
      int ex = 0;
      if (mx > 0.f) frexpf(mx, &ex);           // mx < 2^ex
      const int kh = 14 - ex;                  // |q'| * 2^kh < 2^14
      const float up = exp2f((float)kh);
      *reinterpret_cast<float4*>(&sm.qs[hh][4 * lane]) = make_float4(v[0] * up, v[1] * up, v[2] * up, v[3] * up);
      if (lane == 0) sm.fscale[hh] = exp2f((float)(24 - kh)) * P.sm_scale * 1.4426950408889634f;
      // clear this warp's spilled accumulators
      float* sp = &sm.spill[warp][0][0][0];
      for (int i = lane; i < 3 * SPILL_REGS * 32; i += 32) sp[i] = 0.f;
      if (lane < 3 * GP) (&sm.spill_m[warp][0][0])[lane] = -INFINITY;
    }
    __syncthreads();

    // query fragments: head g, channels {16k + 8p + 2t + e}, pre-divided by 4^j, j = (2k + p) & 3
    __half2 qh[16], ql[16];
#pragma unroll
    for (int r = 0; r < 16; r++) {
      const int c0 = 16 * (r >> 1) + 8 * (r & 1) + 2 * t;
      const float sc = 1.0f / (float)(1 << (2 * (r & 3)));
      float x0 = sm.qs[g][c0] * sc, x1 = sm.qs[g][c0 + 1] * sc;
      __half2 hi2 = __floats2half2_rn(x0, x1);
      float2 hf = __half22float2(hi2);
      qh[r] = hi2;
      ql[r] = __floats2half2_rn(x0 - hf.x, x1 - hf.y);
    }
    const float fsc = sm.fscale[g];

    float acc[8][4];
#pragma unroll
    for (int mu = 0; mu < 8; mu++)
#pragma unroll
      for (int k = 0; k < 4; k++) acc[mu][k] = 0.f;
    float run_m = -INFINITY, run_l = 0.f, run_S = 0.f;
    int cur_mod = -1;

    // ---- this warp's windows: w0 + warp, w0 + warp + NWARP, ...
    const int n_my = seg > warp ? (seg - warp + NWARP - 1) / NWARP : 0;
    const unsigned char* rec0 = cv.record(layer, b, h, 0);
    const unsigned char* mod0 = cv.modality + (size_t)b * cv.capacity;
    auto issue = [&](int k) {
      if (k < n_my) {
        const int win = w0 + warp + k * NWARP;
        unsigned char* dst = sm.stage[warp][k % NSTAGE];
        const unsigned char* src = rec0 + (size_t)win * RECORD_BYTES;
#pragma unroll
        for (int i = 0; i < 6; i++) {
          int c16 = lane + 32 * i;
          if (c16 < RECORD_BYTES / 16) cp_async16(dst + 16 * c16, src + 16 * c16);
        }
        if (lane < 2) cp_async16(dst + RECORD_BYTES + 16 * lane, mod0 + (size_t)win * W + 16 * lane);
      }
      cp_async_commit();
    };
#pragma unroll
    for (int k = 0; k < NSTAGE - 1; k++) issue(k);

    for (int k = 0; k < n_my; k++) {
      issue(k + NSTAGE - 1);
      cp_async_wait<NSTAGE - 1>();
      __syncwarp();
      const unsigned char* st = sm.stage[warp][k % NSTAGE];

      // ================= scores =================
      const uint4* mp = reinterpret_cast<const uint4*>(st + OFF_KM + 64 * t);
      const uint4* sp = reinterpret_cast<const uint4*>(st + OFF_KS + 64 * t);
      float db[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int kq = 0; kq < 4; kq++) {  // bias: sum_c q'_c m_c against the constant operand 4^j 2^-24
        uint4 m4 = mp[kq];
        uint32_t a0, a1, a2, a3;
        split_product(qh[4 * kq + 0], ql[4 * kq + 0], u2h(m4.x), a0, a1);
        split_product(qh[4 * kq + 1], ql[4 * kq + 1], u2h(m4.y), a2, a3);
        mma16816(db, a0, a1, a2, a3, 0x00010001u, 0x00040004u);
        split_product(qh[4 * kq + 2], ql[4 * kq + 2], u2h(m4.z), a0, a1);
        split_product(qh[4 * kq + 3], ql[4 * kq + 3], u2h(m4.w), a2, a3);
        mma16816(db, a0, a1, a2, a3, 0x00100010u, 0x00400040u);
      }
      float d[4][4];
#pragma unroll
      for (int nu = 0; nu < 4; nu++)
#pragma unroll
        for (int i = 0; i < 4; i++) d[nu][i] = db[i];
      {
        const uint4 kc0 = *reinterpret_cast<const uint4*>(st + OFF_KCODE + 16 * lane);
        const uint4 kc1 = *reinterpret_cast<const uint4*>(st + OFF_KCODE + 512 + 16 * lane);
        // word[nu][ww]
        const uint32_t kw[4][2] = {{kc0.x, kc0.y}, {kc0.z, kc0.w}, {kc1.x, kc1.y}, {kc1.z, kc1.w}};
#pragma unroll
        for (int kq = 0; kq < 4; kq++) {
          uint4 s4 = sp[kq];
#pragma unroll
          for (int half = 0; half < 2; half++) {
            const int kappa = 2 * kq + half;
            uint32_t a0, a1, a2, a3;
            split_product(qh[2 * kappa], ql[2 * kappa], u2h(half ? s4.z : s4.x), a0, a1);
            split_product(qh[2 * kappa + 1], ql[2 * kappa + 1], u2h(half ? s4.w : s4.y), a2, a3);
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
      }

      // ================= online softmax (log2 domain) =================
      float sc[4][2], pf[4][2];
      {
        const __half2* knp = reinterpret_cast<const __half2*>(st + OFF_KNORM);
        float mx = -INFINITY;
#pragma unroll
        for (int nu = 0; nu < 4; nu++) {
          float2 kn = __half22float2(knp[4 * nu + t]);
          sc[nu][0] = (d[nu][0] + d[nu][2]) * (kn.x * fsc);
          sc[nu][1] = (d[nu][1] + d[nu][3]) * (kn.y * fsc);
          mx = fmaxf(mx, fmaxf(sc[nu][0], sc[nu][1]));
        }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(run_m, mx);
        if (__any_sync(0xffffffffu, m_new > run_m)) {
          const float alpha = exp2f(run_m - m_new);  // 0 on the first window
          run_l *= alpha;
          run_S *= alpha;
          const float a_lo = __shfl_sync(0xffffffffu, alpha, 8 * t);       // head 2t
          const float a_hi = __shfl_sync(0xffffffffu, alpha, 8 * t + 4);   // head 2t+1
#pragma unroll
          for (int mu = 0; mu < 8; mu++) {
            acc[mu][0] *= a_lo; acc[mu][1] *= a_hi; acc[mu][2] *= a_lo; acc[mu][3] *= a_hi;
          }
          run_m = m_new;
        }
        const __half2* vnp = reinterpret_cast<const __half2*>(st + OFF_VNORM);
#pragma unroll
        for (int nu = 0; nu < 4; nu++) {
          float2 vn = __half22float2(vnp[4 * nu + t]);
          float p0 = exp2f(sc[nu][0] - run_m), p1 = exp2f(sc[nu][1] - run_m);
          run_l += p0 + p1;
          pf[nu][0] = p0 * vn.x;
          pf[nu][1] = p1 * vn.y;
        }
      }

      // ================= values =================
      const unsigned char* wmod = st + RECORD_BYTES;
      const int mymod = wmod[lane];
      const int first = __shfl_sync(0xffffffffu, mymod, 0);
      const bool uniform = __all_sync(0xffffffffu, mymod == first);
      unsigned present = uniform ? (1u << first)
                                 : ((__any_sync(0xffffffffu, mymod == 0) ? 1u : 0u) |
                                    (__any_sync(0xffffffffu, mymod == 1) ? 2u : 0u) |
                                    (__any_sync(0xffffffffu, mymod == 2) ? 4u : 0u));
      const uint4 vc0 = *reinterpret_cast<const uint4*>(st + OFF_VCODE + 16 * lane);
      const uint4 vc1 = *reinterpret_cast<const uint4*>(st + OFF_VCODE + 512 + 16 * lane);
      const uint32_t vw[8] = {vc0.x, vc0.y, vc0.z, vc0.w, vc1.x, vc1.y, vc1.z, vc1.w};
      // numerators as fp16 pairs: p * vnorm * 2^6 / 4^nu, and the same times (3a-b)/(2(b-a))
      constexpr float DELTA_REL = (3.0f * CB_INNER - CB_OUTER) / (2.0f * (CB_OUTER - CB_INNER));
      uint32_t pb[4], pd[4];
#pragma unroll
      for (int nu = 0; nu < 4; nu++) {
        const float c = 64.0f / (float)(1 << (2 * nu));
        pb[nu] = pack_sat(pf[nu][0] * c, pf[nu][1] * c);
        pd[nu] = pack_sat(pf[nu][0] * (c * DELTA_REL), pf[nu][1] * (c * DELTA_REL));
      }
      // process the modalities present, starting with the one already in registers
      for (int pass = 0; pass < 3 && present; pass++) {
        int m = (cur_mod >= 0 && (present >> cur_mod) & 1) ? cur_mod : (__ffs(present) - 1);
        present &= ~(1u << m);
        if (m != cur_mod) {
          // swap accumulators: park the current modality, fetch modality m rescaled to run_m
          if (cur_mod >= 0) {
            float* dst = &sm.spill[warp][cur_mod][0][lane];
#pragma unroll
            for (int mu = 0; mu < 8; mu++)
#pragma unroll
              for (int i = 0; i < 4; i++) dst[(4 * mu + i) * 32] = acc[mu][i];
            dst[32 * 32] = run_S;
            if (t == 0) sm.spill_m[warp][cur_mod][g] = run_m;
          }
          __syncwarp();
          const float* src = &sm.spill[warp][m][0][lane];
          const float sm_lo = sm.spill_m[warp][m][2 * t], sm_hi = sm.spill_m[warp][m][2 * t + 1];
          const float sm_g = sm.spill_m[warp][m][g];
          const float m_lo = __shfl_sync(0xffffffffu, run_m, 8 * t), m_hi = __shfl_sync(0xffffffffu, run_m, 8 * t + 4);
          const float f_lo = sm_lo == -INFINITY ? 0.f : exp2f(sm_lo - m_lo);
          const float f_hi = sm_hi == -INFINITY ? 0.f : exp2f(sm_hi - m_hi);
          const float f_g = sm_g == -INFINITY ? 0.f : exp2f(sm_g - run_m);
#pragma unroll
          for (int mu = 0; mu < 8; mu++) {
            acc[mu][0] = src[(4 * mu + 0) * 32] * f_lo; acc[mu][1] = src[(4 * mu + 1) * 32] * f_hi;
            acc[mu][2] = src[(4 * mu + 2) * 32] * f_lo; acc[mu][3] = src[(4 * mu + 3) * 32] * f_hi;
          }
          run_S = src[32 * 32] * f_g;
          cur_mod = m;
          __syncwarp();
        }
        uint32_t b0[4], b1[4];
        unsigned halfmask = 3u;  // which 16-token halves hold a token of modality m
        if (uniform) {
#pragma unroll
          for (int nu = 0; nu < 4; nu++) { b0[nu] = pb[nu]; b1[nu] = pd[nu]; run_S += pf[nu][0] + pf[nu][1]; }
        } else {
          bool any_lo = false, any_hi = false;
#pragma unroll
          for (int nu = 0; nu < 4; nu++) {
            const bool k0 = wmod[8 * nu + 2 * t] == m, k1 = wmod[8 * nu + 2 * t + 1] == m;
            const uint32_t msk = (k0 ? 0x0000ffffu : 0u) | (k1 ? 0xffff0000u : 0u);
            b0[nu] = pb[nu] & msk;
            b1[nu] = pd[nu] & msk;
            run_S += (k0 ? pf[nu][0] : 0.f) + (k1 ? pf[nu][1] : 0.f);
            if (nu < 2) any_lo |= (k0 | k1); else any_hi |= (k0 | k1);
          }
          halfmask = (__any_sync(0xffffffffu, any_lo) ? 1u : 0u) | (__any_sync(0xffffffffu, any_hi) ? 2u : 0u);
        }
#pragma unroll
        for (int kv = 0; kv < 2; kv++) {
          if (!((halfmask >> kv) & 1)) continue;
          const uint32_t mA = 0x00030003u << (4 * kv), mB = 0x000c000cu << (4 * kv);
          const uint32_t nA = 0x00020002u << (4 * kv), nB = 0x00080008u << (4 * kv);
#pragma unroll
          for (int mu = 0; mu < 8; mu++) {
            const uint32_t w = vw[mu], w8 = w >> 8;
            mma16816(acc[mu], w & mA, w8 & mA, w & mB, w8 & mB, b0[2 * kv], b0[2 * kv + 1]);
            mma16816(acc[mu], w & nA, w8 & nA, w & nB, w8 & nB, b1[2 * kv], b1[2 * kv + 1]);
          }
        }
      }
      __syncwarp();  // every lane is done with this stage before it is refilled
    }
    cp_async_wait<0>();

    // ---- park the live accumulators and merge the warps
    if (cur_mod >= 0) {
      float* dst = &sm.spill[warp][cur_mod][0][lane];
#pragma unroll
      for (int mu = 0; mu < 8; mu++)
#pragma unroll
        for (int i = 0; i < 4; i++) dst[(4 * mu + i) * 32] = acc[mu][i];
      dst[32 * 32] = run_S;
      if (t == 0) sm.spill_m[warp][cur_mod][g] = run_m;
    }
    {
      float lt = run_l;
      lt += __shfl_xor_sync(0xffffffffu, lt, 1);
      lt += __shfl_xor_sync(0xffffffffu, lt, 2);
      if (t == 0) { sm.wm[warp][g] = run_m; sm.wl[warp][g] = lt; }
    }
    __syncthreads();
    PartialF* out = P.partials_f + (size_t)unit + blockIdx.x;
    {
      // every thread needs the merged maxima of the heads it touches
      float M[GP];
#pragma unroll
      for (int j = 0; j < GP; j++) {
        float mj = -INFINITY;
#pragma unroll
        for (int w8 = 0; w8 < NWARP; w8++) mj = fmaxf(mj, sm.wm[w8][j]);
        M[j] = mj;
      }
      if (tid < GP) {
        float L = 0.f;
        for (int w8 = 0; w8 < NWARP; w8++)
          L += sm.wm[w8][tid] == -INFINITY ? 0.f : sm.wl[w8][tid] * exp2f(sm.wm[w8][tid] - M[tid]);
        out->m[tid] = M[tid];
        out->l[tid] = L;
      }
      for (int idx = tid; idx < 3 * SPILL_REGS * 32; idx += NWARP * 32) {
        const int l32 = idx & 31, r = (idx >> 5) % SPILL_REGS, m = idx / (SPILL_REGS * 32);
        const int head = r < 32 ? 2 * (l32 & 3) + (r & 1) : (l32 >> 2);
        float v = 0.f;
#pragma unroll
        for (int w8 = 0; w8 < NWARP; w8++) {
          const float smx = sm.spill_m[w8][m][head];
          if (smx != -INFINITY) v = fmaf(sm.spill[w8][m][r][l32], exp2f(smx - M[head]), v);
        }
        if (r < 32) out->frag[m][r][l32] = v;
        else out->Sp[m][l32] = v;
      }
    }
    __syncthreads();
    pos += seg;
  }
}

// grid (n_kv_heads, batch*layer_count), 128 threads: merge partials, add the raw tail,
// apply R_m^T, normalise
__global__ void __launch_bounds__(128) k_combine_mma(DecodeParams P, int n_cta) {
  __shared__ float vec[3][GP][D];
  __shared__ float tsc[W][GP];       // tail scores (log2 domain)
  __shared__ float Ms[GP], Ls[GP];
  __shared__ int prefix[MAX_ENTRIES + 1];
  const CacheView& cv = P.cv;
  const int h = blockIdx.x, e = blockIdx.y, b = e % cv.batch, li = e / cv.batch, layer = P.layer0 + li;
  const int c = threadIdx.x, G = P.group, Hkv = cv.n_kv_heads;
  const int n_entries = P.layer_count * cv.batch;
  const int total = block_prefix(cv, P.layer0, n_entries, prefix);
  const int per = total > 0 ? (total + n_cta - 1) / n_cta : 1;
  const int seq = cv.seq_len[layer * cv.batch + b];
  const int nwin = seq / W, n_tail = seq - nwin * W;
  const int unit = e * Hkv + h;
  const int start = prefix[e] + h * nwin, end = start + nwin;
  const int cta_lo = nwin > 0 ? start / per : 0, cta_hi = nwin > 0 ? (end - 1) / per : -1;
  const __half* qbase = P.q + (((size_t)li * cv.batch + b) * cv.n_q_heads + h * G) * D;
  const __half* kt = cv.k_tail + cv.tail_off(layer, b, h);
  const __half* vt = cv.v_tail + cv.tail_off(layer, b, h);

  // tail scores: thread -> (token = c & 31, heads (c >> 5) * 2 + {0, 1})
  {
    const int tok = c & 31;
#pragma unroll
    for (int hh = 0; hh < 2; hh++) {
      const int j = (c >> 5) * 2 + hh;
      float s = -INFINITY;
      if (tok < n_tail && j < G) {
        float a = 0.f;
        for (int k = 0; k < D; k += 2) {
          float2 qv = __half22float2(*reinterpret_cast<const __half2*>(qbase + j * D + k));
          float2 kv = __half22float2(*reinterpret_cast<const __half2*>(kt + tok * D + k));
          a = fmaf(qv.x, kv.x, a);
          a = fmaf(qv.y, kv.y, a);
        }
        s = a * P.sm_scale * 1.4426950408889634f;
      }
      tsc[tok][j] = s;
    }
  }
  __syncthreads();
  if (c < GP) {
    float M = -INFINITY;
    for (int ct = cta_lo; ct <= cta_hi; ct++) M = fmaxf(M, P.partials_f[(size_t)unit + ct].m[c]);
    for (int i = 0; i < n_tail; i++) M = fmaxf(M, tsc[i][c]);
    float L = 0.f;
    for (int ct = cta_lo; ct <= cta_hi; ct++) {
      const PartialF& pp = P.partials_f[(size_t)unit + ct];
      if (pp.m[c] != -INFINITY) L += pp.l[c] * exp2f(pp.m[c] - M);
    }
    for (int i = 0; i < n_tail; i++) L += exp2f(tsc[i][c] - M);
    Ms[c] = M;
    Ls[c] = L;
  }
  __syncthreads();
  constexpr float ACC_SCALE = (CB_OUTER - CB_INNER) * 262144.0f;  // (b - a) * 2^18
  float raw[GP];
#pragma unroll
  for (int j = 0; j < GP; j++) {
    raw[j] = 0.f;
    if (j >= G) continue;
    const float M = Ms[j];
    float v[3] = {0.f, 0.f, 0.f};
    const int r = 4 * (c >> 4) + 2 * ((c >> 3) & 1) + (j & 1), l32 = 4 * (c & 7) + (j >> 1);
    for (int ct = cta_lo; ct <= cta_hi; ct++) {
      const PartialF& pp = P.partials_f[(size_t)unit + ct];
      if (pp.m[j] == -INFINITY) continue;
      const float ef = exp2f(pp.m[j] - M);
#pragma unroll
      for (int m = 0; m < 3; m++) {
        // weight sum of head j: the four lanes of quad j hold partial sums
        const float S = pp.Sp[m][4 * j] + pp.Sp[m][4 * j + 1] + pp.Sp[m][4 * j + 2] + pp.Sp[m][4 * j + 3];
        v[m] = fmaf(fmaf(ACC_SCALE, pp.frag[m][r][l32], -CB_OUTER * S), ef, v[m]);
      }
    }
    vec[0][j][c] = v[0]; vec[1][j][c] = v[1]; vec[2][j][c] = v[2];
    float a = 0.f;
    for (int i = 0; i < n_tail; i++) a = fmaf(exp2f(tsc[i][j] - M), __half2float(vt[i * D + c]), a);
    raw[j] = a;
  }
  __syncthreads();
  float o[GP];
#pragma unroll
  for (int j = 0; j < GP; j++) o[j] = 0.f;
  const float* Rset = P.R + ((size_t)li * P.n_R + (P.n_R == 1 ? 0 : h)) * 3 * D * D;
  for (int m = 0; m < 3; m++)
    for (int r = 0; r < D; r++) {
      const float rv = __ldg(Rset + ((size_t)m * D + r) * D + c);
#pragma unroll
      for (int j = 0; j < GP; j++) o[j] = fmaf(rv, vec[m][j][r], o[j]);
    }
#pragma unroll
  for (int j = 0; j < GP; j++) {
    if (j >= G) continue;
    const float L = Ls[j];
    P.out[(((size_t)li * cv.batch + b) * cv.n_q_heads + h * G + j) * D + c] = L > 0.f ? (o[j] + raw[j]) / L : 0.f;
  }
}

okq_status launch_decode_mma(const DecodeParams& P, int n_cta, cudaStream_t s, cudaEvent_t before, cudaEvent_t after) {
  static thread_local bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(k_decode_mma, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(MmaSmem));
    if (e != cudaSuccess) { set_last_cuda_error((int)e); return OKQ_ERR_CUDA; }
    attr_set = true;
  }
  if (before) cudaEventRecord(before, s);
  k_decode_mma<<<n_cta, NWARP * 32, sizeof(MmaSmem), s>>>(P);
  if (after) cudaEventRecord(after, s);
  k_combine_mma<<<dim3(P.cv.n_kv_heads, P.cv.batch * P.layer_count), 128, 0, s>>>(P, n_cta);
  return OKQ_OK;
}

}  // namespace okq
