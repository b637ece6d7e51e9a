// Bulk value quantiser with the per-modality rotation on the 5th-generation tensor cores
// (Eq. 6 then Eq. 3 for whole prefill chunks).
//
// z = R_m v is a dense [tokens x 128] x [128 x 128] contraction.  A CTA takes tiles of 128
// consecutive tokens (four windows) of one (sequence, KV head):
// three roles that meet only at mbarriers:
//   * a loader warp brings each tile of fp16 values with two TMA tensor copies (64 channels x 128
//     tokens, 128-byte swizzle: the K-major layout tcgen05.mma reads) plus the tile's modality bytes
//     (two tile buffers, "full" / "empty" barriers); the values are the B operand as they are (exact);
//   * an MMA warp issues the tensor-core work of a tile as soon as it has landed and one of the two
//     accumulator sets in tensor memory is free ("mma_done" / "acc_free" barriers);
//   * sixteen worker warps compute the norms and turn accumulators into packed codes.
// In detail:
//   * R_m (fp32) is split into two fp16 matrices R_hi + R_lo (the A operand), kept in shared memory
//     while the modality does not change; 16 tcgen05.mma (M = 128, K = 16, N = the windows of the
//     tile that hold the modality) accumulate z^T = R_hi v^T + R_lo v^T in fp32 in tensor memory:
//     lane = output channel, column = token;
//   * in the epilogue a thread owns one channel and reads the 32 tokens of one window with one
//     tcgen05.ld: exactly the (channel, 8 tokens) groups a word of the decode kernel's value-code
//     layout holds, so the words are built in registers (one lane exchange joins the two channels
//     of a word).  The code, the number of thresholds {-T, 0, T} below z / norm, is taken
//     arithmetically: v = sat(2/3 - z / (3 T norm)), k = floor(3 v) with a round-down fused
//     multiply-add against 1.5 * 2^23, code = 3 - k: three full-rate instructions per element.
// The split leaves a relative error of about 2^-22 on z and the tensor cores' accumulation about
// 1e-6, so the arithmetic code is only trusted where z / norm is further than 2^-18 from every
// threshold (the code is taken twice, with the coordinate moved down and up by that band); the few
// coordinates in the band (about 1e-4 of them) are listed and recomputed at the end of the kernel, one per warp at
// a time, with the exact fused-multiply-add chain of the reference arithmetic over the value row, read again from
// global memory; the code in the record is then patched.  Codes and norms (exact summation tree) are therefore bit-identical to the exact path.
//
// Every wait on an mbarrier is bounded; on a timeout the kernel records OKQ_ERR_TIMEOUT in the
// cache's status word, stops issuing work, frees its tensor memory and returns.
#include <cuda.h>   // CUtensorMap and the type of cuTensorMapEncodeTiled only; the entry point is fetched at run time

#include "okq_common.cuh"
#include "okq_device.cuh"

namespace okq {

namespace {

constexpr int TILE = 128;                 // tokens per tile
constexpr int NT = 512;                   // worker threads per CTA: 16 warps, four per tensor-memory lane quarter
constexpr int NT_ALL = NT + 64;           // + the MMA warp (16) and the loader warp (17)
constexpr int TILE_BYTES = TILE * D * 2;  // 32 KB: one fp16 operand tile
constexpr float NEG_INV_3T = -1.0f / (3.0f * CB_THRESH);
constexpr float TWO_THIRDS = 2.0f / 3.0f;          // rounds up: a zero coordinate gives floor(3 v) = 2, code 1
// The code is taken twice, with the coordinate moved down and up by BAND (in units of z / norm: far above the
// rounding noise of the tensor-core product, about 1e-6); where the two disagree the coordinate lies that close to a
// threshold and is recomputed with the exact fused-multiply-add chain of the reference arithmetic.
constexpr float BAND = 0x1p-18f;
constexpr float BAND_V = BAND / (3.0f * CB_THRESH);
constexpr float FLOOR_MAGIC = 12582912.0f;         // 1.5 * 2^23: unit in the last place 1, bits 0x4B400000
// sum over the eight fields (bit 16*e + 2*j) of a word of the magic bits shifted to the field, modulo 2^32
constexpr uint32_t magic_sum() {
  uint32_t s = 0;
  for (int e = 0; e < 2; e++)
    for (int j = 0; j < 4; j++) s += 0x4B400000u << (16 * e + 2 * j);
  return s;
}
constexpr uint32_t MAGIC_SUM = magic_sum();
constexpr long long WAIT_LIMIT_CLOCKS = 4000000000ll;   // about two seconds of SM clocks

// A coordinate too close to a threshold for the tensor-core product to decide: recomputed with the reference
// arithmetic at the end of the kernel (its code is patched in the record), so that the tile pipeline never waits for
// the two rows this needs from global memory.
struct FixItem {
  uint32_t* word;        // code word of the record
  const __half* xrow;    // the token's value row (128 fp16)
  const float* rrow;     // row of the rotation matrix (128 fp32): output channel of the coordinate
  float inv;             // 1 / norm
  int bit;               // bit position of the 2-bit field in the word
};
constexpr int FIX_MAX = 256;

struct TcSmem {
  __align__(1024) unsigned char a[2][TILE_BYTES];      // value tiles (double buffered)
  __align__(1024) unsigned char b[2][2][TILE_BYTES];   // two resident matrices, each as R_hi, R_lo
  __align__(16) float part[2][4][TILE];                // per token: sum of squares of channels [32 q, 32 q + 32)
  __align__(16) float c3[16][W];                       // per worker warp: -1 / (3 T norm) of its window's tokens
  __align__(16) float inv[16][W];                      // per worker warp: 1 / norm of its window's tokens (0 for a zero vector)
  __align__(4) unsigned char mod[2][TILE];             // modality per token of a tile (255 = no token)
  __align__(8) unsigned long long full[2];             // 1 arrival + 32 KB of TMA bytes: tile and modality bytes are in
  __align__(8) unsigned long long empty[2];            // 16 arrivals: every worker warp is done with the buffer
  __align__(8) unsigned long long mma_done[2];         // 1 arrival (tcgen05.commit): accumulator set complete
  __align__(8) unsigned long long acc_free[2];         // 16 arrivals: every worker warp has read the accumulator set
  __align__(8) unsigned long long part_ready[2];       // 16 arrivals: every worker warp has written its partial norms
  __align__(8) unsigned long long slot_ready;          // 16 arrivals: every worker warp has written its share of a rotation matrix
  uint32_t tmem_slot;
  FixItem fix[FIX_MAX];
  int fix_count;
  long long limit;                                     // SM clocks a wait may take
  volatile int abort;                                  // set by a role whose bounded wait ran out
  volatile int tmem_busy;                              // set if products may still be in flight at the end (tensor memory is then not released)
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool elect_one() {
  uint32_t pred = 0;
  asm volatile("{\n\t.reg .b32 rx;\n\t.reg .pred px;\n\telect.sync rx|px, 0xffffffff;\n\tselp.u32 %0, 1, 0, px;\n\t}\n" : "=r"(pred));
  return pred != 0;
}

// shared-memory matrix descriptor: no swizzle, K-major; core matrices of 8 rows x 16 bytes,
// `lbo` bytes between the two 8-element K chunks of one MMA, `sbo` bytes between 8-row groups
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((saddr >> 4) & 0x3fff) | ((uint64_t)((lbo >> 4) & 0x3fff) << 16) |
         ((uint64_t)((sbo >> 4) & 0x3fff) << 32) | ((uint64_t)1 << 46);
}

// byte offset of element (row r, column k) of a 128 x 128 fp16 operand tile
__device__ __forceinline__ uint32_t tile_off(int r, int k) {
  return (uint32_t)((k >> 3) * 2048 + (r >> 3) * 128 + (r & 7) * 16 + (k & 7) * 2);
}

// shared-memory matrix descriptor of a TMA-written tile: K-major, 128-byte swizzle (rows of 64 fp16 = 128
// bytes, 8-row groups 1024 bytes apart; the leading-dimension field is not used by this layout)
__device__ __forceinline__ uint64_t make_desc_sw128(uint32_t saddr) {
  return (uint64_t)((saddr >> 4) & 0x3fff) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}

// byte offset of the 16-byte chunk holding channels [8 kc, 8 kc + 8) of token row r in a TMA-written value
// tile: two halves of 64 channels, 128 bytes per row, chunk index xor-ed with the row inside its 8-row group
__device__ __forceinline__ uint32_t vtile_off(int r, int kc) {
  return (uint32_t)((kc >> 3) * (TILE_BYTES / 2) + r * 128 + (((kc & 7) ^ (r & 7)) << 4));
}

// Bounded wait of a whole warp for one phase of an mbarrier (each try may suspend the thread for a short,
// system-chosen time).  Gives up after about two seconds, or as soon as another role has given up; giving
// up raises the abort flag.
__device__ __forceinline__ bool mbar_wait(TcSmem& sm, unsigned long long* bar, uint32_t parity) {
  const uint32_t mbar = smem_u32(bar);
  bool done = false;
  const long long t0 = clock64();
  while (!done) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                 : "=r"(ok) : "r"(mbar), "r"(parity) : "memory");
    done = ok != 0;
    if (!done && (sm.abort || clock64() - t0 > sm.limit)) break;
  }
  if (!done) sm.abort = 1;
  return __all_sync(0xffffffffu, done);   // called by whole warps: one answer per warp
}
// After a timeout: wait, again with a limit and whatever the abort flag says, for a phase that this warp's own
// asynchronous work (bulk copies, tensor-core products) will complete.  Returns false if it did not.
__device__ __forceinline__ bool mbar_drain(unsigned long long* bar, uint32_t parity) {
  const uint32_t mbar = smem_u32(bar);
  bool done = false;
  const long long t0 = clock64();
  while (!done && clock64() - t0 < WAIT_LIMIT_CLOCKS / 8) {   // a quarter of a second, whatever the caller's limit
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                 : "=r"(ok) : "r"(mbar), "r"(parity) : "memory");
    done = ok != 0;
  }
  return __all_sync(0xffffffffu, done);
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(smem_u32(bar)) : "memory");
}

// The jobs of a tile, derived identically by the MMA warp and every worker warp from the tile's modality
// bytes: `present` = modalities in the tile (bit m); a job takes at most two of them, so a tile with all
// three needs two jobs.  winmask[m] = windows of the tile (bit w) that hold modality m.
struct TileMods {
  unsigned present;
  unsigned winmask[3];
};
__device__ __forceinline__ TileMods tile_mods(const unsigned char* mod, int lane) {
  const uint32_t m4 = reinterpret_cast<const uint32_t*>(mod)[lane];   // 4 tokens per lane, window lane >> 3
  TileMods t;
  t.present = 0;
#pragma unroll
  for (int mm = 0; mm < 3; mm++) {
    const bool has = ((m4 & 0xffu) == mm) | (((m4 >> 8) & 0xffu) == mm) | (((m4 >> 16) & 0xffu) == mm) | ((m4 >> 24) == mm);
    const unsigned bal = __ballot_sync(0xffffffffu, has);
    t.winmask[mm] = ((bal & 0xffu) ? 1u : 0u) | ((bal & 0xff00u) ? 2u : 0u) | ((bal & 0xff0000u) ? 4u : 0u) | ((bal >> 24) ? 8u : 0u);
    if (bal) t.present |= 1u << mm;
  }
  return t;
}
// modalities of job `jt` (0 or 1) of a tile: returns their count (0 = no such job)
__device__ __forceinline__ int job_mods(unsigned present, int jt, int (&mods)[2]) {
  int n = 0;
  unsigned p = present;
  if (jt == 1) {   // the third modality, if there is one
    if (__popc(p) < 3) return 0;
    mods[0] = 2;
    return 1;
  }
  while (p && n < 2) { mods[n++] = __ffs(p) - 1; p &= p - 1; }
  return n;
}

// The two resident rotation matrices (hi/lo pairs), tracked identically by the MMA warp and the worker warps.
// plan() assigns the job's matrices to slots and says which have to be written first; a matrix goes to the
// slot the job's other matrix does not use, else to the one that was not used last.
struct Slots {
  int key[2] = {-1, -1};   // (rotation set * 3 + modality) held by each slot
  int last = 0;
  __device__ __forceinline__ bool plan(int nm, const int (&keys)[2], int (&slot)[2], bool (&need)[2]) {
    for (int mi = 0; mi < 2; mi++) {
      need[mi] = false;
      slot[mi] = mi < nm ? (key[0] == keys[mi] ? 0 : (key[1] == keys[mi] ? 1 : -1)) : -1;
    }
    bool any = false;
    for (int mi = 0; mi < nm; mi++) {
      if (slot[mi] >= 0) continue;
      const int other = nm == 2 ? slot[mi ^ 1] : -1;
      const int victim = other >= 0 ? (other ^ 1) : (last ^ 1);
      key[victim] = keys[mi];
      slot[mi] = victim;
      need[mi] = any = true;
    }
    last = slot[nm - 1];
    return any;
  }
};

}  // namespace

// persistent grid, NT_ALL threads.  Tiles are numbered (b, h, tile-in-sequence), tile = 4 windows; a CTA
// owns a contiguous range of them.  A "job" is one tile and at most two of the modalities present in it
// (one accumulator of 128 columns each); jobs alternate between two accumulator sets in tensor memory.
__global__ void __launch_bounds__(NT_ALL, 1) k_quantize_values_tc(const __grid_constant__ CUtensorMap vmap, CacheView cv, int layer,
                                                             const unsigned char* __restrict__ modality, int n_tokens,
                                                             int n_win, const float* __restrict__ R, int n_R,
                                                             const __half* __restrict__ vrows, long long vs_b, long long vs_h,
                                                             long long vs_t, long long wait_limit, int skip_tile) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  TcSmem& sm = *reinterpret_cast<TcSmem*>(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tiles_per_unit = (n_win + 3) / 4;   // n_win: windows to pack (the schedule may keep recent tokens raw)
  const int n_tiles_all = tiles_per_unit * cv.n_kv_heads * cv.batch;
  // contiguous tile range of this CTA
  const int per_cta = (n_tiles_all + gridDim.x - 1) / gridDim.x;
  const int tile_begin = min(n_tiles_all, (int)blockIdx.x * per_cta);
  const int my_tiles = min(n_tiles_all, tile_begin + per_cta) - tile_begin;

  if (tid == 0) {
    for (int i = 0; i < 2; i++) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(smem_u32(&sm.full[i])));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 16;\n" ::"r"(smem_u32(&sm.empty[i])));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(smem_u32(&sm.mma_done[i])));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 16;\n" ::"r"(smem_u32(&sm.acc_free[i])));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 16;\n" ::"r"(smem_u32(&sm.part_ready[i])));
    }
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 16;\n" ::"r"(smem_u32(&sm.slot_ready)));
    sm.abort = 0;
    sm.tmem_busy = 0;
    sm.fix_count = 0;
    sm.limit = wait_limit;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;\n" ::"r"(smem_u32(&sm.tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
  const uint32_t tmem = sm.tmem_slot;

  // coordinates of the first tile; every role steps them without divisions afterwards
  int cb = 0, ch = 0, cwin0 = 0;
  if (my_tiles > 0) {
    cb = tile_begin / (tiles_per_unit * cv.n_kv_heads);
    const int rem = tile_begin - cb * tiles_per_unit * cv.n_kv_heads;
    ch = rem / tiles_per_unit;
    cwin0 = (rem - ch * tiles_per_unit) * 4;
  }
  auto step_coords = [&]() {
    cwin0 += 4;
    if (cwin0 >= tiles_per_unit * 4) { cwin0 = 0; if (++ch == cv.n_kv_heads) { ch = 0; cb++; } }
  };

  if (warp == 17) {
    // ------------------------------------------------------------------ loader warp
    // tile i of the range goes to buffer i & 1 once the buffer's previous tile (i - 2) has been released.
    // A lane carries the modality bytes of the tokens 4*lane .. 4*lane+3, fetched one tile ahead.
    auto fetch_mod = [&](int i) -> uint32_t {
      uint32_t packed = 0xffffffffu;
      if (i < my_tiles) {
        const int rows = min(TILE, (n_win - cwin0) * W);
        packed = 0;
#pragma unroll
        for (int u = 0; u < 4; u++) {
          const int tok = 4 * lane + u;
          unsigned m = 255;
          if (tok < rows) { m = modality[(size_t)cb * n_tokens + (size_t)cwin0 * W + tok]; m = m > 2 ? 0 : m; }
          packed |= m << (8 * u);
        }
      }
      return packed;
    };
    uint32_t mod_cur = fetch_mod(0);
    int armed = 0;   // tiles whose copies have been issued
    for (int i = 0; i < my_tiles; i++) {
      const int buf = i & 1, fill = i >> 1;
      if (tile_begin + i == skip_tile) {   // testing aid: this tile never arrives, so that every role's wait runs out
        step_coords();
        mod_cur = fetch_mod(i + 1);
        continue;
      }
      if (fill >= 1 && !mbar_wait(sm, &sm.empty[buf], (uint32_t)(fill - 1) & 1u)) break;
      reinterpret_cast<uint32_t*>(sm.mod[buf])[lane] = mod_cur;
      __syncwarp();
      if (lane == 0) {
        // the arrival (release) publishes sm.mod; the phase completes when the 32 KB have landed.  Rows past
        // the end of the sequence are filled with zeros by the copy engine.
        const uint32_t bar = smem_u32(&sm.full[buf]);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"((uint32_t)TILE_BYTES) : "memory");
#pragma unroll
        for (int half = 0; half < 2; half++)
          asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];\n"
                       ::"r"(smem_u32(sm.a[buf]) + half * (TILE_BYTES / 2)), "l"(reinterpret_cast<uint64_t>(&vmap)),
                         "r"(64 * half), "r"(cwin0 * W), "r"(ch), "r"(cb), "r"(bar) : "memory");
      }
      armed = i + 1;
      step_coords();
      mod_cur = fetch_mod(i + 1);
    }
    // after a timeout somewhere: no copy of this warp may still be landing when the block ends
    if (sm.abort)
      for (int i = max(0, armed - 2); i < armed; i++) mbar_drain(&sm.full[i & 1], (uint32_t)(i >> 1) & 1u);
  } else if (warp == 16) {
    // ------------------------------------------------------------------ MMA warp
    Slots slots;
    uint32_t jobidx = 0, refills = 0;
    bool dead = false;
    for (int i = 0; i < my_tiles && !dead; i++) {
      const int buf = i & 1;
      if (!mbar_wait(sm, &sm.full[buf], (uint32_t)(i >> 1) & 1u)) break;
      const TileMods tm = tile_mods(sm.mod[buf], lane);
      for (int jt = 0; jt < 2; jt++) {
        int mods[2] = {0, 0};
        const int nm = job_mods(tm.present, jt, mods);
        if (nm == 0) break;
        const uint32_t a = jobidx & 1u;
        if (jobidx >= 2 && !mbar_wait(sm, &sm.acc_free[a], ((jobidx >> 1) - 1u) & 1u)) { dead = true; break; }
        // resident rotation matrices: the worker warps write a missing one and report on slot_ready
        int slot[2];
        bool need[2];
        const int keys[2] = {(n_R == 1 ? 0 : ch) * 3 + mods[0], (n_R == 1 ? 0 : ch) * 3 + mods[1]};
        if (slots.plan(nm, keys, slot, need)) {
          if (!mbar_wait(sm, &sm.slot_ready, refills & 1u)) { dead = true; break; }
          refills++;
        }
        if (elect_one()) {   // one thread of the converged warp: the compiler keeps the operands in uniform registers
          asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");   // the landed copies -> tensor-core reads
          asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
          for (int mi = 0; mi < nm; mi++) {
            // the windows [w_lo, w_hi] of the tile that hold this modality are the N extent of the MMAs
            const unsigned wm = tm.winmask[mods[mi]];
            const int w_lo = __ffs(wm) - 1, w_hi = 31 - __clz(wm);
            const uint32_t n_ext = 32u * (uint32_t)(w_hi - w_lo + 1);
            const uint32_t idesc = (1u << 4) | ((n_ext >> 3) << 17) | ((128u >> 4) << 24);   // D fp32, A/B fp16 K-major, M = 128
            const uint32_t dcol = tmem + a * 256u + (uint32_t)mi * 128u + 32u * (uint32_t)w_lo;
            const uint64_t da0 = make_desc(smem_u32(sm.b[slot[mi]][0]), 2048, 128);                   // R: M = output channel
            const uint64_t da1 = make_desc(smem_u32(sm.b[slot[mi]][1]), 2048, 128);
            const uint64_t db0 = make_desc_sw128(smem_u32(sm.a[buf]) + 4096u * (uint32_t)w_lo);       // values: N = token
#pragma unroll
            for (int k = 0; k < 16; k++) {
              // next 16 input channels: 4096 bytes further in R; 32 bytes further inside a value row, the second
              // 64 channels in the tile's second half
              const uint64_t da = (k < 8 ? da0 : da1) + (uint64_t)((k & 7) * (4096 >> 4));
              const uint64_t db = db0 + (uint64_t)(((k & 3) * 32 + ((k >> 2) & 1) * (TILE_BYTES / 2)) >> 4);
              asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                           "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}\n"
                           ::"r"(dcol), "l"(da), "l"(db), "r"(idesc), "r"(k ? 1u : 0u), "r"(0u) : "memory");
            }
          }
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(smem_u32(&sm.mma_done[a])) : "memory");
        }
        __syncwarp();
        jobidx++;
      }
      step_coords();
    }
    // nothing may be in flight when tensor memory is released: the last committed job is waited for whatever the
    // abort flag says (every issued product belongs to a committed job); if even that does not answer, tensor
    // memory stays allocated
    if (jobidx >= 1 && !mbar_drain(&sm.mma_done[(jobidx - 1u) & 1u], ((jobidx - 1u) >> 1) & 1u)) sm.tmem_busy = 1;
  } else {
    // ------------------------------------------------------------------ worker warps
    // norm role: token rows 32*eq + lane, channels [32 q, 32 q + 32); epilogue role: channels 32*eq + lane (the
    // warp's tensor-memory lane quarter), window ewq
    const int eq = warp & 3, ewq = warp >> 2;
    Slots slots;
    uint32_t jobidx = 0;
    bool dead = false;
    for (int i = 0; i < my_tiles && !dead; i++) {
      const int buf = i & 1;
      const uint32_t par = (uint32_t)(i >> 1) & 1u;
      if (!mbar_wait(sm, &sm.full[buf], par)) break;
      const TileMods tm = tile_mods(sm.mod[buf], lane);
      const unsigned mymod = sm.mod[buf][32 * ewq + lane];   // token `lane` of this warp's window
      const int wins = min(4, n_win - cwin0);
      {
        // Sum of squares with the exact adjacent-pair tree, split so that shared-memory reads are free of bank
        // conflicts: a 16-byte chunk (8 channels) is three levels of the tree, the warp's four chunks two more;
        // the last two levels (p0 + p1) + (p2 + p3) follow below.
        const int row = 32 * eq + lane, q = ewq;
        float part[4];
#pragma unroll
        for (int c = 0; c < 4; c++) {
          const uint4 raw = *reinterpret_cast<const uint4*>(sm.a[buf] + vtile_off(row, 4 * q + c));
          const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
          float2 x0 = __half22float2(h2[0]), x1 = __half22float2(h2[1]), x2 = __half22float2(h2[2]), x3 = __half22float2(h2[3]);
          float s0 = __fadd_rn(__fmul_rn(x0.x, x0.x), __fmul_rn(x0.y, x0.y));
          float s1 = __fadd_rn(__fmul_rn(x1.x, x1.x), __fmul_rn(x1.y, x1.y));
          float s2 = __fadd_rn(__fmul_rn(x2.x, x2.x), __fmul_rn(x2.y, x2.y));
          float s3 = __fadd_rn(__fmul_rn(x3.x, x3.x), __fmul_rn(x3.y, x3.y));
          part[c] = __fadd_rn(__fadd_rn(s0, s1), __fadd_rn(s2, s3));
        }
        sm.part[buf][q][row] = __fadd_rn(__fadd_rn(part[0], part[1]), __fadd_rn(part[2], part[3]));
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.part_ready[buf]);
      }
      if (!mbar_wait(sm, &sm.part_ready[buf], par)) break;
      if (ewq < wins) {
        // lane: norm of token `lane` of the window; the warp needs all 32 factors -1 / (3 T norm)
        const int tok = 32 * ewq + lane;
        const float sum = __fadd_rn(__fadd_rn(sm.part[buf][0][tok], sm.part[buf][1][tok]),
                                    __fadd_rn(sm.part[buf][2][tok], sm.part[buf][3][tok]));
        float n = __fsqrt_rn(sum);
        n = n > 65504.0f ? 65504.0f : n;
        const __half nh16 = __float2half_rn(n);
        const float nf = __half2float(nh16);
        if (eq == 0) reinterpret_cast<__half*>(cv.body(layer, cb, ch, cwin0 + ewq) + B_VNORM)[norm_pos(lane)] = nh16;
        const float inv = nf != 0.0f ? __fdiv_rn(1.0f, nf) : 0.0f;
        sm.inv[warp][lane] = inv;
        sm.c3[warp][lane] = __fmul_rn(inv, NEG_INV_3T);
      }
      __syncwarp();
      uint32_t wacc[4] = {0u, 0u, 0u, 0u};   // this channel's codes of the window, one word per t (sh = 0 position)
      for (int jt = 0; jt < 2; jt++) {
        int mods[2] = {0, 0};
        const int nm = job_mods(tm.present, jt, mods);
        if (nm == 0) break;
        const uint32_t a = jobidx & 1u;
        {
          // A rotation matrix this job needs is not resident: split R_m into fp16 hi + lo, laid out as the A
          // operand (row = output channel, K = input channel).  Every MMA issued so far has completed (this warp
          // has waited for each), and the job's own MMAs wait for slot_ready.
          int slot[2];
          bool need[2];
          const int keys[2] = {(n_R == 1 ? 0 : ch) * 3 + mods[0], (n_R == 1 ? 0 : ch) * 3 + mods[1]};
          if (slots.plan(nm, keys, slot, need)) {
            for (int mi = 0; mi < nm; mi++) {
              if (!need[mi]) continue;
              const float* Rm = R + (size_t)keys[mi] * D * D;
              for (int idx = tid; idx < D * D / 8; idx += NT) {
                const int n = idx >> 4, kc = idx & 15;
                const float4 x0 = __ldg(reinterpret_cast<const float4*>(Rm + n * D + kc * 8));
                const float4 x1 = __ldg(reinterpret_cast<const float4*>(Rm + n * D + kc * 8 + 4));
                const float xs[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
                __align__(16) __half hi[8], lo[8];
#pragma unroll
                for (int u = 0; u < 8; u++) {
                  hi[u] = __float2half_rn(xs[u]);
                  lo[u] = __float2half_rn(xs[u] - __half2float(hi[u]));
                }
                const uint32_t off = tile_off(n, kc * 8);
                *reinterpret_cast<uint4*>(sm.b[slot[mi]][0] + off) = *reinterpret_cast<const uint4*>(hi);
                *reinterpret_cast<uint4*>(sm.b[slot[mi]][1] + off) = *reinterpret_cast<const uint4*>(lo);
              }
            }
            asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");   // generic-proxy writes -> tensor-core reads
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.slot_ready);
          }
        }
        if (!mbar_wait(sm, &sm.mma_done[a], (jobidx >> 1) & 1u)) { dead = true; break; }
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        const bool last_job = jt == 1 || __popc(tm.present) < 3;
        // the tile's MMAs are complete and this warp keeps what it needs of the buffer in registers (the rare exact
        // recomputation below reads its value row from global memory)
        if (last_job && lane == 0) mbar_arrive(&sm.empty[buf]);
        if (ewq < wins) {
          for (int mi = 0; mi < nm; mi++) {
            const unsigned keep = __ballot_sync(0xffffffffu, mymod == (unsigned)mods[mi]);   // bit i: token i
            if (!keep) continue;
            uint32_t r[32];
            const uint32_t taddr = tmem + ((uint32_t)(eq * 32) << 16) + a * 256u + (uint32_t)mi * 128u + (uint32_t)ewq * 32u;
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
                         : "=r"(r[0]),"=r"(r[1]),"=r"(r[2]),"=r"(r[3]),"=r"(r[4]),"=r"(r[5]),"=r"(r[6]),"=r"(r[7]),"=r"(r[8]),"=r"(r[9]),"=r"(r[10]),"=r"(r[11]),"=r"(r[12]),"=r"(r[13]),"=r"(r[14]),"=r"(r[15]),
                           "=r"(r[16]),"=r"(r[17]),"=r"(r[18]),"=r"(r[19]),"=r"(r[20]),"=r"(r[21]),"=r"(r[22]),"=r"(r[23]),"=r"(r[24]),"=r"(r[25]),"=r"(r[26]),"=r"(r[27]),"=r"(r[28]),"=r"(r[29]),"=r"(r[30]),"=r"(r[31])
                         : "r"(taddr) : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
            // token i = 8*j + 2*t + e sits in word t at bit 16*e + 2*j (+ 8 for the second channel of the word)
            uint32_t kaccA[4] = {0u, 0u, 0u, 0u}, kaccB[4] = {0u, 0u, 0u, 0u};
            const float4* c3p = reinterpret_cast<const float4*>(sm.c3[warp]);
#pragma unroll
            for (int i4 = 0; i4 < 8; i4++) {
              const float4 c4 = c3p[i4];
              const float cs[4] = {c4.x, c4.y, c4.z, c4.w};
#pragma unroll
              for (int u = 0; u < 4; u++) {
                const int t4 = 4 * i4 + u;
                float va, vb, ka, kb;
                asm("fma.rn.sat.f32 %0, %1, %2, %3;\n" : "=f"(va) : "f"(__uint_as_float(r[t4])), "f"(cs[u]), "f"(TWO_THIRDS - BAND_V));
                asm("fma.rn.sat.f32 %0, %1, %2, %3;\n" : "=f"(vb) : "f"(__uint_as_float(r[t4])), "f"(cs[u]), "f"(TWO_THIRDS + BAND_V));
                asm("fma.rm.f32 %0, %1, %2, %3;\n" : "=f"(ka) : "f"(va), "f"(3.0f), "f"(FLOOR_MAGIC));
                asm("fma.rm.f32 %0, %1, %2, %3;\n" : "=f"(kb) : "f"(vb), "f"(3.0f), "f"(FLOOR_MAGIC));
                kaccA[(t4 & 7) >> 1] += __float_as_uint(ka) << (16 * (t4 & 1) + 2 * (t4 >> 3));
                kaccB[(t4 & 7) >> 1] += __float_as_uint(kb) << (16 * (t4 & 1) + 2 * (t4 >> 3));
              }
            }
#pragma unroll
            for (int t = 0; t < 4; t++) {
              // kacc = sum of (magic bits + k) << pos over the word's eight tokens; codes = 3 - k per field
              uint32_t codes = 0x00ff00ffu - (kaccA[t] - MAGIC_SUM);
              uint32_t differ = codes ^ (0x00ff00ffu - (kaccB[t] - MAGIC_SUM));
              uint32_t km = 0x00ff00ffu;
              if (keep != 0xffffffffu) {   // mixed-modality window: only this modality's tokens
                km = 0;
#pragma unroll
                for (int j = 0; j < 4; j++)
#pragma unroll
                  for (int e = 0; e < 2; e++) km |= ((keep >> (8 * j + 2 * t + e)) & 1u) * (3u << (16 * e + 2 * j));
              }
              codes &= km;
              differ &= km;
              while (differ) {   // rare: a coordinate within BAND of a threshold takes the reference arithmetic
                const int pos = (__ffs(differ) - 1) & ~1;               // bit 16 e + 2 j of the field
                const int tok = 8 * ((pos & 15) >> 1) + 2 * t + (pos >> 4);
                const int c = 32 * eq + lane, mu = c >> 4, sh = (c >> 3) & 1, g = c & 7;
                const __half* xrow = vrows + cb * vs_b + ch * vs_h + (long long)((cwin0 + ewq) * W + tok) * vs_t;
                const float* rrow = R + (size_t)((n_R == 1 ? 0 : ch) * 3 + mods[mi]) * D * D + (size_t)c * D;
                const int slot_i = atomicAdd(&sm.fix_count, 1);
                if (slot_i < FIX_MAX) {   // later, by a whole warp (the code written now is one of the two neighbouring levels)
                  FixItem& it = sm.fix[slot_i];
                  it.word = reinterpret_cast<uint32_t*>(cv.body(layer, cb, ch, cwin0 + ewq) + B_VCODE) +
                            vword_index((mu >> 2) * 128 + (4 * g + t) * 4 + (mu & 3));
                  it.xrow = xrow; it.rrow = rrow; it.inv = sm.inv[warp][tok]; it.bit = pos + 8 * sh;
                } else {                  // the list is full: here and now
                  float a = 0.0f;
#pragma unroll 4
                  for (int kc = 0; kc < 16; kc++) {
                    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(xrow) + kc);
                    const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
                    const float4 r0 = __ldg(reinterpret_cast<const float4*>(rrow) + 2 * kc), r1 = __ldg(reinterpret_cast<const float4*>(rrow) + 2 * kc + 1);
                    const float2 x0 = __half22float2(h2[0]), x1 = __half22float2(h2[1]), x2 = __half22float2(h2[2]), x3 = __half22float2(h2[3]);
                    a = __fmaf_rn(r0.x, x0.x, a); a = __fmaf_rn(r0.y, x0.y, a); a = __fmaf_rn(r0.z, x1.x, a); a = __fmaf_rn(r0.w, x1.y, a);
                    a = __fmaf_rn(r1.x, x2.x, a); a = __fmaf_rn(r1.y, x2.y, a); a = __fmaf_rn(r1.z, x3.x, a); a = __fmaf_rn(r1.w, x3.y, a);
                  }
                  const float z = __fmul_rn(a, sm.inv[warp][tok]);
                  const uint32_t code = (uint32_t)((z > -CB_THRESH) + (z > 0.0f) + (z > CB_THRESH));
                  codes = (codes & ~(3u << pos)) | (code << pos);
                }
                differ &= ~(3u << pos);
              }
              wacc[t] |= codes;
            }
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.acc_free[a]);
        jobidx++;
      }
      if (dead) break;
      if (ewq < wins) {
        // join the two channels of each word (c and c ^ 8 are eight lanes apart) and store: channel
        // c = 16*mu + 8*sh + g writes the words t = 2*sh, 2*sh + 1 of (mu, g)
        const int c = 32 * eq + lane, mu = c >> 4, sh = (c >> 3) & 1, g = c & 7;
        uint32_t* words = reinterpret_cast<uint32_t*>(cv.body(layer, cb, ch, cwin0 + ewq) + B_VCODE);
#pragma unroll
        for (int t = 0; t < 4; t++) {
          const uint32_t own = wacc[t] << (8 * sh);
          const uint32_t full = own | __shfl_xor_sync(0xffffffffu, own, 8);
          if ((t >> 1) == sh) words[vword_index((mu >> 2) * 128 + (4 * g + t) * 4 + (mu & 3))] = full;
        }
      }
      __syncwarp();   // sm.c3[warp] is rewritten for the next tile
      step_coords();
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  // ---- the listed coordinates, one per warp at a time: the two rows go through the warp's corner of the (idle) first
  // tile buffer, every lane evaluates the same chain (input index ascending, one rounding per step), lane 0 patches
  {
    const int n_fix = min(sm.fix_count, FIX_MAX);
    unsigned char* scr = sm.a[0] + warp * 1024;
    for (int i = warp; i < n_fix && !sm.abort; i += NT_ALL / 32) {
      const FixItem it = sm.fix[i];
      *reinterpret_cast<float4*>(scr + 16 * lane) = __ldg(reinterpret_cast<const float4*>(it.rrow) + lane);
      if (lane < 16) *reinterpret_cast<uint4*>(scr + 512 + 16 * lane) = __ldg(reinterpret_cast<const uint4*>(it.xrow) + lane);
      __syncwarp();
      float a = 0.0f;
#pragma unroll 4
      for (int kc = 0; kc < 16; kc++) {
        const uint4 raw = *reinterpret_cast<const uint4*>(scr + 512 + 16 * kc);
        const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
        const float4 r0 = *reinterpret_cast<const float4*>(scr + 32 * kc), r1 = *reinterpret_cast<const float4*>(scr + 32 * kc + 16);
        const float2 x0 = __half22float2(h2[0]), x1 = __half22float2(h2[1]), x2 = __half22float2(h2[2]), x3 = __half22float2(h2[3]);
        a = __fmaf_rn(r0.x, x0.x, a); a = __fmaf_rn(r0.y, x0.y, a); a = __fmaf_rn(r0.z, x1.x, a); a = __fmaf_rn(r0.w, x1.y, a);
        a = __fmaf_rn(r1.x, x2.x, a); a = __fmaf_rn(r1.y, x2.y, a); a = __fmaf_rn(r1.z, x3.x, a); a = __fmaf_rn(r1.w, x3.y, a);
      }
      const float z = __fmul_rn(a, it.inv);
      const uint32_t code = (uint32_t)((z > -CB_THRESH) + (z > 0.0f) + (z > CB_THRESH));
      if (lane == 0) {
        atomicAnd(it.word, ~(3u << it.bit));
        atomicOr(it.word, code << it.bit);
      }
      __syncwarp();
    }
  }
  if (tid == 0 && sm.abort) atomicCAS(cv.status, 0, (int)OKQ_ERR_TIMEOUT);
  if (warp == 0 && !sm.tmem_busy) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;\n" ::"r"(tmem) : "memory");
}

namespace {

using EncodeTiledFn = decltype(&cuTensorMapEncodeTiled);

// cuTensorMapEncodeTiled, looked up through the runtime (no link against the driver library)
EncodeTiledFn encode_tiled() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

}  // namespace

okq_status launch_quantize_values_tc(const CacheView& cv, int layer, const __half* v, const int64_t strides[3],
                                     const unsigned char* modality, int n_tokens, int n_win, const float* R, int n_R,
                                     int n_sm, cudaStream_t s, long long wait_limit, int skip_tile) {
  static thread_local unsigned long long attr_mask = 0;
  int attr_dev = 0;
  if (attr_needed(attr_mask, attr_dev)) {
    cudaError_t e = cudaFuncSetAttribute(k_quantize_values_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)sizeof(TcSmem) + 1024);
    if (e != cudaSuccess) { set_last_cuda_error((int)e); return OKQ_ERR_CUDA; }
    attr_done(attr_mask, attr_dev);
  }
  const long long n_tiles = (long long)((n_win + 3) / 4) * cv.n_kv_heads * cv.batch;
  if (n_tiles == 0) return OKQ_OK;
  // the values as a 4-d tensor [batch][head][token][channel] for the copy engine; a box is 64 channels x 128 tokens
  EncodeTiledFn enc = encode_tiled();
  if (!enc) { set_last_cuda_error((int)cudaErrorNotSupported); return OKQ_ERR_CUDA; }
  CUtensorMap vmap;
  const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)n_tokens, (cuuint64_t)cv.n_kv_heads, (cuuint64_t)cv.batch};
  // a dimension of extent 1 is never stepped: give it any legal stride
  const cuuint64_t gstr[3] = {(cuuint64_t)(n_tokens > 1 ? strides[2] : D) * 2, (cuuint64_t)(cv.n_kv_heads > 1 ? strides[1] : D) * 2,
                              (cuuint64_t)(cv.batch > 1 ? strides[0] : D) * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)TILE, 1, 1}, estr[4] = {1, 1, 1, 1};
  for (int i = 0; i < 3; i++)
    if (gstr[i] == 0 || gstr[i] % 16 || gstr[i] >= (1ull << 40)) return OKQ_ERR_UNSUPPORTED;
  const CUresult cr = enc(&vmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<__half*>(v), dims, gstr, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) { set_last_cuda_error((int)cudaErrorInvalidValue); return OKQ_ERR_CUDA; }
  const int grid = (int)(n_tiles < n_sm ? n_tiles : n_sm);
  k_quantize_values_tc<<<grid, NT_ALL, sizeof(TcSmem) + 1024, s>>>(vmap, cv, layer, modality, n_tokens, n_win, R, n_R, v, (long long)strides[0],
                                                                   (long long)strides[1], (long long)strides[2], wait_limit > 0 ? wait_limit : WAIT_LIMIT_CLOCKS, skip_tile);
  return OKQ_OK;
}

}  // namespace okq
