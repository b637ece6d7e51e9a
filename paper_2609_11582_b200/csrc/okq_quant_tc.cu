// Bulk value quantiser with the per-modality rotation on the 5th-generation tensor cores
// (Eq. 6 then Eq. 3 for whole prefill chunks).
//
// z = R_m v is a dense [tokens x 128] x [128 x 128] contraction.  A CTA takes tiles of 128
// consecutive tokens (four windows) of one (sequence, KV head):
//   * the fp16 values are the A operand as they are (exact), staged with cp.async into the
//     no-swizzle K-major core-matrix layout tcgen05.mma reads;
//   * R_m (fp32) is split into two fp16 matrices R_hi + R_lo, kept in shared memory while the
//     modality does not change; 16 tcgen05.mma (M=128, N=128, K=16) accumulate
//     v R_hi^T + v R_lo^T in fp32 in tensor memory;
//   * the epilogue reads each token's row with tcgen05.ld, scales by 1/norm, takes the three
//     threshold compares and packs the codes in the decode kernel's record order.
// The split leaves a relative error of about 2^-22 on z, the same size as the rounding of the
// fp32 fused-multiply-add chain the exact path uses, so a code can differ from the exact path
// only when z lies within ~1e-7 of a threshold.  Norms are computed with the exact summation
// tree and are bit-identical to the exact path.
//
// Every wait on the MMA-completion mbarrier is bounded; on a timeout the kernel records
// OKQ_ERR_TIMEOUT in the cache's status word, stops issuing work, frees its tensor memory and
// returns.
#include "okq_common.cuh"
#include "okq_device.cuh"

namespace okq {

namespace {

constexpr int TILE = 128;               // tokens per tile
constexpr int NT = 512;                 // worker threads per CTA: 16 warps, four per tensor-memory lane quarter
constexpr int NT_ALL = NT + 32;         // plus one warp that only issues the MMAs
constexpr int TILE_BYTES = TILE * D * 2;  // 32 KB: one fp16 operand tile

struct TcSmem {
  __align__(1024) unsigned char a[2][TILE_BYTES];      // value tiles (double buffered)
  __align__(1024) unsigned char b[2][2][TILE_BYTES];   // two resident matrices, each as R_hi, R_lo
  uint32_t cw[2][TILE][8];                             // codes of a tile: per token, 16 channels x 2 bits per word
  float inv[2][TILE];
  __align__(4) unsigned char mod[2][TILE];
  __align__(8) unsigned long long mbar;
  uint32_t tmem_slot;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

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

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(smem_u32(smem)), "l"(gmem));
}

// bounded wait for one phase of the MMA-completion barrier; each try lets the hardware suspend the
// thread for up to about a millisecond, so a completed MMA is normally seen by the first try
__device__ __forceinline__ bool mbar_wait(uint32_t mbar, uint32_t parity) {
  for (int it = 0; it < 4000; it++) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                 : "=r"(ok) : "r"(mbar), "r"(parity), "r"(1000000u) : "memory");
    if (ok) return true;
  }
  return false;
}

}  // namespace

// persistent grid, NT_ALL threads.  Tiles are numbered (b, h, tile-in-sequence), tile = 4 windows; a CTA
// owns a contiguous range of them.  A "job" is
// one (tile, modality present in the tile); the MMAs of job j run on the tensor cores while the
// threads do the epilogue (and packing) of job j-1 out of the other half of tensor memory.
__global__ void __launch_bounds__(NT_ALL, 1) k_quantize_values_tc(CacheView cv, int layer, const __half* __restrict__ v,
                                                             long long sb, long long sh, long long st,
                                                             const unsigned char* __restrict__ modality, int n_tokens,
                                                             const float* __restrict__ R, int n_R) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  TcSmem& sm = *reinterpret_cast<TcSmem*>(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool worker = tid < NT;            // warp 16 only issues MMAs
  const int n_win = n_tokens / W;
  const int tiles_per_unit = (n_win + 3) / 4;
  const int n_tiles_all = tiles_per_unit * cv.n_kv_heads * cv.batch;
  // contiguous tile range of this CTA
  const int per_cta = (n_tiles_all + gridDim.x - 1) / gridDim.x;
  const int tile_begin = min(n_tiles_all, (int)blockIdx.x * per_cta);
  const int n_tiles = min(n_tiles_all, tile_begin + per_cta);   // end of the range

  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(smem_u32(&sm.mbar)));
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;\n" ::"r"(smem_u32(&sm.tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
  const uint32_t tmem = sm.tmem_slot;
  // D fp32, A/B fp16, both K-major, N = 128, M = 128
  const uint32_t idesc = (1u << 4) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
  uint32_t phase = 0;
  int slot_key[2] = {-1, -1};   // (rotation set * 3 + modality) held by each resident slot
  int last_slot = 0;
  bool failed = false;          // uniform across the block

  auto tile_coords = [&](int tile, int& b, int& h, int& win0) {
    b = tile / (tiles_per_unit * cv.n_kv_heads);
    int rem = tile - b * tiles_per_unit * cv.n_kv_heads;
    h = rem / tiles_per_unit;
    win0 = (rem - h * tiles_per_unit) * 4;
  };
  auto issue_tile = [&](int tile, int buf, int b, int h, int win0) {
    if (tile < n_tiles && worker) {
      const int rows = min(TILE, (n_win - win0) * W);
      const __half* src = v + b * sb + h * sh + (long long)win0 * W * st;
      // a warp copies 8 rows x 4 chunks: 64 contiguous bytes per row on the global side, and one
      // 128-byte core matrix per chunk on the shared side (at most 4-way bank conflicts)
      for (int idx = tid; idx < TILE * 16; idx += NT) {
        const int r = (idx & 7) + 8 * ((idx >> 5) & 15), kc = ((idx >> 3) & 3) + 4 * (idx >> 9);
        if (r < rows) cp_async16(sm.a[buf] + tile_off(r, kc * 8), src + (long long)r * st + kc * 8);
      }
    }
    asm volatile("cp.async.commit_group;\n" ::);
  };

  // the tile being prefetched: coordinates and this thread's modality byte
  int nb = 0, nh = 0, nwin0 = 0;
  unsigned char next_mod = 0;
  auto fetch_next_mod = [&](int tile) {
    if (tile < n_tiles && tid < TILE) {
      const int nrows = min(TILE, (n_win - nwin0) * W);
      unsigned char m = 0;
      if (tid < nrows) m = modality[(size_t)nb * n_tokens + (size_t)nwin0 * W + tid];
      next_mod = m > 2 ? 0 : m;
    }
  };
  if (tile_begin < n_tiles) tile_coords(tile_begin, nb, nh, nwin0);
  fetch_next_mod(tile_begin);
  issue_tile(tile_begin, 0, nb, nh, nwin0);

  int tile = tile_begin, buf = 1;       // buf flips when a tile is set up
  int b = 0, h = 0, win0 = 0, wins = 0;
  unsigned pend = 0;                    // modalities of the current tile not yet issued
  int jobs = 0;
  // the previous job, whose accumulator is waiting for its epilogue
  bool p_valid = false, p_last = false;
  int p_buf = 0, p_mod = 0, p_acc = 0, p_b = 0, p_h = 0, p_win0 = 0, p_wins = 0;

  while (true) {
    // ---------------- prepare and issue the next job
    bool have_job = false;
    if (pend == 0 && tile < n_tiles) {
      buf ^= 1;
      b = nb; h = nh; win0 = nwin0;
      wins = min(4, n_win - win0);
      const int rows = wins * W;
      if (tid < TILE) sm.mod[buf][tid] = tid < rows ? next_mod : 255;
      const int ntile = tile + 1;
      if (ntile < n_tiles) {   // next tile of the range: step the coordinates, no divisions
        nwin0 += 4;
        if (nwin0 >= tiles_per_unit * 4) { nwin0 = 0; if (++nh == cv.n_kv_heads) { nh = 0; nb++; } }
      }
      fetch_next_mod(ntile);
      issue_tile(ntile, buf ^ 1, nb, nh, nwin0);                 // prefetch
      asm volatile("cp.async.wait_group 1;\n" ::: "memory");    // this tile has landed
      __syncthreads();
      // norms with the exact adjacent-pair summation tree, four threads per token, read from the staged
      // tile: a 16-byte chunk (8 channels) is three levels of the tree, a thread's four chunks two more,
      // the four threads of a token the last two (shuffles between neighbouring lanes)
      if (worker) {
        const int r = tid >> 2, q = tid & 3;
        float part[4];
#pragma unroll
        for (int i = 0; i < 4; i++) {
          const uint4 raw = *reinterpret_cast<const uint4*>(sm.a[buf] + tile_off(r, (4 * q + i) * 8));
          const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
          float2 x0 = __half22float2(h2[0]), x1 = __half22float2(h2[1]), x2 = __half22float2(h2[2]), x3 = __half22float2(h2[3]);
          float s0 = __fadd_rn(__fmul_rn(x0.x, x0.x), __fmul_rn(x0.y, x0.y));
          float s1 = __fadd_rn(__fmul_rn(x1.x, x1.x), __fmul_rn(x1.y, x1.y));
          float s2 = __fadd_rn(__fmul_rn(x2.x, x2.x), __fmul_rn(x2.y, x2.y));
          float s3 = __fadd_rn(__fmul_rn(x3.x, x3.x), __fmul_rn(x3.y, x3.y));
          part[i] = __fadd_rn(__fadd_rn(s0, s1), __fadd_rn(s2, s3));
        }
        float sum = __fadd_rn(__fadd_rn(part[0], part[1]), __fadd_rn(part[2], part[3]));
        sum = __fadd_rn(sum, __shfl_xor_sync(0xffffffffu, sum, 1));
        sum = __fadd_rn(sum, __shfl_xor_sync(0xffffffffu, sum, 2));
        if (q == 0 && r < rows) {
          float n = __fsqrt_rn(sum);
          n = n > 65504.0f ? 65504.0f : n;
          const __half nh16 = __float2half_rn(n);
          const float nf = __half2float(nh16);
          unsigned char* body = cv.body(layer, b, h, win0 + (r >> 5));
          reinterpret_cast<__half*>(body + B_VNORM)[norm_pos(r & 31)] = nh16;
          sm.inv[buf][r] = nf != 0.0f ? __fdiv_rn(1.0f, nf) : 0.0f;
        }
      }
      {
        const uint32_t m4 = reinterpret_cast<const uint32_t*>(sm.mod[buf])[lane];   // 4 tokens per lane
        unsigned mine = 0;
#pragma unroll
        for (int u = 0; u < 4; u++) {
          const unsigned mm = (m4 >> (8 * u)) & 0xffu;
          if (mm < 3) mine |= 1u << mm;
        }
#pragma unroll
        for (int d = 16; d; d >>= 1) mine |= __shfl_xor_sync(0xffffffffu, mine, d);
        pend = mine;
      }
    }
    int m = 0;
    if (pend) {
      m = __ffs(pend) - 1;
      pend &= ~(1u << m);
      const int key = (n_R == 1 ? 0 : h) * 3 + m;
      int slot = slot_key[0] == key ? 0 : (slot_key[1] == key ? 1 : -1);
      if (slot < 0) {
        // not resident: replace the slot that was not used last.  Split R_m into fp16 hi + lo, laid out
        // as the B operand (row = output channel, K = input channel)
        slot = last_slot ^ 1;
        const float* Rm = R + (size_t)key * D * D;
        for (int idx = tid; idx < (worker ? D * D / 8 : 0); idx += NT) {
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
          *reinterpret_cast<uint4*>(sm.b[slot][0] + off) = *reinterpret_cast<const uint4*>(hi);
          *reinterpret_cast<uint4*>(sm.b[slot][1] + off) = *reinterpret_cast<const uint4*>(lo);
        }
        slot_key[slot] = key;
      }
      last_slot = slot;
      asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");   // generic-proxy writes -> tensor-core reads
      asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
      __syncthreads();
      if (tid == NT) {
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        const uint32_t dcol = tmem + (uint32_t)(jobs & 1) * 128;
#pragma unroll 1
        for (int part = 0; part < 2; part++)
#pragma unroll 1
          for (int s = 0; s < 8; s++) {
            const uint64_t da = make_desc(smem_u32(sm.a[buf]) + s * 4096, 2048, 128);
            const uint64_t db = make_desc(smem_u32(sm.b[slot][part]) + s * 4096, 2048, 128);
            const uint32_t accumulate = (part | s) ? 1u : 0u;
            asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                         "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}\n"
                         ::"r"(dcol), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
          }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(smem_u32(&sm.mbar)) : "memory");
      }
      have_job = true;
    }

    // ---------------- epilogue of the previous job, while the tensor cores work on this one
    if (p_valid && worker) {
      // warp w reads tensor-memory lanes 32*(w&3).. (token rows) and the 32 columns (w>>2)*32.. (output
      // channels).  tcgen05.ld is warp-collective, so every lane reads; only tokens of the job's
      // modality keep the result.
      const int row = (warp & 3) * 32 + lane, cc = warp >> 2;
      const bool mine = sm.mod[p_buf][row] == p_mod;
      const float inv = sm.inv[p_buf][row];
      uint32_t r[32];
      const uint32_t taddr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)p_acc * 128 + cc * 32;
      asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
                   : "=r"(r[0]),"=r"(r[1]),"=r"(r[2]),"=r"(r[3]),"=r"(r[4]),"=r"(r[5]),"=r"(r[6]),"=r"(r[7]),"=r"(r[8]),"=r"(r[9]),"=r"(r[10]),"=r"(r[11]),"=r"(r[12]),"=r"(r[13]),"=r"(r[14]),"=r"(r[15]),
                     "=r"(r[16]),"=r"(r[17]),"=r"(r[18]),"=r"(r[19]),"=r"(r[20]),"=r"(r[21]),"=r"(r[22]),"=r"(r[23]),"=r"(r[24]),"=r"(r[25]),"=r"(r[26]),"=r"(r[27]),"=r"(r[28]),"=r"(r[29]),"=r"(r[30]),"=r"(r[31])
                   : "r"(taddr) : "memory");
      asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
      if (mine) {
#pragma unroll
        for (int half = 0; half < 2; half++) {
          uint32_t word = 0;
#pragma unroll
          for (int u = 0; u < 16; u++) {
            const float z = __fmul_rn(__uint_as_float(r[16 * half + u]), inv);
            word |= (uint32_t)((z > -CB_THRESH) + (z > 0.0f) + (z > CB_THRESH)) << (2 * u);
          }
          sm.cw[p_buf][row][2 * cc + half] = word;
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    }
    if (p_valid && p_last) {
      __syncthreads();   // all codes of the tile are in the buffer (every warp, the issuing one included)
      if (worker) {
        // pack the codes of each window in record order (value codes are the A operand of the decode kernel)
        for (int wi = tid; wi < p_wins * 256; wi += NT) {
          const int wq = wi >> 8, w8 = wi & 255;
          const int mu = (w8 >> 7) * 4 + (w8 & 3);
          const int l = (w8 & 127) >> 2;
          const int g = l >> 2, t = l & 3;
          uint32_t word = 0;
#pragma unroll
          for (int j = 0; j < 4; j++) {
#pragma unroll
            for (int e = 0; e < 2; e++) {
              const int i = 16 * (j >> 1) + 8 * (j & 1) + 2 * t + e;
              const uint32_t src = sm.cw[p_buf][wq * W + i][mu];          // channels 16*mu .. 16*mu+15 of token i
              word |= ((src >> (2 * g)) & 3u) << (16 * e + 2 * j);       // channel 16*mu + g
              word |= ((src >> (2 * (8 + g))) & 3u) << (16 * e + 8 + 2 * j);   // channel 16*mu + 8 + g
            }
          }
          reinterpret_cast<uint32_t*>(cv.body(layer, p_b, p_h, p_win0 + wq) + B_VCODE)[w8] = word;
        }
      }
    }
    if (!have_job) break;

    // ---------------- wait for this job's MMAs (warp 0 polls; the block barrier spreads the answer)
    const bool ok = __syncthreads_and(warp != 0 || mbar_wait(smem_u32(&sm.mbar), phase) ? 1 : 0) != 0;
    phase ^= 1;
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    if (!ok) { failed = true; break; }
    p_valid = true; p_last = pend == 0; p_buf = buf; p_mod = m; p_acc = jobs & 1;
    p_b = b; p_h = h; p_win0 = win0; p_wins = wins;
    jobs++;
    if (pend == 0) tile += 1;
  }
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");
  if (tid == 0 && failed) atomicCAS(cv.status, 0, (int)OKQ_ERR_TIMEOUT);
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;\n" ::"r"(tmem) : "memory");
}

okq_status launch_quantize_values_tc(const CacheView& cv, int layer, const __half* v, const int64_t strides[3],
                                     const unsigned char* modality, int n_tokens, const float* R, int n_R,
                                     int n_sm, cudaStream_t s) {
  static thread_local bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(k_quantize_values_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)sizeof(TcSmem) + 1024);
    if (e != cudaSuccess) { set_last_cuda_error((int)e); return OKQ_ERR_CUDA; }
    attr_set = true;
  }
  const int n_win = n_tokens / W;
  const long long n_tiles = (long long)((n_win + 3) / 4) * cv.n_kv_heads * cv.batch;
  if (n_tiles == 0) return OKQ_OK;
  const int grid = (int)(n_tiles < n_sm ? n_tiles : n_sm);
  k_quantize_values_tc<<<grid, NT_ALL, sizeof(TcSmem) + 1024, s>>>(cv, layer, v, strides[0], strides[1], strides[2],
                                                                modality, n_tokens, R, n_R);
  return OKQ_OK;
}

}  // namespace okq
