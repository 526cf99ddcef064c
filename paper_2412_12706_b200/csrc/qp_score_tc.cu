// S1 on the 5th-generation tensor cores: the window-score sweeps with tcgen05.mma and TMEM.
//
// One thread block owns 128 window-query rows (M) of one (batch, KV head) and walks over a run of
// 128-key tiles (N).  Per tile a single thread issues D/16 tcgen05.mma (bf16 x bf16 -> f32, both
// operands K-major in shared memory with the 128-byte swizzle), the [128 x 128] logit tile lands in
// tensor memory, and the four warps read it back with tcgen05.ld: TMEM lane = query row, so every
// thread owns one row (two warpgroups split the columns) and the softmax statistics of sweep 1 need
// no shuffles at all.  Sweep 2 swaps the operands (TMEM lane = key, column = query row), so the vote
// of a key is again a thread-local sum.
// Two TMEM buffers and two shared-memory stages let the MMA of tile i+1 and the copy of tile i+2
// run under the epilogue of tile i.
//
// Every wait on an mbarrier is bounded: if it runs out, the block records an error word, frees its
// tensor memory and returns.  Outputs and their layout are the ones of score_sweep_kernel.
#include "qp_mma.cuh"

namespace qp {

namespace {

constexpr int TC_THREADS = 256;                     // two warpgroups: each reads half of the tile's columns
constexpr int TC_M = 128, TC_N = 128;
constexpr uint32_t TC_TMEM_COLS = 256;                // two accumulator buffers of 128 columns
constexpr uint32_t TC_SPIN_LIMIT = 1u << 22;

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// bounded wait; false = gave up
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < TC_SPIN_LIMIT; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}

// shared-memory matrix descriptor: K-major, 128-byte swizzle, 8-row groups 1024 B apart
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3ffffu) >> 4);           // start address, 16-byte units
  d |= (uint64_t)1 << 16;                             // leading-dimension byte offset (unused with swizzle): 1
  d |= (uint64_t)(1024 >> 4) << 32;                   // stride between 8-row groups
  d |= (uint64_t)1 << 46;                             // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                             // 128-byte swizzle
  return d;
}
// instruction descriptor: D = f32, A = B = bf16, both K-major, M x N
__host__ __device__ constexpr uint32_t instr_desc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}\n" ::"r"(tmem_d),
      "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
// 2^x by the hardware approximation (about 2 ulp; results below 2^-126 flush to 0)
__device__ __forceinline__ float ex2a(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void cp_async16_zfill(uint32_t saddr, const void* gptr, bool valid) {
  const int n = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(saddr), "l"(gptr), "r"(n));
}

// byte offset of 16-byte chunk c (8 bf16) of row r inside a [128 rows x D] operand: D/64 blocks of
// [128 rows x 128 B], each made of 8-row groups of 1024 B with the chunk index XORed by the row
__device__ __forceinline__ uint32_t sw128_off(int r, int c) {
  return (uint32_t)((c >> 3) * (TC_M * 128) + (r >> 3) * 1024 + (r & 7) * 128 + (((c & 7) ^ (r & 7)) << 4));
}

template <int PASS, int D, int NL>
__global__ void __launch_bounds__(TC_THREADS, 2)
score_sweep_tc_kernel(const __grid_constant__ ScorePtrs<NL> ptrs, int bh0, int BH, int Hq, int Hkv, int L, int w,
                      int n_rb, int n_tiles, int tiles_per_block, float scale_log2,
                      float2* __restrict__ stat_partial, const float2* __restrict__ rowstat,
                      float* __restrict__ votes_partial, int* __restrict__ error_word) {
  constexpr int CPR = D / 8;                           // 16-byte chunks per row
  constexpr uint32_t OPER_BYTES = TC_M * D * 2;        // one operand tile: D/64 swizzled blocks of 16 KB
  extern __shared__ unsigned char smem_raw[];
  __shared__ uint64_t bars[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int give_up;
  __shared__ float sVote[PASS == 2 ? 2 : 1][TC_N];
  __shared__ __align__(16) float2 sRow[PASS == 2 ? TC_M : 1];      // sweep 2: (M, 1/Z) of the block's rows

  const int tid = threadIdx.x, warp = tid >> 5;
  const int rloc = tid & (TC_M - 1), half = tid >> 7, wq = warp & 3;   // row in the block, column half, TMEM lane quarter
  // bh counts (layer, batch, KV head): the scratch arrays are laid out over all of them, the inputs are per layer
  const int split = blockIdx.x, rb = blockIdx.y, bh = bh0 + blockIdx.z, layer = bh / BH, bhl = bh % BH;
  const bf16* __restrict__ Qwin = ptrs.q[layer];
  const bf16* __restrict__ K = ptrs.k[layer];
  const int b = bhl / Hkv, hk = bhl % Hkv, G = Hq / Hkv, P = L - w, R = G * w;
  const int tile_lo = split * tiles_per_block;
  const int n_vis = PASS == 1 ? n_tiles : (P + TC_N - 1) / TC_N;    // sweep 2 only needs prefix columns
  const int tile_hi = min(n_vis, tile_lo + tiles_per_block);
  if (tile_lo >= tile_hi) return;
  const int n_loc = tile_hi - tile_lo;

  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;     // operands need 1024-byte alignment
  const uint32_t sQ = sbase, sK0 = sbase + OPER_BYTES;              // then two K stages
  const uint32_t bar0 = smem_u32(&bars[0]);

  if (tid == 0) {
    mbar_init(bar0, 1);
    mbar_init(bar0 + 8, 1);
    give_up = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(TC_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }

  // stage a [128 x D] bf16 operand (rows beyond `rows_valid` are zero)
  auto stage_rows = [&](uint32_t dst, const bf16* src, int rows_valid) {
#pragma unroll
    for (int i = 0; i < TC_M * CPR / TC_THREADS; ++i) {
      const int idx = tid + TC_THREADS * i, r = idx / CPR, c = idx % CPR;
      const bool ok = r < rows_valid;
      cp_async16_zfill(dst + sw128_off(r, c), src + (ok ? (size_t)r * D + c * 8 : 0), ok);
    }
  };
  const bf16* Qh = Qwin + ((size_t)(b * Hq + hk * G) * w + (size_t)rb * TC_M) * D;
  const bf16* Kh = K + (size_t)bhl * L * D;
  stage_rows(sQ, Qh, min(TC_M, R - rb * TC_M));
  stage_rows(sK0, Kh + (size_t)tile_lo * TC_N * D, min(TC_N, L - tile_lo * TC_N));
  cp_async_commit();
  if (n_loc > 1) stage_rows(sK0 + OPER_BYTES, Kh + (size_t)(tile_lo + 1) * TC_N * D, min(TC_N, L - (tile_lo + 1) * TC_N));
  cp_async_commit();

  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
  const uint32_t tmem_base = tmem_base_slot;
  constexpr uint32_t IDESC = instr_desc(TC_M, TC_N);

  // issue the D/16 MMAs of local tile j (shared-memory stage j & 1 -> TMEM buffer j & 1)
  auto issue_mma = [&](int j) {
    const uint32_t sK = sK0 + (j & 1) * OPER_BYTES, tm = tmem_base + (j & 1) * TC_N;
#pragma unroll
    for (int kb = 0; kb < D / 64; ++kb)
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (PASS == 1)      // rows = queries, columns = keys
          umma_bf16(tm, smem_desc(sQ + kb * (TC_M * 128) + k * 32), smem_desc(sK + kb * (TC_N * 128) + k * 32), IDESC,
                    (kb | k) ? 1u : 0u);
        else                // rows = keys, columns = queries
          umma_bf16(tm, smem_desc(sK + kb * (TC_N * 128) + k * 32), smem_desc(sQ + kb * (TC_M * 128) + k * 32), IDESC,
                    (kb | k) ? 1u : 0u);
    umma_commit(bar0 + (j & 1) * 8);
  };

  // this thread's query row and its statistics
  const int row = rb * TC_M + rloc;
  const int lim = min(P + (row % w), L - 1);            // last key this row may see
  if (PASS == 2 && tid < TC_M) sRow[tid] = rowstat[(size_t)(bh * n_rb + rb) * TC_M + tid];   // visible after the next barrier

  cp_async_wait<1>();                                   // Q and the first K tile have landed
  asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
  __syncthreads();
  if (tid == 0) issue_mma(0);

  for (int j = 0; j < n_loc; ++j) {
    if (j + 1 < n_loc) {                                // next tile's operands -> MMA under this tile's epilogue
      cp_async_wait<0>();
      asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
      __syncthreads();
      if (tid == 0) issue_mma(j + 1);
    }
    const bool ok = mbar_wait(bar0 + (j & 1) * 8, (j >> 1) & 1);
    if (!ok) give_up = 1;
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    __syncthreads();                                    // everyone sees the outcome; stage j & 1 is free again
    if (give_up) break;
    if (j + 2 < n_loc) {
      const int tl = tile_lo + j + 2;
      stage_rows(sK0 + (j & 1) * OPER_BYTES, Kh + (size_t)tl * TC_N * D, min(TC_N, L - tl * TC_N));
    }
    cp_async_commit();

    const int tile = tile_lo + j, key0 = tile * TC_N;
    const uint32_t taddr = tmem_base + ((uint32_t)(wq * 32) << 16) + (j & 1) * TC_N + half * (TC_N / 2);
    const int col0 = key0 + half * (TC_N / 2);
    if constexpr (PASS == 1) {
      // TMEM lane = query row: this thread folds its row's 64 columns into a running (max, sum)
      float m = -INFINITY, s = 0.f;
      const bool all_visible = key0 + TC_N - 1 <= P;            // every row sees every key up to P
#pragma unroll 1
      for (int c0 = 0; c0 < TC_N / 2; c0 += 32) {
        float v[32];
        tmem_ld32(taddr + c0, v);
        if (all_visible) {
          float cm = v[0];
#pragma unroll
          for (int i = 1; i < 32; ++i) cm = fmaxf(cm, v[i]);
          const float mn = fmaxf(m, cm * scale_log2);           // scale > 0: max commutes with it
          float acc = 0.f;
#pragma unroll
          for (int i = 0; i < 32; ++i) acc += ex2a(fmaf(v[i], scale_log2, -mn));
          s = fmaf(s, ex2a(m - mn), acc);
          m = mn;
        } else {
          float cm = -INFINITY;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            v[i] = col0 + c0 + i <= lim ? v[i] * scale_log2 : -INFINITY;
            cm = fmaxf(cm, v[i]);
          }
          if (cm != -INFINITY) {
            const float mn = fmaxf(m, cm);
            float acc = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i) acc += ex2a(v[i] - mn);
            s = fmaf(s, ex2a(m - mn), acc);
            m = mn;
          }
        }
      }
      // one (max, sum) per row and 64-column half tile
      stat_partial[(((size_t)(bh * n_rb + rb) * n_tiles + tile) * 2 + half) * TC_M + rloc] = make_float2(m, s);
    } else {
      // operands swapped: TMEM lane = key, column = query row, so a key's vote is a thread-local sum over
      // the rows.  Only prefix keys (< P) are written and every row sees all of them: no mask needed;
      // rows beyond R carry 1/Z = 0.
      float vote = 0.f;
#pragma unroll 1
      for (int c0 = 0; c0 < TC_N / 2; c0 += 32) {
        float v[32];
        tmem_ld32(taddr + c0, v);
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float4 ms = *reinterpret_cast<const float4*>(&sRow[half * (TC_N / 2) + c0 + i]);   // (M, 1/Z) x 2 rows
          vote = fmaf(ex2a(fmaf(v[i], scale_log2, -ms.x)), ms.y, vote);
          vote = fmaf(ex2a(fmaf(v[i + 1], scale_log2, -ms.z)), ms.w, vote);
        }
      }
      sVote[half][rloc] = vote;
      __syncthreads();
      if (tid < TC_N && key0 + tid < P)
        votes_partial[(size_t)(bh * n_rb + rb) * P + key0 + tid] = sVote[0][tid] + sVote[1][tid];
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();                                    // TMEM buffer j & 1 and sVote may be overwritten
  }

  cp_async_wait<0>();
  if (give_up && tid == 0) atomicExch(error_word, 1);
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(TC_TMEM_COLS) : "memory");
  }
}

}  // namespace

bool score_tc_supported(int D) { return D == 128 || D == 64; }

namespace {
template <int PASS, int D, int NL>
cudaError_t launch_tc(dim3 grid, int bh0, cudaStream_t st, const ScorePtrs<NL>& ptrs, const ScoreDims& d, const ScoreWorkspace& s,
                      int per, float scale_log2, float2* stat_partial, const float2* rowstat, float* votes_partial,
                      int* error_word) {
  constexpr size_t smem = 3 * (size_t)TC_M * D * 2 + 1024;   // Q + two K stages + alignment slack
  static unsigned char done[64] = {};
  const cudaError_t e = allow_smem(score_sweep_tc_kernel<PASS, D, NL>, smem, done);
  if (e != cudaSuccess) return e;
  score_sweep_tc_kernel<PASS, D, NL><<<grid, TC_THREADS, smem, st>>>(ptrs, bh0, d.Bt * d.Hkv, d.Hq, d.Hkv, d.L, d.w, s.n_rb,
                                                                    s.n_tiles, per, scale_log2, stat_partial, rowstat,
                                                                    votes_partial, error_word);
  return cudaGetLastError();
}

template <int NL>
cudaError_t launch_sweep(int pass, const ScorePtrs<NL>& ptrs, int bh0, int BH, const ScoreDims& d, const ScoreWorkspace& s,
                         float scale_log2, float2* stat_partial, const float2* rowstat, float* votes_partial,
                         int* error_word, cudaStream_t st) {
  const int tiles = pass == 1 ? s.n_tiles : s.n_vote_tiles;
  // enough blocks for two per SM over a few waves, at least two tiles per block
  long long per = ((long long)tiles * s.n_rb * BH + 591) / 592;
  if (per < 2) per = 2;
  if (per > 32) per = 32;
  const int splits = (int)((tiles + per - 1) / per);
  const dim3 grid(splits, s.n_rb, BH);
  if (d.D == 128)
    return pass == 1 ? launch_tc<1, 128, NL>(grid, bh0, st, ptrs, d, s, (int)per, scale_log2, stat_partial, rowstat, votes_partial, error_word)
                     : launch_tc<2, 128, NL>(grid, bh0, st, ptrs, d, s, (int)per, scale_log2, stat_partial, rowstat, votes_partial, error_word);
  return pass == 1 ? launch_tc<1, 64, NL>(grid, bh0, st, ptrs, d, s, (int)per, scale_log2, stat_partial, rowstat, votes_partial, error_word)
                   : launch_tc<2, 64, NL>(grid, bh0, st, ptrs, d, s, (int)per, scale_log2, stat_partial, rowstat, votes_partial, error_word);
}
}  // namespace

// s: the scratch layout for batch * n_layers batch entries (the layers are stacked along the batch dimension)
// bh0, bh_count: the (layer, batch, KV head) triples this launch covers
cudaError_t launch_score_sweep_tc(int pass, int n_layers, const void* const* q, const void* const* k, const ScoreDims& d,
                                  const ScoreWorkspace& s, float scale_log2, float2* stat_partial, const float2* rowstat,
                                  float* votes_partial, int* error_word, cudaStream_t st, int bh0, int bh_count) {
  if (n_layers == 1) {
    ScorePtrs<1> p;
    p.q[0] = static_cast<const bf16*>(q[0]);
    p.k[0] = static_cast<const bf16*>(k[0]);
    return launch_sweep<1>(pass, p, bh0, bh_count, d, s, scale_log2, stat_partial, rowstat, votes_partial, error_word, st);
  }
  ScorePtrs<QP_MAX_LAYERS> p;
  for (int l = 0; l < n_layers; ++l) {
    p.q[l] = static_cast<const bf16*>(q[l]);
    p.k[l] = static_cast<const bf16*>(k[l]);
  }
  return launch_sweep<QP_MAX_LAYERS>(pass, p, bh0, bh_count, d, s, scale_log2, stat_partial, rowstat, votes_partial,
                                     error_word, st);
}

}  // namespace qp
