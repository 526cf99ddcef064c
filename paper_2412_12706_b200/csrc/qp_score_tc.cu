// S1 on the 5th-generation tensor cores: the window-score sweeps with TMA, tcgen05.mma and TMEM.
//
// One thread block owns 128 window-query rows (M) of one (batch, KV head) and walks over a run of
// 128-key tiles (N).  The block is specialised by warp and its parts talk through mbarriers only:
//   warp 8     one lane asks the TMA unit for the next key tile ([128 keys x D] bf16 into one of two
//              shared-memory stages, 128-byte swizzle) as soon as the MMAs that read the stage have retired;
//   warp 9     one lane issues the D/16 tcgen05.mma of a tile (bf16 x bf16 -> f32, both operands K-major
//              in shared memory) into one of two [128 x 128] tensor-memory buffers once the tile has landed
//              and the buffer's previous reader is done;
//   warps 0-7  two groups of four warps read the buffers back with tcgen05.ld: group 0 takes the even
//              tiles (buffer 0), group 1 the odd ones, so a thread owns one TMEM lane of a whole tile: a
//              query row in sweep 1 (running max and sum, no shuffles), a key in sweep 2 (the operands are
//              swapped, so the vote of a key is again a thread-local sum).  The next chunk of 32 columns
//              is in flight while a chunk is folded, and the buffer is handed back before the last chunk's
//              arithmetic.
// With two blocks per SM four such groups keep the exponential unit busy while the others wait.
//
// Every wait on an mbarrier is bounded: if it runs out, the block records an error word, waits (bounded)
// for the copies it still has in flight, frees its tensor memory and returns.
#include <cuda.h>

#include <algorithm>
#include <cstring>

#include "qp_mma.cuh"

namespace qp {

namespace {

constexpr int TC_M = 128, TC_N = 128;
constexpr int TC_EPI_WARPS = 8;                       // two groups of four: one TMEM buffer each
constexpr int TC_THREADS = (TC_EPI_WARPS + 2) * 32;   // + the copy warp and the MMA warp
constexpr uint32_t TC_TMEM_COLS = 256;                // two accumulator buffers of 128 columns
constexpr uint32_t TC_SPIN_LIMIT = 1u << 22;

// mbarriers of one block
enum : int { BAR_K_FULL = 0, BAR_K_EMPTY = 2, BAR_T_FULL = 4, BAR_T_EMPTY = 6, BAR_COUNT = 8 };

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
// bounded wait; false = gave up (or another part of the block already has)
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const volatile int* give_up) {
  for (uint32_t i = 0; i < TC_SPIN_LIMIT; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 255u) == 255u && *give_up) return false;
  }
  return false;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
// one box of a 2-D tensor map into shared memory; completion is counted in bytes on `bar`
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
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
// 32 columns of this warp's 32 TMEM lanes; the registers hold nothing until tmem_wait has returned them
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
// waits for every tcgen05.ld of this thread; the registers pass through it, so no use of them can be scheduled earlier
__device__ __forceinline__ void tmem_wait(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;\n"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                 "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]),
                 "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
                 "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}
// 2^x by the hardware approximation (about 2 ulp; results below 2^-126 flush to 0)
__device__ __forceinline__ float ex2a(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
// 2^x for x <= 0 on the FMA and integer pipes: x = n + f with n the nearest integer (1.5 * 2^23 trick) and |f| <= 1/2,
// 2^f by the degree-5 minimax polynomial (relative error 7.5e-8, 2.4e-7 with fp32 rounding), 2^n added into the
// exponent field.  Arguments below -126 are clamped (the result, about 1e-38, stands for the hardware's 0).
__device__ __forceinline__ float ex2p(float x) {
  constexpr float kMagic = 12582912.f;
  x = fmaxf(x, -126.f);
  const float t = x + kMagic;
  const float f = x - (t - kMagic);
  float p = 0x1.5c08e6p-10f;
  p = fmaf(p, f, 0x1.3d0c52p-7f);
  p = fmaf(p, f, 0x1.c6b6e4p-5f);
  p = fmaf(p, f, 0x1.ebf918p-3f);
  p = fmaf(p, f, 0x1.62e428p-1f);
  p = fmaf(p, f, 0x1.000002p+0f);
  return __uint_as_float(__float_as_uint(p) + (__float_as_uint(t) << 23));
}
// Every QP_EXP_POLY-th exponential of the sweeps goes through ex2p instead of the 16-per-clock hardware unit, which is
// the busiest unit of these kernels (0: none).  Measured for the whole score stage with 0 / 6 / 4 / 3: 196.6 / 186.7 /
// 187.7 / 195.2 us for the 70B shapes at batch 4, 115.9 / 111.5 / 110.3 / 112.1 us at 128k.
#ifndef QP_EXP_POLY
#define QP_EXP_POLY 6
#endif
__device__ __forceinline__ float ex2_mixed(float x, int i) {
  return QP_EXP_POLY > 0 && i % QP_EXP_POLY == QP_EXP_POLY - 1 ? ex2p(x) : ex2a(x);
}
__device__ __forceinline__ void cp_async16_zfill(uint32_t saddr, const void* gptr, bool valid) {
  const int n = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(saddr), "l"(gptr), "r"(n));
}

// byte offset of 16-byte chunk c (8 bf16) of row r inside a [128 rows x D] operand: D/64 blocks of
// [128 rows x 128 B], each made of 8-row groups of 1024 B with the chunk index XORed by the row (the
// layout the TMA unit writes for a [128 x 64] box with the 128-byte swizzle at a 1024-byte aligned address)
__device__ __forceinline__ uint32_t sw128_off(int r, int c) {
  return (uint32_t)((c >> 3) * (TC_M * 128) + (r >> 3) * 1024 + (r & 7) * 128 + (((c & 7) ^ (r & 7)) << 4));
}

// per-layer inputs of a sweep: the keys as a tensor map over [batch * KV heads * L, D], the window queries as a pointer
template <int NL>
struct ScoreMaps {
  CUtensorMap k[NL];
  const bf16* q[NL];
};

// sweep 1: folds 32 logits of a row into its running (max, sum)
__device__ __forceinline__ void fold_row(const uint32_t (&r)[32], bool all_visible, int col0, int lim, float scale_log2,
                                         float& m, float& s) {
  if (all_visible) {
    float cm = __uint_as_float(r[0]);
#pragma unroll
    for (int i = 1; i < 32; ++i) cm = fmaxf(cm, __uint_as_float(r[i]));
    const float mn = fmaxf(m, cm * scale_log2);               // scale > 0: max commutes with it
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) acc += ex2_mixed(fmaf(__uint_as_float(r[i]), scale_log2, -mn), i);
    s = fmaf(s, ex2a(m - mn), acc);
    m = mn;
  } else {
    float v[32], cm = -INFINITY;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      v[i] = col0 + i <= lim ? __uint_as_float(r[i]) * scale_log2 : -INFINITY;
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
// sweep 2: adds the probabilities of 32 query rows (columns c0 .. c0+31 of the swapped tile) to a key's vote
__device__ __forceinline__ void fold_vote(const uint32_t (&r)[32], const float2* sRow, int c0, float scale_log2, float& vote) {
#pragma unroll
  for (int i = 0; i < 32; i += 2) {
    const float4 ms = *reinterpret_cast<const float4*>(&sRow[c0 + i]);   // (M, 1/Z) x 2 rows
    vote = fmaf(ex2_mixed(fmaf(__uint_as_float(r[i]), scale_log2, -ms.x), i), ms.y, vote);
    vote = fmaf(ex2_mixed(fmaf(__uint_as_float(r[i + 1]), scale_log2, -ms.z), i + 1), ms.w, vote);
  }
}

template <int PASS, int D, int NL>
__global__ void __launch_bounds__(TC_THREADS, 2)
score_sweep_tc_kernel(const __grid_constant__ ScoreMaps<NL> maps, int bh0, int BH, int Hq, int Hkv, int L, int w,
                      int n_rb, int n_tiles, int tiles_per_block, int n_splits, float scale_log2,
                      float2* __restrict__ stat_partial, const float2* __restrict__ rowstat,
                      float* __restrict__ votes_partial, int* __restrict__ error_word) {
  constexpr int CPR = D / 8;                           // 16-byte chunks per row
  constexpr uint32_t OPER_BYTES = TC_M * D * 2;        // one operand tile: D/64 swizzled blocks of 16 KB
  extern __shared__ unsigned char smem_raw[];
  __shared__ uint64_t bars[BAR_COUNT];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int give_up;
  __shared__ __align__(16) float2 sRow[TC_M];          // sweep 2: (M, 1/Z) of the block's rows; sweep 1: group 1's result

  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  chain_enter();
  // bh counts (layer, batch, KV head): the scratch arrays are laid out over all of them, the inputs are per layer
  const int split = blockIdx.x, rb = blockIdx.y, bh = bh0 + blockIdx.z, layer = bh / BH, bhl = bh % BH;
  const int b = bhl / Hkv, hk = bhl % Hkv, G = Hq / Hkv, P = L - w, R = G * w;
  const int tile_lo = split * tiles_per_block;
  const int n_vis = PASS == 1 ? n_tiles : (P + TC_N - 1) / TC_N;    // sweep 2 only needs prefix columns
  const int tile_hi = min(n_vis, tile_lo + tiles_per_block);
  if (tile_lo >= tile_hi) return;
  const int n_loc = tile_hi - tile_lo;

  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;     // operands need 1024-byte alignment
  const uint32_t sQ = sbase, sK0 = sbase + OPER_BYTES;              // then two K stages
  const uint32_t bar0 = smem_u32(&bars[0]);
  auto bar = [&](int which, int i) { return bar0 + (uint32_t)(which + i) * 8u; };
  const volatile int* gu = &give_up;

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(BAR_K_FULL, i), 1);                // the copy lane's expect_tx; the bytes complete it
      mbar_init(bar(BAR_K_EMPTY, i), 1);               // a tcgen05.commit
      mbar_init(bar(BAR_T_FULL, i), 1);                // a tcgen05.commit
      mbar_init(bar(BAR_T_EMPTY, i), 4 * 32);          // every thread of the reading group
    }
    give_up = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == TC_EPI_WARPS + 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(TC_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }

  // the block's [128 x D] window-query rows (rows beyond R are zero), by every thread
  {
    const bf16* Qh = maps.q[layer] + ((size_t)(b * Hq + hk * G) * w + (size_t)rb * TC_M) * D;
    const int rows_valid = min(TC_M, R - rb * TC_M);
    for (int idx = tid; idx < TC_M * CPR; idx += TC_THREADS) {
      const int r = idx / CPR, c = idx % CPR;
      const bool ok = r < rows_valid;
      cp_async16_zfill(sQ + sw128_off(r, c), Qh + (ok ? (size_t)r * D + c * 8 : 0), ok);
    }
    cp_async_commit();
  }
  if (PASS == 2 && tid < TC_M) {
    if (rowstat) {
      sRow[tid] = rowstat[(size_t)(bh * n_rb + rb) * TC_M + tid];
    } else {
      // sweep 1 left n_splits (max, sum) pairs per row: every block folds those of its 128 rows itself, in the same
      // fixed order, instead of a kernel of its own between the sweeps (four loads in flight at a time)
      const float2* p = stat_partial + (size_t)(bh * n_rb + rb) * n_splits * TC_M + tid;
      float m = -INFINITY, z = 0.f;
      for (int i0 = 0; i0 < n_splits; i0 += 4) {
        float2 v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = p[(size_t)min(i0 + i, n_splits - 1) * TC_M];
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (i0 + i < n_splits && v[i].x != -INFINITY) {
            const float mn = fmaxf(m, v[i].x);
            z = z * exp2f(m - mn) + v[i].y * exp2f(v[i].x - mn);
            m = mn;
          }
      }
      const bool valid = rb * TC_M + tid < R;
      sRow[tid] = make_float2(valid ? m : 0.f, valid ? __fdiv_rn(1.0f, z) : 0.f);
    }
  }
  cp_async_wait<0>();
  asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();                                     // barriers, TMEM base, Q and sRow are visible
  asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
  const uint32_t tmem_base = tmem_base_slot;

  float m_run = -INFINITY, s_run = 0.f;                // sweep 1: this thread's row over the group's tiles

  if (warp == TC_EPI_WARPS) {
    // ---- copy warp: tile j -> stage j & 1 once the MMAs of tile j - 2 have retired
    const CUtensorMap* map = &maps.k[layer];
    int issued = 0;
    bool ok = true;
    for (int j = 0; j < n_loc && ok; ++j) {
      const int st = j & 1;
      if (j >= 2) ok = mbar_wait(bar(BAR_K_EMPTY, st), (uint32_t)(((j >> 1) - 1) & 1), gu);
      if (!ok) break;
      if (lane == 0) {
        mbar_expect_tx(bar(BAR_K_FULL, st), OPER_BYTES);
        const int y = bhl * L + (tile_lo + j) * TC_N;
#pragma unroll
        for (int kb = 0; kb < D / 64; ++kb)
          tma_load_2d(sK0 + st * OPER_BYTES + kb * (TC_N * 128), map, kb * 64, y, bar(BAR_K_FULL, st));
      }
      issued = j + 1;
      __syncwarp();
    }
    if (!ok) {
      give_up = 1;
      // the copies still on their way land in this block's shared memory: wait for them before it is given up
      for (int j = max(0, issued - 2); j < issued; ++j) {
        bool landed = false;
        for (uint32_t i = 0; i < TC_SPIN_LIMIT && !landed; ++i) landed = mbar_try_wait(bar(BAR_K_FULL, j & 1), (uint32_t)((j >> 1) & 1));
      }
    }
  } else if (warp == TC_EPI_WARPS + 1) {
    // ---- MMA warp: tile j from stage j & 1 into TMEM buffer j & 1
    constexpr uint32_t IDESC = instr_desc(TC_M, TC_N);
    bool ok = true;
    for (int j = 0; j < n_loc && ok; ++j) {
      const int st = j & 1;
      ok = mbar_wait(bar(BAR_K_FULL, st), (uint32_t)((j >> 1) & 1), gu);
      if (ok && j >= 2) ok = mbar_wait(bar(BAR_T_EMPTY, st), (uint32_t)(((j >> 1) - 1) & 1), gu);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
      if (lane == 0) {
        const uint32_t sK = sK0 + st * OPER_BYTES, tm = tmem_base + st * TC_N;
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
        umma_commit(bar(BAR_K_EMPTY, st));              // the stage may be refilled ...
        umma_commit(bar(BAR_T_FULL, st));               // ... and the tile read, once these MMAs have retired
      }
      __syncwarp();
    }
    if (!ok) give_up = 1;
  } else {
    // ---- reading groups: group gq takes the tiles j = gq, gq + 2, ... from TMEM buffer gq
    const int gq = warp >> 2, wq = warp & 3, rloc = wq * 32 + lane;
    const int row = rb * TC_M + rloc;
    const int lim = min(P + (row % w), L - 1);          // sweep 1: last key this row may see
    const uint32_t taddr = tmem_base + ((uint32_t)(wq * 32) << 16) + gq * TC_N;
    bool ok = true;
    for (int j = gq; j < n_loc; j += 2) {
      ok = mbar_wait(bar(BAR_T_FULL, gq), (uint32_t)((j >> 1) & 1), gu);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
      const int key0 = (tile_lo + j) * TC_N;
      uint32_t va[32], vb[32];
      float vote = 0.f;
      const bool all_visible = key0 + TC_N - 1 <= P;    // every row sees every key up to P
      auto fold = [&](const uint32_t (&r)[32], int c0) {
        if constexpr (PASS == 1) fold_row(r, all_visible, key0 + c0, lim, scale_log2, m_run, s_run);
        else fold_vote(r, sRow, c0, scale_log2, vote);
      };
      tmem_ld32_issue(taddr, va);
      tmem_wait(va);
      tmem_ld32_issue(taddr + 32, vb);
      fold(va, 0);
      tmem_wait(vb);
      tmem_ld32_issue(taddr + 64, va);
      fold(vb, 32);
      tmem_wait(va);
      tmem_ld32_issue(taddr + 96, vb);
      fold(va, 64);
      tmem_wait(vb);
      asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
      mbar_arrive(bar(BAR_T_EMPTY, gq));                // the buffer is free for tile j + 2
      fold(vb, 96);
      if constexpr (PASS == 2) {
        // only prefix keys (< P) are written and every row sees all of them: no mask needed; rows beyond R
        // carry 1/Z = 0
        if (key0 + rloc < P) votes_partial[(size_t)(bh * n_rb + rb) * P + key0 + rloc] = vote;
      }
    }
    if (!ok) give_up = 1;
    if (PASS == 1 && gq == 1) sRow[rloc] = make_float2(m_run, s_run);
  }

  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();                                      // every part is done with shared and tensor memory
  if (PASS == 1 && warp < 4) {
    // one (max, sum) per row and block: the even tiles' pair, then the odd tiles'
    const int rloc = warp * 32 + lane;
    const float2 o = sRow[rloc];
    const float mn = fmaxf(m_run, o.x);
    float s = 0.f;
    if (m_run != -INFINITY) s = s_run * ex2a(m_run - mn);
    if (o.x != -INFINITY) s = fmaf(o.y, ex2a(o.x - mn), s);
    stat_partial[((size_t)(bh * n_rb + rb) * n_splits + split) * TC_M + rloc] = make_float2(mn, s);
  }
  if (give_up && tid == 0) atomicExch(error_word, 1);
  if (warp == TC_EPI_WARPS + 1) {
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(TC_TMEM_COLS) : "memory");
  }
}

}  // namespace

bool score_tc_supported(int D) { return D == 128 || D == 64; }

namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
// the driver's tensor-map encoder, looked up through the runtime (the library does not link against the driver)
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
// keys of one layer as a [rows x D] bf16 matrix, fetched in boxes of [128 rows x 64 columns] with the 128-byte swizzle;
// boxes that reach past the last row are filled with zeros
cudaError_t key_map(CUtensorMap* map, const void* k, long long rows, int D) {
  EncodeTiledFn enc = encode_tiled();
  if (!enc) return cudaErrorNotSupported;
  const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)D * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)TC_N};
  const cuuint32_t elem[2] = {1, 1};
  const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(k), dims, strides, box, elem,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int PASS, int D, int NL>
cudaError_t launch_tc(dim3 grid, int bh0, int BH, cudaStream_t st, const ScoreMaps<NL>& maps, const ScoreDims& d,
                      const ScoreWorkspace& s, int per, float scale_log2, float2* stat_partial, const float2* rowstat,
                      float* votes_partial, int* error_word, int n_stat) {
  constexpr size_t smem = 3 * (size_t)TC_M * D * 2 + 1024;   // Q + two K stages + alignment slack
  static unsigned char done[64] = {};
  const cudaError_t e = allow_smem(score_sweep_tc_kernel<PASS, D, NL>, smem, done);
  if (e != cudaSuccess) return e;
  return launch_chained(score_sweep_tc_kernel<PASS, D, NL>, grid, dim3(TC_THREADS), smem, st, maps, bh0, BH, d.Hq, d.Hkv, d.L,
                        d.w, s.n_rb, s.n_tiles, per, PASS == 1 ? (int)grid.x : n_stat, scale_log2, stat_partial, rowstat,
                        votes_partial, error_word);
}

template <int NL>
cudaError_t launch_sweep(int pass, int n_layers, const void* const* q, const void* const* k, int bh0, int bh_count,
                         const ScoreDims& d, const ScoreWorkspace& s, float scale_log2, float2* stat_partial,
                         const float2* rowstat, float* votes_partial, int* error_word, cudaStream_t st, int* n_splits, int n_stat) {
  const int BH = d.Bt * d.Hkv;                          // (batch, KV head) pairs of one layer
  if ((long long)BH * d.L > 0x7fffffffLL - TC_N) return cudaErrorInvalidValue;   // row coordinates are 32-bit
  // the two sweeps of a call (and repeated calls on the same buffers) ask for the same maps: keep the last set
  struct Last {
    int n = 0, D = 0;
    long long rows = 0;
    const void* k[QP_MAX_LAYERS];
    CUtensorMap map[QP_MAX_LAYERS];
  };
  static thread_local Last last;
  const long long rows = (long long)BH * d.L;
  bool same = last.n == n_layers && last.D == d.D && last.rows == rows;
  for (int l = 0; same && l < n_layers; ++l) same = last.k[l] == k[l];
  if (!same) {
    last.n = 0;
    for (int l = 0; l < n_layers; ++l) {
      const cudaError_t e = key_map(&last.map[l], k[l], rows, d.D);
      if (e != cudaSuccess) return e;
      last.k[l] = k[l];
    }
    last.n = n_layers; last.D = d.D; last.rows = rows;
  }
  ScoreMaps<NL> maps;
  memset(&maps, 0, sizeof(maps));
  for (int l = 0; l < n_layers; ++l) {
    maps.q[l] = static_cast<const bf16*>(q[l]);
    maps.k[l] = last.map[l];
  }
  const int tiles = pass == 1 ? s.n_tiles : s.n_vote_tiles;
  // Blocks along the keys.  All blocks of a launch take the same time per tile and two fit on an SM, so the launch
  // lasts about ceil(blocks / 2 SMs) rounds of (tiles per block + a fixed cost of about three tiles for the block's
  // set-up and first copy): take the split with the shortest such schedule, at least two tiles per block.
  const int slots = 2 * sm_count();
  long long per = 2;
  double best = 1e300;
  for (int cand = 1; cand <= std::max(1, tiles / 2); ++cand) {
    const long long p = std::max<long long>(2, (tiles + cand - 1) / cand);
    const long long blocks = ((tiles + p - 1) / p) * s.n_rb * bh_count;
    const double cost = (double)((blocks + slots - 1) / slots) * (double)(p + 3);
    if (cost < best) { best = cost; per = p; }
  }
  const int splits = (int)((tiles + per - 1) / per);
  if (n_splits) *n_splits = splits;
  const dim3 grid(splits, s.n_rb, bh_count);
  if (d.D == 128)
    return pass == 1 ? launch_tc<1, 128, NL>(grid, bh0, BH, st, maps, d, s, (int)per, scale_log2, stat_partial, rowstat, votes_partial, error_word, n_stat)
                     : launch_tc<2, 128, NL>(grid, bh0, BH, st, maps, d, s, (int)per, scale_log2, stat_partial, rowstat, votes_partial, error_word, n_stat);
  return pass == 1 ? launch_tc<1, 64, NL>(grid, bh0, BH, st, maps, d, s, (int)per, scale_log2, stat_partial, rowstat, votes_partial, error_word, n_stat)
                   : launch_tc<2, 64, NL>(grid, bh0, BH, st, maps, d, s, (int)per, scale_log2, stat_partial, rowstat, votes_partial, error_word, n_stat);
}
}  // namespace

// s: the scratch layout for batch * n_layers batch entries (the layers are stacked along the batch dimension)
// bh0, bh_count: the (layer, batch, KV head) triples this launch covers; *n_splits: blocks along the keys, i.e. the
// (max, sum) pairs sweep 1 leaves per row in stat_partial [triple, row block, split, 128 rows]; sweep 2 with
// rowstat == nullptr folds n_stat such pairs per row itself
cudaError_t launch_score_sweep_tc(int pass, int n_layers, const void* const* q, const void* const* k, const ScoreDims& d,
                                  const ScoreWorkspace& s, float scale_log2, float2* stat_partial, const float2* rowstat,
                                  float* votes_partial, int* error_word, cudaStream_t st, int bh0, int bh_count,
                                  int* n_splits, int n_stat) {
#define QP_SWEEP(NL) \
  return launch_sweep<NL>(pass, n_layers, q, k, bh0, bh_count, d, s, scale_log2, stat_partial, rowstat, votes_partial, \
                          error_word, st, n_splits, n_stat)
  if (n_layers == 1) QP_SWEEP(1);
  if (n_layers <= 8) QP_SWEEP(8);
  if (n_layers <= 32) QP_SWEEP(32);
  QP_SWEEP(QP_MAX_LAYERS);
#undef QP_SWEEP
}

}  // namespace qp
