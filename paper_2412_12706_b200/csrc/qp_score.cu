// S1: observation-window scores — launch sequence and the small kernels around the two tensor-core sweeps.
//
// For one (batch, KV head) the R = G*w window-query rows form a [R x D] matrix and the keys a [L x D]
// matrix; the logits are their product (a dense contraction: qp_score_tc.cu runs it on tcgen05).  The row
// softmax needs every visible key of a row before any column can be normalised, hence two sweeps over K:
//   sweep 1  per (run of key tiles, row) running (max, sum of exp) -> stat partials
//   merge    per row: global max M and 1/Z (folded by every block of sweep 2 for its own rows; a kernel of its own
//            only when sweep 1 left more than 64 pairs per row)
//   sweep 2  recompute the tile's logits, p = exp2(t - M)/Z, sum the tile's columns over the
//            rows of the block                                     -> vote partials
//   pool     sum the row blocks, zero-padded moving average of width `pool`.
// Every reduction has a fixed order, so the scores are bit-reproducible; there are no floating-point atomics.
#include <algorithm>

#include "qp_common.cuh"

namespace qp {

namespace {

constexpr int SC_TILE = 128;     // keys per thread block
constexpr int SC_RB = 128;       // window-query rows per thread block (8 warps x 16 rows)

__host__ __device__ inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// per row: M = max over tiles, Z = sum_i s_i * 2^(m_i - M); stores (M, 1/Z); rows beyond R get 1/Z = 0.
// One block per (batch, KV head, row block, group of RM_ROWS rows): thread (row, slice) folds partials slice,
// slice + RM_SLICES, ... into a running (max, sum) pair with coalesced reads across rows; the slices are then
// combined in a fixed order.
constexpr int RM_SLICES = 32, RM_ROWS = 32, RM_PARTS = SC_RB / RM_ROWS;
__global__ void __launch_bounds__(RM_ROWS * RM_SLICES)
rowstat_merge_kernel(const float2* __restrict__ stat_partial, int blk0, int n_rb, int n_tiles, int R,
                     float2* __restrict__ rowstat) {
  __shared__ float2 part[RM_SLICES][RM_ROWS];
  chain_enter();
  const int blk = blk0 + blockIdx.x / RM_PARTS, rb = blk % n_rb;
  const int rl = threadIdx.x % RM_ROWS, sl = threadIdx.x / RM_ROWS, row = (blockIdx.x % RM_PARTS) * RM_ROWS + rl;
  const float2* p = stat_partial + (size_t)blk * n_tiles * SC_RB + row;
  float m = -INFINITY, z = 0.f;
  for (int i = sl; i < n_tiles; i += RM_SLICES) {
    const float2 s = p[(size_t)i * SC_RB];
    if (s.x != -INFINITY) {
      const float mn = fmaxf(m, s.x);
      z = z * exp2f(m - mn) + s.y * exp2f(s.x - mn);
      m = mn;
    }
  }
  part[sl][rl] = make_float2(m, z);
  __syncthreads();
  if (sl == 0) {
    float M = -INFINITY;
#pragma unroll
    for (int k = 0; k < RM_SLICES; ++k) M = fmaxf(M, part[k][rl].x);
    float Z = 0.f;
#pragma unroll
    for (int k = 0; k < RM_SLICES; ++k)
      if (part[k][rl].x != -INFINITY) Z += part[k][rl].y * exp2f(part[k][rl].x - M);
    const bool valid = rb * SC_RB + row < R;
    rowstat[(size_t)blk * SC_RB + row] = make_float2(valid ? M : 0.f, valid ? __fdiv_rn(1.0f, Z) : 0.f);
  }
}

// scores[j] = (sum over |t| <= r of vote[j + t], zero outside [0, P)) / pool with vote = the sum of the row blocks'
// partial votes.  A block stages the votes of its PK_OUT outputs and their halo in shared memory (zeros outside the
// prefix, so the window sum needs no bounds test) and every thread then forms PK_OUT / PK_THREADS outputs.
constexpr int PK_THREADS = 256, PK_PER = 4, PK_OUT = PK_THREADS * PK_PER, PK_MAX_HALO = 32;
__global__ void __launch_bounds__(PK_THREADS)
pool_kernel(const float* __restrict__ votes_partial, int n_rb, int P, int pool, float* __restrict__ scores) {
  __shared__ float sv[PK_OUT + 2 * PK_MAX_HALO];
  chain_enter();
  const int bh = blockIdx.y, j0 = blockIdx.x * PK_OUT, r = (pool - 1) / 2;
  const float* vp = votes_partial + (size_t)bh * n_rb * P;
  for (int i = threadIdx.x; i < PK_OUT + 2 * r; i += PK_THREADS) {
    const int jj = j0 - r + i;
    float v = 0.f;
    if (jj >= 0 && jj < P)
      for (int rb = 0; rb < n_rb; ++rb) v += vp[(size_t)rb * P + jj];
    sv[i] = v;
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < PK_PER; ++k) {
    const int t = threadIdx.x + k * PK_THREADS, j = j0 + t;
    if (j >= P) break;
    float acc = 0.f;
    for (int dlt = 0; dlt <= 2 * r; ++dlt) acc += sv[t + dlt];
    scores[(size_t)bh * P + j] = __fdiv_rn(acc, (float)pool);
  }
}

}  // namespace

ScoreWorkspace score_workspace(int Bt, int Hq, int Hkv, int L, int w) {
  ScoreWorkspace s{};
  const int BH = Bt * Hkv, R = (Hq / Hkv) * w, P = L - w;
  s.n_rb = (R + SC_RB - 1) / SC_RB;
  s.n_tiles = (L + SC_TILE - 1) / SC_TILE;
  s.n_vote_tiles = (P + SC_TILE - 1) / SC_TILE;
  size_t off = 0;
  // (max, sum) per row and sweep-1 block: at most one block per two key tiles
  s.stat_partial = off;  off += align256((size_t)BH * s.n_rb * ((s.n_tiles + 1) / 2) * SC_RB * sizeof(float2));
  s.rowstat = off;       off += align256((size_t)BH * s.n_rb * SC_RB * sizeof(float2));
  s.votes_partial = off; off += align256((size_t)BH * s.n_rb * P * sizeof(float));
  s.pooled = off;        off += align256((size_t)BH * P * sizeof(float));
  s.error = off;         off += 256;
  s.total = off;
  return s;
}

cudaError_t launch_window_scores_layers(int n_layers, const void* const* Qwin, const void* const* K, const ScoreDims& d,
                                        float* scores, void* ws, cudaStream_t st) {
  const ScoreWorkspace s = score_workspace(d.Bt * n_layers, d.Hq, d.Hkv, d.L, d.w);
  const int BH = d.Bt * d.Hkv * n_layers, P = d.L - d.w, R = (d.Hq / d.Hkv) * d.w;
  char* base = static_cast<char*>(ws);
  float2* stat_partial = reinterpret_cast<float2*>(base + s.stat_partial);
  float2* rowstat = reinterpret_cast<float2*>(base + s.rowstat);
  float* votes_partial = reinterpret_cast<float*>(base + s.votes_partial);
  const float scale_log2 = (float)(1.4426950408889634 / sqrt((double)d.D));
  if (!score_tc_supported(d.D)) return cudaErrorInvalidValue;   // other head dimensions are rejected before this point
  // 5th-generation tensor-core path; the word at s.error becomes 1 if a block ever gave up on a wait
  int* err = reinterpret_cast<int*>(base + s.error);
  cudaError_t e = cudaMemsetAsync(err, 0, sizeof(int), st);
  if (e != cudaSuccess) return e;
  // The two sweeps of a (batch, KV head) read the same keys, so the keys cross the HBM interface twice.  Taking the
  // heads in groups whose keys fit in the L2 cache (sweep 1 -> merge -> sweep 2 per group) lets the second sweep find
  // them there, but the smaller launches fill the SMs worse and lose more at their ends than the cache hits save:
  // measured for the whole score stage with groups of 0 (off) / 64 / 100 MB: 250 / 396 / 361 us at 32k x batch 8,
  // 128 / 210 / 188 us at 128k, 222 / 259 / 244 us for the 70B shapes.  Off by default.
#ifndef QP_SCORE_GROUP_MB
#define QP_SCORE_GROUP_MB 0
#endif
  const size_t head_bytes = (size_t)d.L * d.D * 2;
  int per_group = QP_SCORE_GROUP_MB > 0 ? (int)std::max<size_t>(1, ((size_t)QP_SCORE_GROUP_MB << 20) / head_bytes) : BH;
  if ((long long)per_group * s.n_tiles * s.n_rb < 2 * 296) per_group = BH;     // small problems: one group
  for (int bh0 = 0; bh0 < BH; bh0 += per_group) {
    const int cnt = std::min(per_group, BH - bh0);
    int n_splits = 0;
    e = launch_score_sweep_tc(1, n_layers, Qwin, K, d, s, scale_log2, stat_partial, nullptr, nullptr, err, st, bh0, cnt,
                              &n_splits);
    if (e != cudaSuccess) return e;
    // the row statistics are folded inside sweep 2 unless sweep 1 left very many pairs per row
    const bool fold_in_sweep = n_splits <= 64;
    if (!fold_in_sweep) {
      e = launch_chained(rowstat_merge_kernel, dim3(cnt * s.n_rb * RM_PARTS), dim3(RM_ROWS * RM_SLICES), 0, st,
                         (const float2*)stat_partial, bh0 * s.n_rb, s.n_rb, n_splits, R, rowstat);
      if (e != cudaSuccess) return e;
    }
    e = launch_score_sweep_tc(2, n_layers, Qwin, K, d, s, scale_log2, stat_partial, fold_in_sweep ? nullptr : rowstat,
                              votes_partial, err, st, bh0, cnt, nullptr, n_splits);
    if (e != cudaSuccess) return e;
  }
  return launch_chained(pool_kernel, dim3((P + PK_OUT - 1) / PK_OUT, BH), dim3(PK_THREADS), 0, st,
                        (const float*)votes_partial, s.n_rb, P, d.pool, scores);
}

cudaError_t launch_window_scores(const void* Qwin, const void* K, const ScoreDims& d, float* scores, void* ws,
                                 cudaStream_t st) {
  const void* qs[1] = {Qwin};
  const void* ks[1] = {K};
  return launch_window_scores_layers(1, qs, ks, d, scores, ws, st);
}

}  // namespace qp
