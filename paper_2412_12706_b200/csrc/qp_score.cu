// S1: observation-window scores.
//
// For one (batch, KV head) the R = G*w window-query rows form a [R x D] matrix and the
// keys a [L x D] matrix; the logits are their product (a dense contraction, so it runs on
// the tensor cores: bf16 operands, whose products are exact in fp32, fp32 accumulation).
// The row softmax needs every visible key of a row before any column can be normalised,
// hence two sweeps over K:
//   sweep 1  per (key tile, row) running (max, sum of exp)        -> stat partials
//   merge    per row: global max M and 1/Z
//   sweep 2  recompute the tile's logits, p = exp2(t - M)/Z, sum the tile's columns over
//            the rows of the block                                 -> vote partials
//   pool     sum the row blocks, zero-padded moving average of width `pool`.
// Every reduction has a fixed order (shuffles, then a serial loop), so the scores are
// bit-reproducible; there are no floating-point atomics.
#include "qp_common.cuh"

namespace qp {

namespace {

constexpr int SC_TILE = 128;     // keys per thread block
constexpr int SC_RB = 128;       // window-query rows per thread block (8 warps x 16 rows)
constexpr int SC_THREADS = 256;

__host__ __device__ inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

template <int D, int PASS>
__global__ void __launch_bounds__(SC_THREADS)
score_sweep_kernel(const bf16* __restrict__ Qwin, const bf16* __restrict__ K, int Hq, int Hkv, int L, int w,
                   int n_rb, int n_tiles, float scale_log2, float2* __restrict__ stat_partial,
                   const float2* __restrict__ rowstat, float* __restrict__ votes_partial) {
  constexpr int LDS = D + 8;  // padded smem row: consecutive rows fall into different 16-byte bank groups
  __shared__ __align__(16) bf16 sK[SC_TILE * LDS];
  __shared__ float sVote[PASS == 2 ? 8 : 1][SC_TILE];

  const int tile = blockIdx.x, rb = blockIdx.y, bh = blockIdx.z;
  const int b = bh / Hkv, hk = bh % Hkv, G = Hq / Hkv, P = L - w, R = G * w;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int key0 = tile * SC_TILE;

  // stage the key tile (rows beyond L are zero)
  const bf16* Kh = K + (size_t)bh * L * D;
  for (int c = tid; c < SC_TILE * (D / 8); c += SC_THREADS) {
    const int row = c / (D / 8), col = (c % (D / 8)) * 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (key0 + row < L) v = *reinterpret_cast<const uint4*>(Kh + (size_t)(key0 + row) * D + col);
    *reinterpret_cast<uint4*>(sK + row * LDS + col) = v;
  }

  // A fragments: this warp's 16 query rows, all of D, kept in registers
  const int r_lo = rb * SC_RB + warp * 16 + g, r_hi = r_lo + 8;
  const bf16* Qh = Qwin + ((size_t)(b * Hq + hk * G) * w) * D;  // the R rows of this KV head are contiguous
  uint32_t a[D / 16][4];
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
    const int c0 = ks * 16 + 2 * t;
    a[ks][0] = r_lo < R ? *reinterpret_cast<const uint32_t*>(Qh + (size_t)r_lo * D + c0) : 0u;
    a[ks][1] = r_hi < R ? *reinterpret_cast<const uint32_t*>(Qh + (size_t)r_hi * D + c0) : 0u;
    a[ks][2] = r_lo < R ? *reinterpret_cast<const uint32_t*>(Qh + (size_t)r_lo * D + c0 + 8) : 0u;
    a[ks][3] = r_hi < R ? *reinterpret_cast<const uint32_t*>(Qh + (size_t)r_hi * D + c0 + 8) : 0u;
  }
  __syncthreads();

  // logits of 16 rows x 128 keys
  float acc[SC_TILE / 8][4];
  const uint32_t sbase = smem_u32(sK) + (uint32_t)(((lane & 7) * LDS + (lane >> 3) * 8) * 2);
#pragma unroll
  for (int nt = 0; nt < SC_TILE / 8; ++nt) {
    acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < D / 16; ks += 2) {
      uint32_t b0, b1, b2, b3;
      ldmatrix_x4(b0, b1, b2, b3, sbase + (uint32_t)((nt * 8 * LDS + ks * 16) * 2));
      mma_bf16_m16n8k16(acc[nt], a[ks], b0, b1);
      mma_bf16_m16n8k16(acc[nt], a[ks + 1], b2, b3);
    }
  }

  // a row at window position i sees keys 0 .. P+i (causal) and nothing beyond L
  const int lim_lo = min(P + (r_lo % w), L - 1), lim_hi = min(P + (r_hi % w), L - 1);
  const float NEG = -INFINITY;
#pragma unroll
  for (int nt = 0; nt < SC_TILE / 8; ++nt) {
    const int j = key0 + nt * 8 + 2 * t;
    acc[nt][0] = j <= lim_lo ? acc[nt][0] * scale_log2 : NEG;
    acc[nt][1] = j + 1 <= lim_lo ? acc[nt][1] * scale_log2 : NEG;
    acc[nt][2] = j <= lim_hi ? acc[nt][2] * scale_log2 : NEG;
    acc[nt][3] = j + 1 <= lim_hi ? acc[nt][3] * scale_log2 : NEG;
  }

  if constexpr (PASS == 1) {
    float m_lo = NEG, m_hi = NEG;
#pragma unroll
    for (int nt = 0; nt < SC_TILE / 8; ++nt) {
      m_lo = fmaxf(m_lo, fmaxf(acc[nt][0], acc[nt][1]));
      m_hi = fmaxf(m_hi, fmaxf(acc[nt][2], acc[nt][3]));
    }
    m_lo = fmaxf(m_lo, __shfl_xor_sync(0xffffffffu, m_lo, 1));
    m_lo = fmaxf(m_lo, __shfl_xor_sync(0xffffffffu, m_lo, 2));
    m_hi = fmaxf(m_hi, __shfl_xor_sync(0xffffffffu, m_hi, 1));
    m_hi = fmaxf(m_hi, __shfl_xor_sync(0xffffffffu, m_hi, 2));
    float s_lo = 0.f, s_hi = 0.f;
    if (m_lo != NEG) {
#pragma unroll
      for (int nt = 0; nt < SC_TILE / 8; ++nt) s_lo += exp2f(acc[nt][0] - m_lo) + exp2f(acc[nt][1] - m_lo);
    }
    if (m_hi != NEG) {
#pragma unroll
      for (int nt = 0; nt < SC_TILE / 8; ++nt) s_hi += exp2f(acc[nt][2] - m_hi) + exp2f(acc[nt][3] - m_hi);
    }
    s_lo += __shfl_xor_sync(0xffffffffu, s_lo, 1);
    s_lo += __shfl_xor_sync(0xffffffffu, s_lo, 2);
    s_hi += __shfl_xor_sync(0xffffffffu, s_hi, 1);
    s_hi += __shfl_xor_sync(0xffffffffu, s_hi, 2);
    if (t == 0) {
      float2* o = stat_partial + ((size_t)(bh * n_rb + rb) * n_tiles + tile) * SC_RB + warp * 16 + g;
      o[0] = make_float2(m_lo, s_lo);
      o[8] = make_float2(m_hi, s_hi);
    }
  } else {
    const float2 st_lo = rowstat[(size_t)(bh * n_rb + rb) * SC_RB + warp * 16 + g];
    const float2 st_hi = rowstat[(size_t)(bh * n_rb + rb) * SC_RB + warp * 16 + g + 8];
#pragma unroll
    for (int nt = 0; nt < SC_TILE / 8; ++nt) {
      // exp2f(-inf) = 0 covers the masked entries; rows beyond R carry 1/Z = 0
      float c0 = exp2f(acc[nt][0] - st_lo.x) * st_lo.y + exp2f(acc[nt][2] - st_hi.x) * st_hi.y;
      float c1 = exp2f(acc[nt][1] - st_lo.x) * st_lo.y + exp2f(acc[nt][3] - st_hi.x) * st_hi.y;
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) {
        c0 += __shfl_xor_sync(0xffffffffu, c0, o);
        c1 += __shfl_xor_sync(0xffffffffu, c1, o);
      }
      if (g == 0) {
        sVote[warp][nt * 8 + 2 * t] = c0;
        sVote[warp][nt * 8 + 2 * t + 1] = c1;
      }
    }
    __syncthreads();
    if (tid < SC_TILE && key0 + tid < P) {
      float v = 0.f;
#pragma unroll
      for (int wp = 0; wp < 8; ++wp) v += sVote[wp][tid];
      votes_partial[(size_t)(bh * n_rb + rb) * P + key0 + tid] = v;
    }
  }
}

// per row: M = max over tiles, Z = sum_i s_i * 2^(m_i - M); stores (M, 1/Z); rows beyond R get 1/Z = 0.
// One block per (batch, KV head, row block): thread (row, slice) folds tiles slice, slice+8, ... into a running
// (max, sum) pair with coalesced reads across rows; the eight slices are then combined in a fixed order.
constexpr int RM_SLICES = 8;
__global__ void __launch_bounds__(SC_RB * RM_SLICES)
rowstat_merge_kernel(const float2* __restrict__ stat_partial, int n_rb, int n_tiles, int R,
                     float2* __restrict__ rowstat) {
  __shared__ float2 part[RM_SLICES][SC_RB];
  const int blk = blockIdx.x, rb = blk % n_rb, row = threadIdx.x % SC_RB, sl = threadIdx.x / SC_RB;
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
  part[sl][row] = make_float2(m, z);
  __syncthreads();
  if (sl == 0) {
    float M = -INFINITY;
#pragma unroll
    for (int k = 0; k < RM_SLICES; ++k) M = fmaxf(M, part[k][row].x);
    float Z = 0.f;
#pragma unroll
    for (int k = 0; k < RM_SLICES; ++k)
      if (part[k][row].x != -INFINITY) Z += part[k][row].y * exp2f(part[k][row].x - M);
    const bool valid = rb * SC_RB + row < R;
    rowstat[(size_t)blk * SC_RB + row] = make_float2(valid ? M : 0.f, valid ? __fdiv_rn(1.0f, Z) : 0.f);
  }
}

__global__ void __launch_bounds__(256)
pool_kernel(const float* __restrict__ votes_partial, int n_rb, int P, int pool, float* __restrict__ scores) {
  const int bh = blockIdx.y, j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= P) return;
  const int r = (pool - 1) / 2;
  float acc = 0.f;
  for (int dlt = -r; dlt <= r; ++dlt) {
    const int jj = j + dlt;
    if (jj < 0 || jj >= P) continue;
    float v = 0.f;
    for (int rb = 0; rb < n_rb; ++rb) v += votes_partial[(size_t)(bh * n_rb + rb) * P + jj];
    acc += v;
  }
  scores[(size_t)bh * P + j] = __fdiv_rn(acc, (float)pool);
}

}  // namespace

ScoreWorkspace score_workspace(int Bt, int Hq, int Hkv, int L, int w) {
  ScoreWorkspace s{};
  const int BH = Bt * Hkv, R = (Hq / Hkv) * w, P = L - w;
  s.n_rb = (R + SC_RB - 1) / SC_RB;
  s.n_tiles = (L + SC_TILE - 1) / SC_TILE;
  s.n_vote_tiles = (P + SC_TILE - 1) / SC_TILE;
  size_t off = 0;
  // (max, sum) per row and key tile; the tensor-memory sweep keeps one per 64-column half tile
  s.stat_partial = off;  off += align256((size_t)BH * s.n_rb * s.n_tiles * 2 * SC_RB * sizeof(float2));
  s.rowstat = off;       off += align256((size_t)BH * s.n_rb * SC_RB * sizeof(float2));
  s.votes_partial = off; off += align256((size_t)BH * s.n_rb * P * sizeof(float));
  s.pooled = off;        off += align256((size_t)BH * P * sizeof(float));
  s.error = off;         off += 256;
  s.total = off;
  return s;
}

cudaError_t launch_window_scores(const void* Qwin, const void* K, const ScoreDims& d, float* scores, void* ws,
                                 cudaStream_t st) {
  const ScoreWorkspace s = score_workspace(d.Bt, d.Hq, d.Hkv, d.L, d.w);
  const int BH = d.Bt * d.Hkv, P = d.L - d.w, R = (d.Hq / d.Hkv) * d.w;
  char* base = static_cast<char*>(ws);
  float2* stat_partial = reinterpret_cast<float2*>(base + s.stat_partial);
  float2* rowstat = reinterpret_cast<float2*>(base + s.rowstat);
  float* votes_partial = reinterpret_cast<float*>(base + s.votes_partial);
  const float scale_log2 = (float)(1.4426950408889634 / sqrt((double)d.D));
  const bf16* q = static_cast<const bf16*>(Qwin);
  const bf16* k = static_cast<const bf16*>(K);
  dim3 g1(s.n_tiles, s.n_rb, BH), g2(s.n_vote_tiles, s.n_rb, BH);
  if (score_tc_supported(d.D)) {
    // 5th-generation tensor-core path; the word at s.error becomes 1 if a block ever gave up on a wait
    int* err = reinterpret_cast<int*>(base + s.error);
    cudaError_t e = cudaMemsetAsync(err, 0, sizeof(int), st);
    if (e != cudaSuccess) return e;
    e = launch_score_sweep_tc(1, q, k, d, s, scale_log2, stat_partial, nullptr, nullptr, err, st);
    if (e != cudaSuccess) return e;
    rowstat_merge_kernel<<<BH * s.n_rb, SC_RB * RM_SLICES, 0, st>>>(stat_partial, s.n_rb, 2 * s.n_tiles, R, rowstat);
    e = launch_score_sweep_tc(2, q, k, d, s, scale_log2, nullptr, rowstat, votes_partial, err, st);
    if (e != cudaSuccess) return e;
    pool_kernel<<<dim3((P + 255) / 256, BH), 256, 0, st>>>(votes_partial, s.n_rb, P, d.pool, scores);
    return cudaGetLastError();
  }
  if (d.D == 128) {
    score_sweep_kernel<128, 1><<<g1, SC_THREADS, 0, st>>>(q, k, d.Hq, d.Hkv, d.L, d.w, s.n_rb, s.n_tiles,
                                                         scale_log2, stat_partial, nullptr, nullptr);
  } else {
    score_sweep_kernel<64, 1><<<g1, SC_THREADS, 0, st>>>(q, k, d.Hq, d.Hkv, d.L, d.w, s.n_rb, s.n_tiles,
                                                        scale_log2, stat_partial, nullptr, nullptr);
  }
  rowstat_merge_kernel<<<BH * s.n_rb, SC_RB * RM_SLICES, 0, st>>>(stat_partial, s.n_rb, s.n_tiles, R, rowstat);
  if (d.D == 128) {
    score_sweep_kernel<128, 2><<<g2, SC_THREADS, 0, st>>>(q, k, d.Hq, d.Hkv, d.L, d.w, s.n_rb, s.n_tiles,
                                                         scale_log2, nullptr, rowstat, votes_partial);
  } else {
    score_sweep_kernel<64, 2><<<g2, SC_THREADS, 0, st>>>(q, k, d.Hq, d.Hkv, d.L, d.w, s.n_rb, s.n_tiles,
                                                        scale_log2, nullptr, rowstat, votes_partial);
  }
  pool_kernel<<<dim3((P + 255) / 256, BH), 256, 0, st>>>(votes_partial, s.n_rb, P, d.pool, scores);
  return cudaGetLastError();
}

}  // namespace qp
