// S2: per-head top-k by radix select + ordered compaction.
//
// One thread block per (batch, KV head).  The k-th largest score is found digit by digit
// (four 8-bit histograms over an order-preserving integer image of the floats); a final
// ordered sweep emits, in ascending position, every element above the threshold plus the
// first `need` elements equal to it, which is exactly "largest score first, lower position
// first among equals" without sorting.  Integer work only: results are exact.
#include <cooperative_groups.h>

#include "qp_checked.cuh"
#include "qp_common.cuh"

namespace qp {

namespace {

constexpr int TK_THREADS = 1024;
constexpr int TK_UNROLL = 8;
constexpr int TKR_BINS = 4096;     // histogram bins of the register kernel's 12-bit digits

// Outputs of the layers of one launch: block (layer, bh) reads scores[(layer * BH + bh) * P ..] and writes
// kept[layer][bh * n_keep[layer] ..].
template <int NL>
struct TopkOut {
  int32_t* kept[NL];
  int n_keep[NL];
};

// monotone map float -> uint32 (larger float = larger integer); -0 is treated as +0
__device__ __forceinline__ uint32_t order_key(float f) {
  const uint32_t u = __float_as_uint(f + 0.0f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <int NL>
__global__ void __launch_bounds__(TK_THREADS)
topk_kernel(const float* __restrict__ scores, int L, int w, int BH, const __grid_constant__ TopkOut<NL> o) {
  chain_enter();
  const int layer = blockIdx.x / BH, n_keep = o.n_keep[layer];
  const int P = L - w, k = n_keep - w;
  const int bh = blockIdx.x % BH, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* s = scores + (size_t)blockIdx.x * P;
  int32_t* out = o.kept[layer] + (size_t)bh * n_keep;

  for (int i = tid; i < w; i += TK_THREADS) out[k + i] = P + i;   // window tokens are always kept
  if (k >= P) {                                                    // keep everything
    for (int j = tid; j < P; j += TK_THREADS) out[j] = j;
    return;
  }

  __shared__ unsigned hist[256];
  __shared__ unsigned sh_prefix, sh_need;
  __shared__ unsigned warp_gt[32], warp_eq[32];

  unsigned prefix = 0, mask = 0, need = (unsigned)k;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    // scores cluster in a few exponents, so most elements of a warp share a digit: lanes with equal digits
    // elect one leader that adds their count (one shared-memory atomic per distinct digit and warp)
    // (only worth it for the two leading digits; the trailing ones are spread out).  TK_UNROLL loads are
    // issued before any of them is used, so a sweep costs one memory latency per TK_UNROLL * 1024 elements.
    for (int base = 0; base < P; base += TK_UNROLL * TK_THREADS) {
      float f[TK_UNROLL];
#pragma unroll
      for (int q = 0; q < TK_UNROLL; ++q) {
        const int j = base + q * TK_THREADS + tid;
        f[q] = j < P ? s[j] : 0.f;
      }
#pragma unroll
      for (int q = 0; q < TK_UNROLL; ++q) {
        const int j = base + q * TK_THREADS + tid;
        if (base + q * TK_THREADS >= P) break;
        const uint32_t u = order_key(f[q]);
        const bool cand = j < P && (u & mask) == prefix;
        const unsigned digit = (u >> shift) & 255u;
        if (shift >= 16) {
          const unsigned peers = __match_any_sync(0xffffffffu, cand ? digit : 256u + lane);
          if (cand && lane == __ffs(peers) - 1) atomicAdd(&hist[digit], (unsigned)__popc(peers));
        } else if (cand) {
          atomicAdd(&hist[digit], 1u);
        }
      }
    }
    __syncthreads();
    if (warp == 0) {
      // lane l owns bins 8l .. 8l+7; find the bin where the count from the top reaches `need`
      unsigned c[8], tot = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { c[i] = hist[8 * lane + i]; tot += c[i]; }
      unsigned suf = tot;                                   // bins of this lane and all higher lanes
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned v = __shfl_down_sync(0xffffffffu, suf, o);
        if (lane + o < 32) suf += v;
      }
      const unsigned above = suf - tot;
      if (above < need && suf >= need) {                    // exactly one lane
        unsigned cum = above;
        int bsel = 7;
        for (; bsel > 0; --bsel) {
          if (cum + c[bsel] >= need) break;
          cum += c[bsel];
        }
        sh_need = need - cum;                               // still to take among elements with this digit
        sh_prefix = prefix | ((unsigned)(8 * lane + bsel) << shift);
      }
    }
    __syncthreads();
    prefix = sh_prefix;
    need = sh_need;
    mask |= 0xffu << shift;
  }
  const uint32_t T = prefix;   // image of the k-th largest score; `need` elements equal to it are kept

  unsigned run_g = 0, run_e = 0;                            // kept / equal elements before this chunk (all threads agree)
  for (int base0 = 0; base0 < P; base0 += TK_UNROLL * TK_THREADS) {
    float f[TK_UNROLL];
#pragma unroll
    for (int q = 0; q < TK_UNROLL; ++q) {
      const int j = base0 + q * TK_THREADS + tid;
      f[q] = j < P ? s[j] : 0.f;
    }
#pragma unroll
    for (int q = 0; q < TK_UNROLL; ++q) {
      const int base = base0 + q * TK_THREADS;
      if (base >= P) break;
      const int j = base + tid;
      const uint32_t u = order_key(f[q]);
      const bool gt = j < P && u > T, eq = j < P && u == T;
      const unsigned bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
      const unsigned lt_mask = (1u << lane) - 1u;
      if (lane == 0) { warp_gt[warp] = __popc(bg); warp_eq[warp] = __popc(be); }
      __syncthreads();
      // exclusive prefix of the 32 warp counts, computed by every warp with shuffles
      unsigned wg = warp_gt[lane], we = warp_eq[lane], sg = wg, se = we;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned vg = __shfl_up_sync(0xffffffffu, sg, o), ve = __shfl_up_sync(0xffffffffu, se, o);
        if (lane >= o) { sg += vg; se += ve; }
      }
      const unsigned tot_g = __shfl_sync(0xffffffffu, sg, 31), tot_e = __shfl_sync(0xffffffffu, se, 31);
      const unsigned pre_g = __shfl_sync(0xffffffffu, sg - wg, warp), pre_e = __shfl_sync(0xffffffffu, se - we, warp);
      const unsigned pg = run_g + pre_g + __popc(bg & lt_mask), pe = run_e + pre_e + __popc(be & lt_mask);
      if ((gt || (eq && pe < need)) && QP_IN_RANGE(pg + min(pe, need), k, QP_SITE_TOPK_OUT)) out[pg + min(pe, need)] = j;
      run_g += tot_g;
      run_e += tot_e;
      __syncthreads();                                      // warp_gt / warp_eq are rewritten by the next chunk
    }
  }
}

// The same selection for P <= ITEMS * 1024 with the keys held in registers: the scores are read from memory once
// (all loads in flight together) instead of five times, the digit passes (three here, over wider digits) and the
// compaction run from registers, and the ordered compaction needs one block-wide prefix over (chunk, warp) counts instead of one
// per chunk.  Element j = q * 1024 + tid is item q of thread tid, so ascending position = (q, warp, lane) order.
template <int ITEMS, int NL>
__global__ void __launch_bounds__(TK_THREADS)
topk_reg_kernel(const float* __restrict__ scores, int L, int w, int BH, const __grid_constant__ TopkOut<NL> o) {
  chain_enter();
  const int layer = blockIdx.x / BH, n_keep = o.n_keep[layer];
  const int P = L - w, k = n_keep - w;
  const int bh = blockIdx.x % BH, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* s = scores + (size_t)blockIdx.x * P;
  int32_t* out = o.kept[layer] + (size_t)bh * n_keep;

  for (int i = tid; i < w; i += TK_THREADS) out[k + i] = P + i;   // window tokens are always kept
  if (k >= P) {                                                    // keep everything
    for (int j = tid; j < P; j += TK_THREADS) out[j] = j;
    return;
  }

  __shared__ unsigned hist[TKR_BINS];
  __shared__ unsigned warp_tot[32];
  __shared__ unsigned sh_prefix, sh_need;
  __shared__ unsigned cnt_g[ITEMS][32], cnt_e[ITEMS][32];        // per (chunk, warp): counts, then exclusive prefixes
  __shared__ unsigned row_g[ITEMS], row_e[ITEMS];                // per chunk: totals, then exclusive prefixes

  uint32_t key[ITEMS];                                           // order-preserving images; valid where j < P
#pragma unroll
  for (int q = 0; q < ITEMS; ++q) {
    const int j = q * TK_THREADS + tid;
    key[q] = order_key(j < P ? s[j] : 0.f);
  }

  // Three digit passes of 12, 12 and 8 bits over a 4096-bin histogram.  The leading 12 bits (sign, exponent, three
  // mantissa bits) of real scores take dozens of values, so the lanes of a warp mostly hit different bins and plain
  // shared-memory atomics do; only a warp whose 32 candidates all carry one digit (constant scores) adds once.
  unsigned prefix = 0, mask = 0, need = (unsigned)k;
#pragma unroll 1
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 20 : pass == 1 ? 8 : 0;
    const unsigned dmask = pass == 2 ? 255u : (unsigned)(TKR_BINS - 1);
#pragma unroll
    for (int i = 0; i < TKR_BINS / TK_THREADS; ++i) hist[tid + i * TK_THREADS] = 0;
    __syncthreads();
#pragma unroll
    for (int q = 0; q < ITEMS; ++q) {
      if (q * TK_THREADS >= P) break;
      const bool cand = q * TK_THREADS + tid < P && (key[q] & mask) == prefix;
      const unsigned digit = (key[q] >> shift) & dmask;
      if (pass == 0) {
        const unsigned d0 = __shfl_sync(0xffffffffu, digit, 0);
        if (__all_sync(0xffffffffu, cand && digit == d0)) {
          if (lane == 0) atomicAdd(&hist[d0], 32u);
        } else if (cand) {
          atomicAdd(&hist[digit], 1u);
        }
      } else if (cand) {
        atomicAdd(&hist[digit], 1u);
      }
    }
    __syncthreads();
    // thread t owns bins 4t .. 4t+3; find the bin where the count from the top reaches `need`
    unsigned c[TKR_BINS / TK_THREADS], tot = 0;
#pragma unroll
    for (int i = 0; i < TKR_BINS / TK_THREADS; ++i) { c[i] = hist[(TKR_BINS / TK_THREADS) * tid + i]; tot += c[i]; }
    unsigned suf = tot;                                          // this thread and the higher lanes of its warp
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned v = __shfl_down_sync(0xffffffffu, suf, o);
      if (lane + o < 32) suf += v;
    }
    if (lane == 0) warp_tot[warp] = suf;
    __syncthreads();
    unsigned higher = 0;                                         // the warps above this one
    for (int wv = warp + 1; wv < 32; ++wv) higher += warp_tot[wv];
    const unsigned incl = suf + higher, above = incl - tot;
    if (above < need && incl >= need) {                          // exactly one thread
      unsigned cum = above;
      int bsel = TKR_BINS / TK_THREADS - 1;
      for (; bsel > 0; --bsel) {
        if (cum + c[bsel] >= need) break;
        cum += c[bsel];
      }
      sh_need = need - cum;
      sh_prefix = prefix | ((unsigned)((TKR_BINS / TK_THREADS) * tid + bsel) << shift);
    }
    __syncthreads();
    prefix = sh_prefix;
    need = sh_need;
    mask |= dmask << shift;
  }
  const uint32_t T = prefix;   // image of the k-th largest score; `need` elements equal to it are kept

  // ---- ordered compaction: counts per (chunk, warp), one block-wide exclusive prefix, then the writes
#pragma unroll
  for (int q = 0; q < ITEMS; ++q) {
    const bool in = q * TK_THREADS + tid < P;
    const unsigned bg = __ballot_sync(0xffffffffu, in && key[q] > T), be = __ballot_sync(0xffffffffu, in && key[q] == T);
    if (lane == 0) { cnt_g[q][warp] = __popc(bg); cnt_e[q][warp] = __popc(be); }
  }
  __syncthreads();
  for (int q = warp; q < ITEMS; q += 32) {                       // warp q scans chunk q's 32 warp counts
    const unsigned wg = cnt_g[q][lane], we = cnt_e[q][lane];
    unsigned sg = wg, se = we;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned vg = __shfl_up_sync(0xffffffffu, sg, o), ve = __shfl_up_sync(0xffffffffu, se, o);
      if (lane >= o) { sg += vg; se += ve; }
    }
    cnt_g[q][lane] = sg - wg;
    cnt_e[q][lane] = se - we;
    if (lane == 31) { row_g[q] = sg; row_e[q] = se; }
  }
  __syncthreads();
  if (warp == 0) {                                               // exclusive prefix of the chunk totals (ITEMS <= 32)
    const unsigned wg = lane < ITEMS ? row_g[lane] : 0u, we = lane < ITEMS ? row_e[lane] : 0u;
    unsigned sg = wg, se = we;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned vg = __shfl_up_sync(0xffffffffu, sg, o), ve = __shfl_up_sync(0xffffffffu, se, o);
      if (lane >= o) { sg += vg; se += ve; }
    }
    if (lane < ITEMS) { row_g[lane] = sg - wg; row_e[lane] = se - we; }
  }
  __syncthreads();
  const unsigned lt_mask = (1u << lane) - 1u;
#pragma unroll
  for (int q = 0; q < ITEMS; ++q) {
    if (q * TK_THREADS >= P) break;
    const int j = q * TK_THREADS + tid;
    const bool gt = j < P && key[q] > T, eq = j < P && key[q] == T;
    const unsigned bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
    const unsigned pg = row_g[q] + cnt_g[q][warp] + __popc(bg & lt_mask);
    const unsigned pe = row_e[q] + cnt_e[q][warp] + __popc(be & lt_mask);
    if ((gt || (eq && pe < need)) && QP_IN_RANGE(pg + min(pe, need), k, QP_SITE_TOPK_OUT)) out[pg + min(pe, need)] = j;
  }
}

// The same selection for long prefixes (up to CTAS * TKC_ITEMS * 1024 positions; CTAS = 8, or 4 or 2 for mid head counts) by a
// thread-block cluster per
// (layer, batch, KV head): CTA c of the cluster holds the contiguous segment [c * S, (c + 1) * S) of the prefix in
// registers, builds its own digit histogram in shared memory, and every CTA then sums the cluster's histograms
// through distributed shared memory, so all of them take the same decision without any global traffic.
constexpr int TKC_CTAS = 8;
constexpr int TKC_ITEMS = 16;

template <int NL, int CTAS>
__global__ void __cluster_dims__(CTAS, 1, 1) __launch_bounds__(TK_THREADS)
topk_cluster_kernel(const float* __restrict__ scores, int L, int w, int BH, const __grid_constant__ TopkOut<NL> o) {
  chain_enter();
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const int head = blockIdx.x / CTAS, crank = (int)cluster.block_rank();
  const int layer = head / BH, n_keep = o.n_keep[layer];
  const int P = L - w, k = n_keep - w;
  const int bh = head % BH, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* s = scores + (size_t)head * P;
  int32_t* out = o.kept[layer] + (size_t)bh * n_keep;

  if (crank == 0)
    for (int i = tid; i < w; i += TK_THREADS) out[k + i] = P + i;  // window tokens are always kept
  if (k >= P) {                                                    // keep everything (the whole cluster leaves)
    for (int j = crank * TK_THREADS + tid; j < P; j += CTAS * TK_THREADS) out[j] = j;
    return;
  }

  __shared__ unsigned h12[TKR_BINS];                             // this CTA's histogram of a 12-bit digit
  __shared__ unsigned xch[4][256];                               // exchanged counts, one buffer per step in rotation
  __shared__ unsigned ghist[256];                                // the cluster's counts of the step
  __shared__ unsigned sh_sel, sh_need;
  __shared__ unsigned cnt_g[TKC_ITEMS][32], cnt_e[TKC_ITEMS][32];
  __shared__ unsigned row_g[TKC_ITEMS], row_e[TKC_ITEMS];
  __shared__ unsigned tot_ge[2];                                 // this CTA's kept / equal totals

  const int S = (P + CTAS - 1) / CTAS;                   // positions per CTA
  const int seg0 = crank * S, seg_n = max(0, min(S, P - seg0));  // this CTA's segment
  uint32_t key[TKC_ITEMS];
#pragma unroll
  for (int q = 0; q < TKC_ITEMS; ++q) {
    const int i = q * TK_THREADS + tid;
    key[q] = order_key(i < seg_n ? s[seg0 + i] : 0.f);
  }

  // Three scans of the keys (digits of 12, 12 and 8 bits, plain shared-memory atomics as in the register kernel).  A
  // 12-bit histogram stays in this CTA: what the cluster exchanges through distributed shared memory is its fold to
  // 256 coarse bins (the digit's upper 8 bits) and then the 16 fine bins inside the chosen coarse bin, 272 counts per
  // CTA instead of 4096, with one hardware cluster barrier per exchange (five in all).
  unsigned prefix = 0, mask = 0, need = (unsigned)k;
  int step = 0;                                                  // exchange steps so far: buffer xch[step & 3]
  // sums the CTAs' `n_bins` counts of buffer `buf`, finds the bin where the count from the top reaches `need`;
  // every CTA takes the same decision
  auto exchange_select = [&](int n_bins) -> unsigned {
    unsigned* mine = xch[step & 3];
    cluster.sync();                                              // every CTA's counts of this step are in place
    if (tid < n_bins) {
      unsigned sum = 0;
#pragma unroll
      for (int c = 0; c < CTAS; ++c) sum += cluster.map_shared_rank(mine, c)[tid];
      ghist[tid] = sum;
    } else if (tid < 256) {
      ghist[tid] = 0;
    }
    __syncthreads();
    if (warp == 0) {
      unsigned c[8], tot = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { c[i] = ghist[8 * lane + i]; tot += c[i]; }
      unsigned suf = tot;
#pragma unroll
      for (int o2 = 1; o2 < 32; o2 <<= 1) {
        const unsigned v = __shfl_down_sync(0xffffffffu, suf, o2);
        if (lane + o2 < 32) suf += v;
      }
      const unsigned above = suf - tot;
      if (above < need && suf >= need) {                         // exactly one lane
        unsigned cum = above;
        int bsel = 7;
        for (; bsel > 0; --bsel) {
          if (cum + c[bsel] >= need) break;
          cum += c[bsel];
        }
        sh_need = need - cum;
        sh_sel = (unsigned)(8 * lane + bsel);
      }
    }
    __syncthreads();
    need = sh_need;
    ++step;
    return sh_sel;
  };
#pragma unroll 1
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 20 : pass == 1 ? 8 : 0;
    const unsigned dmask = pass == 2 ? 255u : (unsigned)(TKR_BINS - 1);
#pragma unroll
    for (int i = 0; i < TKR_BINS / TK_THREADS; ++i) h12[tid + i * TK_THREADS] = 0;
    __syncthreads();
#pragma unroll
    for (int q = 0; q < TKC_ITEMS; ++q) {
      if (q * TK_THREADS >= seg_n) break;
      const bool cand = q * TK_THREADS + tid < seg_n && (key[q] & mask) == prefix;
      const unsigned digit = (key[q] >> shift) & dmask;
      if (pass == 0) {
        const unsigned d0 = __shfl_sync(0xffffffffu, digit, 0);
        if (__all_sync(0xffffffffu, cand && digit == d0)) {
          if (lane == 0) atomicAdd(&h12[d0], 32u);
        } else if (cand) {
          atomicAdd(&h12[digit], 1u);
        }
      } else if (cand) {
        atomicAdd(&h12[digit], 1u);
      }
    }
    __syncthreads();
    if (pass == 2) {                                             // 8-bit digit: the histogram itself is exchanged
      if (tid < 256) xch[step & 3][tid] = h12[tid];
      const unsigned sel = exchange_select(256);
      prefix |= sel;
      mask |= 255u;
    } else {
      if (tid < 256) {                                           // fold to the digit's upper 8 bits
        unsigned sum = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) sum += h12[16 * tid + i];
        xch[step & 3][tid] = sum;
      }
      const unsigned coarse = exchange_select(256);
      if (tid < 16) xch[step & 3][tid] = h12[16 * coarse + tid];  // the 16 fine bins inside it
      const unsigned fine = exchange_select(16);
      prefix |= (16u * coarse + fine) << shift;
      mask |= dmask << shift;
    }
  }
  const uint32_t T = prefix;

  // ---- ordered compaction: counts per (chunk, warp) inside the CTA, CTA totals across the cluster
#pragma unroll
  for (int q = 0; q < TKC_ITEMS; ++q) {
    const bool in = q * TK_THREADS + tid < seg_n;
    const unsigned bg = __ballot_sync(0xffffffffu, in && key[q] > T), be = __ballot_sync(0xffffffffu, in && key[q] == T);
    if (lane == 0) { cnt_g[q][warp] = __popc(bg); cnt_e[q][warp] = __popc(be); }
  }
  __syncthreads();
  for (int q = warp; q < TKC_ITEMS; q += 32) {
    const unsigned wg = cnt_g[q][lane], we = cnt_e[q][lane];
    unsigned sg = wg, se = we;
#pragma unroll
    for (int o2 = 1; o2 < 32; o2 <<= 1) {
      const unsigned vg = __shfl_up_sync(0xffffffffu, sg, o2), ve = __shfl_up_sync(0xffffffffu, se, o2);
      if (lane >= o2) { sg += vg; se += ve; }
    }
    cnt_g[q][lane] = sg - wg;
    cnt_e[q][lane] = se - we;
    if (lane == 31) { row_g[q] = sg; row_e[q] = se; }
  }
  __syncthreads();
  if (warp == 0) {
    const unsigned wg = lane < TKC_ITEMS ? row_g[lane] : 0u, we = lane < TKC_ITEMS ? row_e[lane] : 0u;
    unsigned sg = wg, se = we;
#pragma unroll
    for (int o2 = 1; o2 < 32; o2 <<= 1) {
      const unsigned vg = __shfl_up_sync(0xffffffffu, sg, o2), ve = __shfl_up_sync(0xffffffffu, se, o2);
      if (lane >= o2) { sg += vg; se += ve; }
    }
    if (lane < TKC_ITEMS) { row_g[lane] = sg - wg; row_e[lane] = se - we; }
    if (lane == 31) { tot_ge[0] = sg; tot_ge[1] = se; }
  }
  cluster.sync();                                                // every CTA's totals are in place
  unsigned base_g = 0, base_e = 0;                               // kept / equal elements in the segments before this one
  for (int c = 0; c < crank; ++c) {
    const unsigned* t = cluster.map_shared_rank(tot_ge, c);
    base_g += t[0];
    base_e += t[1];
  }
  const unsigned lt_mask = (1u << lane) - 1u;
#pragma unroll
  for (int q = 0; q < TKC_ITEMS; ++q) {
    if (q * TK_THREADS >= seg_n) break;
    const int i = q * TK_THREADS + tid;
    const bool gt = i < seg_n && key[q] > T, eq = i < seg_n && key[q] == T;
    const unsigned bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
    const unsigned pg = base_g + row_g[q] + cnt_g[q][warp] + __popc(bg & lt_mask);
    const unsigned pe = base_e + row_e[q] + cnt_e[q][warp] + __popc(be & lt_mask);
    if ((gt || (eq && pe < need)) && QP_IN_RANGE(pg + min(pe, need), k, QP_SITE_TOPK_OUT)) out[pg + min(pe, need)] = seg0 + i;
  }
  cluster.sync();                                                // no CTA leaves while another may still read its totals
}

}  // namespace

namespace {
template <int NL>
cudaError_t launch_topk(const float* scores, int blocks, int BH, int L, int w, const TopkOut<NL>& o, cudaStream_t st) {
  const int P = L - w;
  // a cluster per head also pays for prefixes of 8k to 32k positions when the heads alone would leave most SMs
  // idle (measured at 32k positions: 19.5 us against 24.8 us for 8 heads)
  const bool few_heads = blocks * TKC_CTAS <= sm_count();
  // between the two: a cluster of four or two per head while that still fits in one round of the SMs (measured at
  // 32k positions: 32 heads 24.8 -> 16.7 us with four)
  if (!few_heads && P > 8 * TK_THREADS) {
    if (P <= 4 * TKC_ITEMS * TK_THREADS && blocks * 4 <= sm_count())
      return launch_chained(topk_cluster_kernel<NL, 4>, dim3(blocks * 4), dim3(TK_THREADS), 0, st, scores, L, w, BH, o);
    if (P <= 2 * TKC_ITEMS * TK_THREADS && blocks * 2 <= sm_count())
      return launch_chained(topk_cluster_kernel<NL, 2>, dim3(blocks * 2), dim3(TK_THREADS), 0, st, scores, L, w, BH, o);
  }
  if (P <= 8 * TK_THREADS) return launch_chained(topk_reg_kernel<8, NL>, dim3(blocks), dim3(TK_THREADS), 0, st, scores, L, w, BH, o);
  else if (P <= 32 * TK_THREADS && !few_heads)
    return launch_chained(topk_reg_kernel<32, NL>, dim3(blocks), dim3(TK_THREADS), 0, st, scores, L, w, BH, o);
  else if (P <= TKC_CTAS * TKC_ITEMS * TK_THREADS)
    return launch_chained(topk_cluster_kernel<NL, TKC_CTAS>, dim3(blocks * TKC_CTAS), dim3(TK_THREADS), 0, st, scores, L, w, BH, o);
  return launch_chained(topk_kernel<NL>, dim3(blocks), dim3(TK_THREADS), 0, st, scores, L, w, BH, o);
}
}  // namespace

cudaError_t launch_select_topk(const float* scores, int BH, int L, int w, int n_keep, int32_t* kept, cudaStream_t st) {
  TopkOut<1> o;
  o.kept[0] = kept;
  o.n_keep[0] = n_keep;
  return launch_topk<1>(scores, BH, BH, L, w, o, st);
}

cudaError_t launch_select_topk_layers(int n_layers, const float* scores, int BH, int L, int w, const int* n_keep,
                                      int32_t* const* kept, cudaStream_t st) {
  if (n_layers == 1) return launch_select_topk(scores, BH, L, w, n_keep[0], kept[0], st);
  TopkOut<QP_MAX_LAYERS> o;
  for (int l = 0; l < n_layers; ++l) {
    o.kept[l] = kept[l];
    o.n_keep[l] = n_keep[l];
  }
  return launch_topk<QP_MAX_LAYERS>(scores, n_layers * BH, BH, L, w, o, st);
}

// ---- head-level budgets: how many tokens each KV head of a layer keeps when the heads share the layer's budget
namespace {
// kept_flat [Bt, k_total + 1]: ascending indices h*P + j of the k_total marked positions of a batch entry (the
// last entry is the selection kernel's window slot and is ignored).  One block per batch entry: a thread per
// head counts its marked positions by two binary searches, thread 0 then applies the rounding rule in order.
__global__ void __launch_bounds__(64)
head_budget_kernel(const int32_t* __restrict__ kept_flat, int k_total, int Hkv, int P, int L, int w, int n_mean,
                   int unit, int32_t* __restrict__ n_heads) {
  extern __shared__ int s_n[];
  const int b = blockIdx.x;
  const int32_t* kf = kept_flat + (size_t)b * (k_total + 1);
  auto lower = [&](long long key) {                 // first position whose index is >= key
    int lo = 0, hi = k_total;
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if ((long long)kf[mid] < key) lo = mid + 1; else hi = mid;
    }
    return lo;
  };
  const int n_min = (w / unit) * unit + unit, n_max = max(n_min, (L / unit) * unit);
  for (int h = threadIdx.x; h < Hkv; h += blockDim.x) {
    const int raw = lower((long long)(h + 1) * P) - lower((long long)h * P) + w;
    s_n[h] = min(n_max, max(n_min, (raw / unit) * unit));
  }
  __syncthreads();
  if (threadIdx.x != 0) return;
  long long total = 0;
  for (int h = 0; h < Hkv; ++h) total += s_n[h];
  while (total > (long long)Hkv * n_mean) {        // the largest head (lowest first among equals) gives back a unit
    int best = 0;
    for (int h = 1; h < Hkv; ++h)
      if (s_n[h] > s_n[best]) best = h;
    if (s_n[best] <= n_min) break;
    s_n[best] -= unit;
    total -= unit;
  }
  for (int h = 0; h < Hkv; ++h) n_heads[(size_t)b * Hkv + h] = s_n[h];
}
}  // namespace

cudaError_t launch_head_budgets(const float* scores, int Bt, int Hkv, int L, int w, int n_mean, int unit,
                                int32_t* n_heads, int32_t* kept_flat, cudaStream_t st) {
  const int P = L - w;
  const long long k_total = std::min<long long>((long long)Hkv * (n_mean - w), (long long)Hkv * P);
  // the marked positions: top-k over the row of all heads' scores (ties to the lower flat index = lower head,
  // then lower position); the selection kernel wants a window, so the row gets one extra position
  const cudaError_t e = launch_select_topk(scores, Bt, Hkv * P + 1, 1, (int)k_total + 1, kept_flat, st);
  if (e != cudaSuccess) return e;
  head_budget_kernel<<<Bt, 64, Hkv * sizeof(int), st>>>(kept_flat, (int)k_total, Hkv, P, L, w, n_mean, unit, n_heads);
  return cudaGetLastError();
}

#ifdef QP_CHECKED
cudaError_t topk_check_read(unsigned int (&out)[4]) { return checked::read_and_clear(out); }
#endif

}  // namespace qp
