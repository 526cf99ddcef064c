// S2: per-head top-k by radix select + ordered compaction.
//
// One thread block per (batch, KV head).  The k-th largest score is found digit by digit
// (four 8-bit histograms over an order-preserving integer image of the floats); a final
// ordered sweep emits, in ascending position, every element above the threshold plus the
// first `need` elements equal to it, which is exactly "largest score first, lower position
// first among equals" without sorting.  Integer work only: results are exact.
#include "qp_common.cuh"

namespace qp {

namespace {

constexpr int TK_THREADS = 1024;

// monotone map float -> uint32 (larger float = larger integer); -0 is treated as +0
__device__ __forceinline__ uint32_t order_key(float f) {
  const uint32_t u = __float_as_uint(f + 0.0f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__global__ void __launch_bounds__(TK_THREADS)
topk_kernel(const float* __restrict__ scores, int L, int w, int n_keep, int32_t* __restrict__ kept) {
  const int P = L - w, k = n_keep - w;
  const int bh = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* s = scores + (size_t)bh * P;
  int32_t* out = kept + (size_t)bh * n_keep;

  for (int i = tid; i < w; i += TK_THREADS) out[k + i] = P + i;   // window tokens are always kept
  if (k >= P) {                                                    // keep everything
    for (int j = tid; j < P; j += TK_THREADS) out[j] = j;
    return;
  }

  __shared__ unsigned hist[256];
  __shared__ unsigned sh_prefix, sh_need;
  __shared__ unsigned warp_gt[32], warp_eq[32];
  __shared__ unsigned run_gt, run_eq;

  unsigned prefix = 0, mask = 0, need = (unsigned)k;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int j = tid; j < P; j += TK_THREADS) {
      const uint32_t u = order_key(s[j]);
      if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      unsigned cum = 0;
      int b = 255;
      for (; b > 0; --b) {
        if (cum + hist[b] >= need) break;
        cum += hist[b];
      }
      sh_need = need - cum;                 // still to take among elements with this digit
      sh_prefix = prefix | ((unsigned)b << shift);
    }
    __syncthreads();
    prefix = sh_prefix;
    need = sh_need;
    mask |= 0xffu << shift;
    __syncthreads();
  }
  const uint32_t T = prefix;   // image of the k-th largest score; `need` elements equal to it are kept

  if (tid == 0) { run_gt = 0; run_eq = 0; }
  __syncthreads();
  for (int base = 0; base < P; base += TK_THREADS) {
    const int j = base + tid;
    uint32_t u = 0;
    bool gt = false, eq = false;
    if (j < P) { u = order_key(s[j]); gt = u > T; eq = u == T; }
    const unsigned bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
    const unsigned lt_mask = (1u << lane) - 1u;
    if (lane == 0) { warp_gt[warp] = __popc(bg); warp_eq[warp] = __popc(be); }
    __syncthreads();
    unsigned pg = run_gt + __popc(bg & lt_mask), pe = run_eq + __popc(be & lt_mask);
    for (int wp = 0; wp < warp; ++wp) { pg += warp_gt[wp]; pe += warp_eq[wp]; }
    if (gt || (eq && pe < need)) out[pg + min(pe, need)] = j;
    __syncthreads();
    if (tid == TK_THREADS - 1) {
      run_gt = pg + (gt ? 1u : 0u);
      run_eq = pe + (eq ? 1u : 0u);
    }
    __syncthreads();
  }
}

}  // namespace

cudaError_t launch_select_topk(const float* scores, int BH, int L, int w, int n_keep, int32_t* kept, cudaStream_t st) {
  topk_kernel<<<BH, TK_THREADS, 0, st>>>(scores, L, w, n_keep, kept);
  return cudaGetLastError();
}

}  // namespace qp
