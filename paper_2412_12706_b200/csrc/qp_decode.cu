// S4 + S5: split-K decode attention over the packed pruned cache.
//
// Grid = (token splits, batch x KV heads, layers).  A thread block streams its token range
// of one KV head once; the G query heads of that KV head share the stream.  Dequantisation
// (code * scale + zero) happens in registers, the softmax is the usual running (max, sum)
// form in the log2 domain, and each block leaves one partial (m, l, acc[D]) per query head.
// A second kernel merges the partials of a (batch, query head) in a fixed order.
// No block ever waits for another one.
#include <algorithm>

#include "qp_checked.cuh"
#include "qp_common.cuh"

namespace qp {

namespace {

constexpr int DG_THREADS = 128;
constexpr int DG_WARPS = 4;
constexpr int MAXG = 8;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Reference-shaped kernel: any supported (B, g, D, G).  One lane per token on the key side,
// one lane per channel (stride 32) on the value side.
// ex: key grouping axis and outlier side lists of the other quantization strategies (single layer); a listed
// element was stored with code 0, so the dense arithmetic sees its group's zero point z there and the listed
// value x enters as a correction x - z, applied in list order (fixed order of additions).
template <int BITS>
__global__ void __launch_bounds__(DG_THREADS)
decode_generic_kernel(const __grid_constant__ DecTable tab, const DecDims dm, float* __restrict__ partials,
                      const DecEx ex) {
  constexpr int PER = BITS < 16 ? 32 / BITS : 1;
  constexpr uint32_t QMAX = BITS < 16 ? (1u << BITS) - 1u : 0u;
  const int layer = blockIdx.z, bh = blockIdx.y, split = blockIdx.x;
  const DecLayer& ly = tab.l[layer];
  const int n = ly.n, ns = ly.ns, t_begin = split * tab.chunk;
  if (t_begin >= n) return;
  const int t_end = min(n, t_begin + tab.chunk);
  const int D = dm.D, G = dm.Hq / dm.Hkv, g = dm.group, wpg = g * BITS / 32, ngv = D / g;
  const int b = bh / dm.Hkv, hk = bh % dm.Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_splits = (n + tab.chunk - 1) / tab.chunk;

  __shared__ float sq[MAXG][128];
  __shared__ float s_m[DG_WARPS][MAXG], s_l[DG_WARPS][MAXG];
  __shared__ float s_acc[DG_WARPS][MAXG][128];

  const float scale_log2 = 1.4426950408889634f * rsqrtf((float)D);
  const uint16_t* q = static_cast<const uint16_t*>(ly.q) + (size_t)(b * dm.Hq + hk * G) * D;
  for (int i = tid; i < G * D; i += DG_THREADS) sq[i / D][i % D] = bf16_bits_to_f32(q[i]) * scale_log2;
  __syncthreads();

  float m[MAXG], l[MAXG], acc[MAXG][4];
#pragma unroll
  for (int h = 0; h < MAXG; ++h) {
    m[h] = -INFINITY;
    l[h] = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[h][i] = 0.f;
  }

  const uint32_t* kc = static_cast<const uint32_t*>(ly.kc);
  const uint32_t* vc = static_cast<const uint32_t*>(ly.vc);
  const uint16_t* k16 = static_cast<const uint16_t*>(ly.kc);
  const uint16_t* v16 = static_cast<const uint16_t*>(ly.vc);

  for (int tile = t_begin + warp * 32; tile < t_end; tile += DG_WARPS * 32) {
    const int tok = tile + lane;
    const bool valid = tok < t_end;
    const int tk = valid ? tok : t_end - 1;
    float lg[MAXG];
#pragma unroll
    for (int h = 0; h < MAXG; ++h) lg[h] = 0.f;
    if constexpr (BITS < 16) {
      if (ex.k_axis == 1) {                                     // this lane's token: D/g groups of g channels
        const size_t row = ((size_t)bh * ns + tk) * ngv;
        for (int v = 0; v < ngv; ++v) {
          const float sc = __half2float(ly.ks[row + v]), zr = __half2float(ly.kz[row + v]);
          const uint32_t* wp = kc + (row + v) * wpg;
          for (int wd = 0; wd < wpg; ++wd) {
            const uint32_t word = wp[wd];
#pragma unroll
            for (int i = 0; i < PER; ++i) {
              const float kf = fmaf((float)((word >> (i * BITS)) & QMAX), sc, zr);
              const int d = v * g + wd * PER + i;
#pragma unroll
              for (int h = 0; h < MAXG; ++h)
                if (h < G) lg[h] = fmaf(sq[h][d], kf, lg[h]);
            }
          }
        }
      } else {
        const int u = tk / g, e = tk % g;
        const size_t base = ((size_t)bh * (ns / g) + u) * D;
        const int wsel = e / PER, sh = (e % PER) * BITS;
        for (int d = 0; d < D; ++d) {
          const uint32_t c = (kc[(base + d) * wpg + wsel] >> sh) & QMAX;
          const float kf = fmaf((float)c, __half2float(ly.ks[base + d]), __half2float(ly.kz[base + d]));
#pragma unroll
          for (int h = 0; h < MAXG; ++h)
            if (h < G) lg[h] = fmaf(sq[h][d], kf, lg[h]);
        }
      }
      if (ex.has_side) {                                        // key outliers of this tile, in list order
        const int32_t* tp = ex.k.tile_ptr + (size_t)bh * (ex.k.n_tiles + 1) + (tile >> 5);
        const int32_t* sidx = ex.k.idx + (size_t)bh * ex.k.cap;
        const uint16_t* sval = ex.k.val + (size_t)bh * ex.k.cap;
        const bool ptr_ok = QP_IN_RANGE(tp[0], ex.k.cap + 1, QP_SITE_SIDE_PTR) && QP_IN_RANGE(tp[1], ex.k.cap + 1, QP_SITE_SIDE_PTR);
        for (int i = ptr_ok ? tp[0] : 0; i < (ptr_ok ? tp[1] : 0); ++i) {
          const int fi = sidx[i], t2 = fi / D, d = fi % D;      // warp-uniform
          if (!QP_IN_RANGE(fi, (long long)n * D, QP_SITE_SIDE_IDX)) continue;
          if (t2 == tok) {
            const size_t gi = ex.k_axis == 1 ? ((size_t)bh * ns + t2) * ngv + d / g
                                             : ((size_t)bh * (ns / g) + t2 / g) * D + d;
            const float delta = bf16_bits_to_f32(sval[i]) - __half2float(ly.kz[gi]);
#pragma unroll
            for (int h = 0; h < MAXG; ++h)
              if (h < G) lg[h] = fmaf(sq[h][d], delta, lg[h]);
          }
        }
      }
    } else {
      const uint16_t* row = k16 + ((size_t)bh * ns + tk) * D;
      for (int d = 0; d < D; ++d) {
        const float kf = bf16_bits_to_f32(row[d]);
#pragma unroll
        for (int h = 0; h < MAXG; ++h)
          if (h < G) lg[h] = fmaf(sq[h][d], kf, lg[h]);
      }
    }
    float p[MAXG];
#pragma unroll
    for (int h = 0; h < MAXG; ++h) {
      p[h] = 0.f;
      if (h < G) {
        const float v = valid ? lg[h] : -INFINITY;
        const float mnew = fmaxf(m[h], warp_max(v));      // finite: lane 0 of a tile is always valid
        p[h] = valid ? exp2f(v - mnew) : 0.f;
        const float corr = exp2f(m[h] - mnew);             // 0 on the first tile (m = -inf)
        l[h] = l[h] * corr + warp_sum(p[h]);
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[h][i] *= corr;
        m[h] = mnew;
      }
    }
    const int nt = min(32, t_end - tile);
    for (int tt = 0; tt < nt; ++tt) {
      const int tok2 = tile + tt;
      float vf[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int d = lane + 32 * i;
        vf[i] = 0.f;
        if (d < D) {
          if constexpr (BITS < 16) {
            const int e2 = d % g;
            const size_t gi = ((size_t)bh * ns + tok2) * ngv + d / g;
            const uint32_t c = (vc[gi * wpg + e2 / PER] >> ((e2 % PER) * BITS)) & QMAX;
            vf[i] = fmaf((float)c, __half2float(ly.vs[gi]), __half2float(ly.vz[gi]));
          } else {
            vf[i] = bf16_bits_to_f32(v16[((size_t)bh * ns + tok2) * D + d]);
          }
        }
      }
#pragma unroll
      for (int h = 0; h < MAXG; ++h)
        if (h < G) {
          const float ph = __shfl_sync(0xffffffffu, p[h], tt);
#pragma unroll
          for (int i = 0; i < 4; ++i) acc[h][i] = fmaf(ph, vf[i], acc[h][i]);
        }
    }
    if constexpr (BITS < 16) {
      if (ex.has_side) {                                        // value outliers of this tile, in list order
        const int32_t* tp = ex.v.tile_ptr + (size_t)bh * (ex.v.n_tiles + 1) + (tile >> 5);
        const int32_t* sidx = ex.v.idx + (size_t)bh * ex.v.cap;
        const uint16_t* sval = ex.v.val + (size_t)bh * ex.v.cap;
        const bool ptr_ok = QP_IN_RANGE(tp[0], ex.v.cap + 1, QP_SITE_SIDE_PTR) && QP_IN_RANGE(tp[1], ex.v.cap + 1, QP_SITE_SIDE_PTR);
        for (int i = ptr_ok ? tp[0] : 0; i < (ptr_ok ? tp[1] : 0); ++i) {
          const int fi = sidx[i], t2 = fi / D, d = fi % D;      // warp-uniform
          if (!QP_IN_RANGE(fi, (long long)n * D, QP_SITE_SIDE_IDX) || t2 < tile || t2 >= tile + 32) continue;
          const size_t gi = ((size_t)bh * ns + t2) * ngv + d / g;
          const float delta = bf16_bits_to_f32(sval[i]) - __half2float(ly.vz[gi]);
#pragma unroll
          for (int h = 0; h < MAXG; ++h)
            if (h < G) {
              const float ph = __shfl_sync(0xffffffffu, p[h], t2 - tile);
              if ((d & 31) == lane) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                  if (j == (d >> 5)) acc[h][j] = fmaf(ph, delta, acc[h][j]);
              }
            }
        }
      }
    }
  }

  // combine the four warps, fixed order
#pragma unroll
  for (int h = 0; h < MAXG; ++h)
    if (h < G) {
      if (lane == 0) { s_m[warp][h] = m[h]; s_l[warp][h] = l[h]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (lane + 32 * i < D) s_acc[warp][h][lane + 32 * i] = acc[h][i];
    }
  __syncthreads();
  const size_t slot = (size_t)ly.part_base + (size_t)bh * n_splits + split;
  for (int idx = tid; idx < G * D; idx += DG_THREADS) {
    const int h = idx / D, d = idx % D;
    float M = -INFINITY;
#pragma unroll
    for (int wp = 0; wp < DG_WARPS; ++wp) M = fmaxf(M, s_m[wp][h]);
    float Ls = 0.f, A = 0.f;
#pragma unroll
    for (int wp = 0; wp < DG_WARPS; ++wp)
      if (s_m[wp][h] != -INFINITY) {
        const float f = exp2f(s_m[wp][h] - M);
        Ls = fmaf(s_l[wp][h], f, Ls);
        A = fmaf(s_acc[wp][h][d], f, A);
      }
    float* o = partials + (slot * G + h) * (size_t)(D + 2);
    if (d == 0) { o[0] = M; o[1] = Ls; }
    o[2 + d] = A;
  }
}

// S5: log-sum-exp merge of the split partials of one (layer, batch, query head)
__global__ void __launch_bounds__(128)
decode_merge_kernel(const __grid_constant__ DecTable tab, const DecDims dm, const float* __restrict__ partials) {
  const int layer = blockIdx.y, bq = blockIdx.x, d = threadIdx.x;
  const DecLayer& ly = tab.l[layer];
  const int D = dm.D, G = dm.Hq / dm.Hkv;
  if (d >= D) return;
  const int b = bq / dm.Hq, h = bq % dm.Hq, bh = b * dm.Hkv + h / G, hl = h % G;
  const int n_splits = (ly.n + tab.chunk - 1) / tab.chunk;
  const float* base = partials + (((size_t)ly.part_base + (size_t)bh * n_splits) * G + hl) * (size_t)(D + 2);
  const size_t stride = (size_t)G * (D + 2);
  float M = -INFINITY;
  for (int s = 0; s < n_splits; ++s) M = fmaxf(M, base[s * stride]);
  float Ls = 0.f, A = 0.f;
  for (int s = 0; s < n_splits; ++s) {
    const float f = exp2f(base[s * stride] - M);
    Ls = fmaf(base[s * stride + 1], f, Ls);
    A = fmaf(base[s * stride + 2 + d], f, A);
  }
  static_cast<bf16*>(ly.out)[(size_t)bq * D + d] = __float2bfloat16_rn(__fdiv_rn(A, Ls));
}

}  // namespace

int sm_count() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

namespace {

size_t record_bytes(const DecDims& d) { return (size_t)(d.Hq / d.Hkv) * (size_t)(d.D + 2) * sizeof(float); }
size_t round256(size_t x) { return (x + 255) & ~(size_t)255; }

// chunked kernel: about eight blocks per SM, in whole 128-token units
int chunk_tokens(long long total_tokens) {
  long long c = (total_tokens + 148 * 8 - 1) / (148 * 8);
  c = (c + 127) / 128 * 128;
  if (c < 128) c = 128;
  if (c > 4096) c = 4096;
  return (int)c;
}

}  // namespace

size_t decode_plan(DecTable& tab, const DecDims& d, bool paired) {
  const int BH = d.Bt * d.Hkv;
  if (decode_mma_supported(d)) {
    long long T = 0;
    for (int l = 0; l < tab.n_layers; ++l) {
      tab.l[l].tile_base = (int)T;
      tab.l[l].part_base = 0;
      T += (long long)BH * ((tab.l[l].n + 31) / 32);
    }
    long long W = (long long)sm_count() * decode_mma_workers_per_sm(d);
    tab.wide = 0;
    tab.paired = paired ? 1 : 0;
    int wide_min = 0;
    const long long Ww = (long long)sm_count() * decode_mma_wide_workers_per_sm(d, &wide_min);
    const long long merge_blocks = ((long long)d.Bt * d.Hq * tab.n_layers + 3) / 4;
    // long ranges and a merge grid too large to sit beside the attention blocks anyway: more, narrower workers
    if (Ww > 0 && Ww <= kMaxDecodeWorkers && T >= Ww * wide_min && merge_blocks > 2 * sm_count()) {
      W = Ww;
      tab.wide = 1;
    }
    if (W > kMaxDecodeWorkers) W = kMaxDecodeWorkers;
    const int tmin = decode_mma_tiles_per_worker_min(d, T, paired);
    if (!tab.wide && W > (T + tmin - 1) / tmin) W = (T + tmin - 1) / tmin;
    if (W < 1) W = 1;
    while (W > 1 && T * W >= (1ll << 31)) W /= 2;               // the merge kernel's range arithmetic is 32-bit
    tab.total_tiles = (int)T;
    tab.n_workers = (int)W;
    tab.chunk = 0;
    return decode_workspace_layout(tab, d).total_bytes();
  }
  return decode_plan_chunked(tab, d);
}

DecWorkspace decode_workspace_layout(const DecTable& tab, const DecDims& d) {
  const size_t heads = (size_t)tab.n_layers * d.Bt * d.Hkv;
  return DecWorkspace{round256((heads + (size_t)tab.n_workers) * record_bytes(d))};
}

size_t decode_workspace_bound(const DecDims& d, int n_keep) {
  const size_t BH = (size_t)d.Bt * d.Hkv;
  const size_t chunked = BH * (size_t)((n_keep + 127) / 128) * record_bytes(d);   // 128 tokens = smallest split
  const size_t flat = 2 * round256((BH + kMaxDecodeWorkers) * record_bytes(d));
  return chunked > flat ? chunked : flat;
}

cudaError_t launch_decode(const DecTable& tab, const DecDims& d, void* workspace, int parity, cudaStream_t st,
                          bool overlap_prev, const TailTable* tails) {
  if (decode_mma_supported(d)) {
    const DecWorkspace ws = decode_workspace_layout(tab, d);
    unsigned char* base = static_cast<unsigned char*>(workspace);
    return launch_decode_mma(tab, d, reinterpret_cast<float*>(base + (parity ? ws.record_bytes : 0)), st, overlap_prev,
                             tails);
  }
  float* partials = static_cast<float*>(workspace);
  int max_splits = 1;
  for (int l = 0; l < tab.n_layers; ++l) max_splits = max(max_splits, (tab.l[l].n + tab.chunk - 1) / tab.chunk);
  const dim3 grid(max_splits, d.Bt * d.Hkv, tab.n_layers);
  const DecEx none{};
  switch (d.bits) {
    case 2: decode_generic_kernel<2><<<grid, DG_THREADS, 0, st>>>(tab, d, partials, none); break;
    case 4: decode_generic_kernel<4><<<grid, DG_THREADS, 0, st>>>(tab, d, partials, none); break;
    case 8: decode_generic_kernel<8><<<grid, DG_THREADS, 0, st>>>(tab, d, partials, none); break;
    case 16: decode_generic_kernel<16><<<grid, DG_THREADS, 0, st>>>(tab, d, partials, none); break;
    default: return cudaErrorInvalidValue;
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (tails) return launch_merge_tail(tab, d, partials, *tails, st, false);
  decode_merge_kernel<<<dim3(d.Bt * d.Hq, tab.n_layers), 128, 0, st>>>(tab, d, partials);
  return cudaGetLastError();
}

// One layer under a quantization strategy: the chunked kernel with the strategy's key axis and side lists, then
// the chunked merge.  tab: planned with decode_plan_chunked.
cudaError_t launch_decode_ex(const DecTable& tab, const DecDims& d, const DecEx& ex, void* workspace, cudaStream_t st) {
  float* partials = static_cast<float*>(workspace);
  int max_splits = 1;
  for (int l = 0; l < tab.n_layers; ++l) max_splits = max(max_splits, (tab.l[l].n + tab.chunk - 1) / tab.chunk);
  const dim3 grid(max_splits, d.Bt * d.Hkv, tab.n_layers);
  switch (d.bits) {
    case 2: decode_generic_kernel<2><<<grid, DG_THREADS, 0, st>>>(tab, d, partials, ex); break;
    case 4: decode_generic_kernel<4><<<grid, DG_THREADS, 0, st>>>(tab, d, partials, ex); break;
    case 8: decode_generic_kernel<8><<<grid, DG_THREADS, 0, st>>>(tab, d, partials, ex); break;
    default: return cudaErrorInvalidValue;
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  decode_merge_kernel<<<dim3(d.Bt * d.Hq, tab.n_layers), 128, 0, st>>>(tab, d, partials);
  return cudaGetLastError();
}

size_t decode_plan_flat(DecTable& tab, const DecDims& d, int workers_per_sm, int tiles_per_worker_min) {
  const int BH = d.Bt * d.Hkv;
  long long T = 0;
  for (int l = 0; l < tab.n_layers; ++l) {
    tab.l[l].tile_base = (int)T;
    tab.l[l].part_base = 0;
    T += (long long)BH * ((tab.l[l].n + 31) / 32);
  }
  long long W = std::min<long long>((long long)sm_count() * workers_per_sm, kMaxDecodeWorkers);
  W = std::min(W, (T + tiles_per_worker_min - 1) / tiles_per_worker_min);
  if (W < 1) W = 1;
  while (W > 1 && T * W >= (1ll << 31)) W /= 2;
  tab.total_tiles = (int)T;
  tab.n_workers = (int)W;
  tab.chunk = tab.wide = tab.paired = 0;
  return decode_workspace_layout(tab, d).record_bytes;
}

size_t decode_plan_chunked(DecTable& tab, const DecDims& d) {
  const int BH = d.Bt * d.Hkv;
  long long total_tokens = 0;
  for (int l = 0; l < tab.n_layers; ++l) total_tokens += (long long)BH * tab.l[l].n;
  tab.chunk = chunk_tokens(total_tokens);
  tab.total_tiles = tab.n_workers = tab.wide = tab.paired = 0;
  size_t slots = 0;
  for (int l = 0; l < tab.n_layers; ++l) {
    tab.l[l].part_base = (int)slots;
    tab.l[l].tile_base = 0;
    slots += (size_t)BH * ((tab.l[l].n + tab.chunk - 1) / tab.chunk);
  }
  return slots * record_bytes(d);
}

#ifdef QP_CHECKED
cudaError_t decode_check_read(unsigned int (&out)[4]) { return checked::read_and_clear(out); }
#endif

}  // namespace qp
