// S5 for a cache with a tail: log-sum-exp merge of the split partials of one (layer, batch, query head)
// plus the attention over the tail's unquantized tokens (Eq. 2: tokens appended during decoding that
// do not fill a quantization group yet).
//
// The tail is tiny (fewer than g <= 128 tokens of D <= 128 channels per KV head) and bf16, so it never
// enters the packed-cache kernels: the warp that merges a query head's records computes the tail's logits
// itself, in fp32, and folds them into the same running (max, sum, acc) before it normalises.
// One warp per (layer, batch, query head); lane c owns channels 4c .. 4c+3.
#include <algorithm>

#include "qp_mma.cuh"

namespace qp {

namespace {

constexpr int MT_WARPS = 4;

__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__global__ void __launch_bounds__(MT_WARPS * 32)
decode_merge_tail_kernel(const __grid_constant__ DecTable tab, const __grid_constant__ TailTable tails, const DecDims dm,
                         const float* __restrict__ partials) {
  const int D = dm.D, G = dm.Hq / dm.Hkv, BH = dm.Bt * dm.Hkv, n_bq = dm.Bt * dm.Hq;
  const int lane = threadIdx.x & 31, n_items = n_bq * tab.n_layers;
  const size_t stride = (size_t)G * (D + 2);
  const bool chan = 4 * lane < D;                                // this lane owns four channels
  const float scale_log2 = 1.4426950408889634f * rsqrtf((float)D);
  asm volatile("griddepcontrol.launch_dependents;\n" ::);
  asm volatile("griddepcontrol.wait;\n" ::: "memory");          // returns at once when launched in plain stream order
  for (int item = blockIdx.x * MT_WARPS + (threadIdx.x >> 5); item < n_items; item += gridDim.x * MT_WARPS) {
    const int layer = item / n_bq, bq = item % n_bq;
    const DecLayer& ly = tab.l[layer];
    const TailLayer& tl = tails.l[layer];
    const int b = bq / dm.Hq, h = bq % dm.Hq, bh = b * dm.Hkv + h / G, hl = h % G;
    // the records of this head: `count` of them, `stride` floats apart, from `base`
    const float* base;
    int count;
    if (tab.n_workers > 0) {                                     // flat-range decomposition: slots head + worker
      const unsigned T = (unsigned)tab.total_tiles, W = (unsigned)tab.n_workers;
      const int tph = (ly.n + 31) >> 5;
      const unsigned first = (unsigned)ly.tile_base + (unsigned)bh * tph;
      const int w_lo = (int)(((first + 1u) * W - 1u) / T), w_hi = (int)(((first + tph) * W - 1u) / T);
      const size_t head = (size_t)layer * BH + bh;
      base = partials + ((head + w_lo) * G + hl) * (size_t)(D + 2);
      count = w_hi - w_lo + 1;
    } else {                                                     // chunked decomposition: slots of (head, split)
      const int n_splits = (ly.n + tab.chunk - 1) / tab.chunk;
      base = partials + (((size_t)ly.part_base + (size_t)bh * n_splits) * G + hl) * (size_t)(D + 2);
      count = n_splits;
    }

    // ---- tail logits (log2 domain, like the records' maxima): token 32j + s is kept by lane s in lt[j]
    const int nt = tl.n_tail;
    const uint16_t* kt = static_cast<const uint16_t*>(tl.kt) + (size_t)bh * dm.group * D + 4 * lane;
    const uint16_t* vt = static_cast<const uint16_t*>(tl.vt) + (size_t)bh * dm.group * D + 4 * lane;
    float q0 = 0.f, q1 = 0.f, q2 = 0.f, q3 = 0.f;
    if (chan && nt > 0) {
      const uint2 qw = *reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(ly.q) + (size_t)bq * D + 4 * lane);
      q0 = bf16lo(qw.x) * scale_log2; q1 = bf16hi(qw.x) * scale_log2;
      q2 = bf16lo(qw.y) * scale_log2; q3 = bf16hi(qw.y) * scale_log2;
    }
    float lt[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < 4; ++j)
      for (int s = 0; s < 32 && 32 * j + s < nt; ++s) {
        float part = 0.f;
        if (chan) {
          const uint2 kw = *reinterpret_cast<const uint2*>(kt + (size_t)(32 * j + s) * D);
          part = fmaf(q0, bf16lo(kw.x), fmaf(q1, bf16hi(kw.x), fmaf(q2, bf16lo(kw.y), q3 * bf16hi(kw.y))));
        }
        const float dot = warp_sum_f(part);
        if (lane == s) lt[j] = dot;
      }

    // ---- common reference maximum
    float M = fmaxf(fmaxf(lt[0], lt[1]), fmaxf(lt[2], lt[3]));
    for (int r = lane; r < count; r += 32) M = fmaxf(M, base[r * stride]);
    M = warp_max_f(M);

    // ---- records, then tail tokens, in a fixed order
    float Ls = 0.f, A0 = 0.f, A1 = 0.f, A2 = 0.f, A3 = 0.f;
    if (chan)
      for (int r = 0; r < count; ++r) {
        const float* rec = base + r * stride;
        const float2 ml = *reinterpret_cast<const float2*>(rec);
        const float2 a01 = *reinterpret_cast<const float2*>(rec + 2 + 4 * lane);
        const float2 a23 = *reinterpret_cast<const float2*>(rec + 4 + 4 * lane);
        const float f = exp2f(ml.x - M);
        Ls = fmaf(ml.y, f, Ls);
        A0 = fmaf(a01.x, f, A0); A1 = fmaf(a01.y, f, A1);
        A2 = fmaf(a23.x, f, A2); A3 = fmaf(a23.y, f, A3);
      }
#pragma unroll
    for (int j = 0; j < 4; ++j)
      for (int s = 0; s < 32 && 32 * j + s < nt; ++s) {
        const float p = exp2f(__shfl_sync(0xffffffffu, lt[j], s) - M);
        if (chan) {
          const uint2 vw = *reinterpret_cast<const uint2*>(vt + (size_t)(32 * j + s) * D);
          Ls += p;
          A0 = fmaf(p, bf16lo(vw.x), A0); A1 = fmaf(p, bf16hi(vw.x), A1);
          A2 = fmaf(p, bf16lo(vw.y), A2); A3 = fmaf(p, bf16hi(vw.y), A3);
        }
      }
    if (!chan) continue;
    const float inv = __fdiv_rn(1.0f, Ls);
    __nv_bfloat162 o01 = __floats2bfloat162_rn(A0 * inv, A1 * inv), o23 = __floats2bfloat162_rn(A2 * inv, A3 * inv);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t*>(&o01);
    packed.y = *reinterpret_cast<uint32_t*>(&o23);
    *reinterpret_cast<uint2*>(static_cast<bf16*>(ly.out) + (size_t)bq * D + 4 * lane) = packed;
  }
}

}  // namespace

cudaError_t launch_merge_tail(const DecTable& tab, const DecDims& d, const float* partials, const TailTable& tails,
                              cudaStream_t st, bool programmatic) {
  const int items = d.Bt * d.Hq * tab.n_layers;
  const int row_blocks = (items + MT_WARPS - 1) / MT_WARPS;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(std::min(row_blocks, 8 * sm_count()));
  cfg.blockDim = dim3(MT_WARPS * 32);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = programmatic ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, decode_merge_tail_kernel, tab, tails, d, partials);
}

}  // namespace qp
