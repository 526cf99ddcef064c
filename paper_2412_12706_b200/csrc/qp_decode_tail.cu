// S5 for a cache with a tail: log-sum-exp merge of the split partials of one (layer, batch, query head)
// plus the attention over the tail's unquantized tokens (Eq. 2: tokens appended during decoding that
// do not fill a quantization group yet).
//
// The tail is tiny (fewer than g <= 128 tokens of D <= 128 channels per KV head) and bf16, so it never
// enters the packed-cache kernels: the warp that merges a query head's records computes the tail's logits
// itself, in fp32, and folds them into the same running (max, sum, acc) before it normalises.
// A warp per (layer, batch, query head); lane c owns channels 4c .. 4c+3.
#include <algorithm>

#include "qp_mma.cuh"

namespace qp {

namespace {

__device__ __forceinline__ float warp_max_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// One block per (layer, batch, KV head, pair of query heads of its group), one warp per query head, no shared
// staging of the tail: it is read straight from global memory, several rows at a time so that the loads do not
// wait for one another.  Two warps, at most 64 registers per thread and 1 KB of shared memory: a block fits
// into what the resident blocks of the attention kernels leave free, as the plain merge kernel's blocks do, and
// the whole grid becomes resident early; that is what lets the next call's kernels start beside this one.
constexpr int MT_WARPS = 2;
__global__ void __launch_bounds__(MT_WARPS * 32, 16)
decode_merge_tail_kernel(const __grid_constant__ DecTable tab, const __grid_constant__ TailTable tails, const DecDims dm,
                         const float* __restrict__ partials) {
  __shared__ __align__(16) float s_q[MT_WARPS][128];             // a warp's scaled query row
  const int D = dm.D, G = dm.Hq / dm.Hkv, BH = dm.Bt * dm.Hkv;
  const int tid = threadIdx.x, lane = tid & 31;
  const int ppg = (G + MT_WARPS - 1) / MT_WARPS;                 // blocks per KV head
  const int hl = (blockIdx.x % ppg) * MT_WARPS + (tid >> 5);     // query head within the group
  const bool live = hl < G;                                      // (an odd group leaves one warp without a head)
  const int layer = blockIdx.x / (ppg * BH), bh = blockIdx.x / ppg % BH;
  const DecLayer& ly = tab.l[layer];
  const TailLayer& tl = tails.l[layer];
  const int nt = tl.n_tail, RS = D * 2;                         // bytes per tail row
  const unsigned char* sK = static_cast<const unsigned char*>(tl.kt) + (size_t)bh * dm.group * D * 2;
  const unsigned char* sV = static_cast<const unsigned char*>(tl.vt) + (size_t)bh * dm.group * D * 2;
  float* sq = s_q[tid >> 5];
  const size_t stride = (size_t)G * (D + 2);
  const bool chan = 4 * lane < D;                                // this lane owns four channels
  const float scale_log2 = 1.4426950408889634f * rsqrtf((float)D);
  asm volatile("griddepcontrol.launch_dependents;\n" ::);
  asm volatile("griddepcontrol.wait;\n" ::: "memory");          // returns at once when launched in plain stream order

  // ---- the records of this query head: `count` of them, `stride` floats apart, from `base`
  const int b = bh / dm.Hkv, h = (bh % dm.Hkv) * G + hl, bq = b * dm.Hq + h;
  const float* base;
  int count;
  if (tab.n_workers > 0) {                                       // flat-range decomposition: slots head + worker
    const unsigned T = (unsigned)tab.total_tiles, W = (unsigned)tab.n_workers;
    const int tph = (ly.n + 31) >> 5;
    const unsigned first = (unsigned)ly.tile_base + (unsigned)bh * tph;
    const int w_lo = (int)(((first + 1u) * W - 1u) / T), w_hi = (int)(((first + tph) * W - 1u) / T);
    const size_t head = (size_t)layer * BH + bh;
    base = partials + ((head + w_lo) * G + hl) * (size_t)(D + 2);
    count = w_hi - w_lo + 1;
  } else {                                                       // chunked decomposition: slots of (head, split)
    const int n_splits = (ly.n + tab.chunk - 1) / tab.chunk;
    base = partials + (((size_t)ly.part_base + (size_t)bh * n_splits) * G + hl) * (size_t)(D + 2);
    count = n_splits;
  }
  float M = -INFINITY;
  if (live)
    for (int r = lane; r < count; r += 32) M = fmaxf(M, base[r * stride]);
  if (chan && live) {
    const uint2 qw = *reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(ly.q) + (size_t)bq * D + 4 * lane);
    *reinterpret_cast<float4*>(sq + 4 * lane) = make_float4(bf16lo(qw.x) * scale_log2, bf16hi(qw.x) * scale_log2,
                                                            bf16lo(qw.y) * scale_log2, bf16hi(qw.y) * scale_log2);
  }
  if (!live) return;
  __syncwarp();

  // ---- tail logits (log2 domain, like the records' maxima): lane s computes the dot product of token 32j + s
  float lt[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int tk = 32 * j + lane;
    if (tk < nt) {
      const uint4* row = reinterpret_cast<const uint4*>(sK + tk * RS);
      float d0 = 0.f, d1 = 0.f;
#pragma unroll 4
      for (int c = 0; c < D / 8; ++c) {
        const uint4 kw = row[c];
        const float4 qa = *reinterpret_cast<const float4*>(sq + 8 * c), qb = *reinterpret_cast<const float4*>(sq + 8 * c + 4);
        d0 = fmaf(qa.x, bf16lo(kw.x), fmaf(qa.y, bf16hi(kw.x), fmaf(qa.z, bf16lo(kw.y), fmaf(qa.w, bf16hi(kw.y), d0))));
        d1 = fmaf(qb.x, bf16lo(kw.z), fmaf(qb.y, bf16hi(kw.z), fmaf(qb.z, bf16lo(kw.w), fmaf(qb.w, bf16hi(kw.w), d1))));
      }
      lt[j] = d0 + d1;
    }
  }

  // ---- common reference maximum
  M = warp_max_f(fmaxf(M, fmaxf(fmaxf(lt[0], lt[1]), fmaxf(lt[2], lt[3]))));

  // ---- records, then tail tokens, in a fixed order
  float Ls = 0.f, A0 = 0.f, A1 = 0.f, A2 = 0.f, A3 = 0.f;
  if (chan)
    for (int r0 = 0; r0 < count; r0 += 4) {                      // four records' loads in flight together
      float2 ml[4], a01[4], a23[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float* rec = base + min(r0 + i, count - 1) * stride;   // past the end: the last record again, weight 0
        ml[i] = *reinterpret_cast<const float2*>(rec);
        a01[i] = *reinterpret_cast<const float2*>(rec + 2 + 4 * lane);
        a23[i] = *reinterpret_cast<const float2*>(rec + 4 + 4 * lane);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float f = r0 + i < count ? exp2f(ml[i].x - M) : 0.f;
        Ls = fmaf(ml[i].y, f, Ls);
        A0 = fmaf(a01[i].x, f, A0); A1 = fmaf(a01[i].y, f, A1);
        A2 = fmaf(a23[i].x, f, A2); A3 = fmaf(a23[i].y, f, A3);
      }
    }
  // value rows four at a time (row index clamped; the weight past the end is 0)
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float pj = exp2f(lt[j] - M);                           // weight of token 32j + lane (0 past the end)
    for (int t0 = 32 * j; t0 < min(nt, 32 * j + 32); t0 += 4) {
      uint2 vw[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        vw[i] = chan ? *reinterpret_cast<const uint2*>(sV + (size_t)min(t0 + i, nt - 1) * RS + 8 * lane) : make_uint2(0u, 0u);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float p = __shfl_sync(0xffffffffu, pj, (t0 + i) & 31);
        Ls += p;
        A0 = fmaf(p, bf16lo(vw[i].x), A0); A1 = fmaf(p, bf16hi(vw[i].x), A1);
        A2 = fmaf(p, bf16lo(vw[i].y), A2); A3 = fmaf(p, bf16hi(vw[i].y), A3);
      }
    }
  }
  if (!chan) return;
  const float inv = __fdiv_rn(1.0f, Ls);
  __nv_bfloat162 o01 = __floats2bfloat162_rn(A0 * inv, A1 * inv), o23 = __floats2bfloat162_rn(A2 * inv, A3 * inv);
  uint2 packed;
  packed.x = *reinterpret_cast<uint32_t*>(&o01);
  packed.y = *reinterpret_cast<uint32_t*>(&o23);
  *reinterpret_cast<uint2*>(static_cast<bf16*>(ly.out) + (size_t)bq * D + 4 * lane) = packed;
}

}  // namespace

cudaError_t launch_merge_tail(const DecTable& tab, const DecDims& d, const float* partials, const TailTable& tails,
                              cudaStream_t st, bool programmatic) {
  const int G = d.Hq / d.Hkv;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(tab.n_layers * d.Bt * d.Hkv * ((G + MT_WARPS - 1) / MT_WARPS));
  cfg.blockDim = dim3(32 * MT_WARPS);
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
