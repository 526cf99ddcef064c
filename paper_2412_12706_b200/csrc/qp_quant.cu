// S3: fused gather + asymmetric min/max group quantization + packing.
//
// One thread block per (batch, KV head, run of g kept tokens).  The g kept key rows are
// gathered into shared memory with 16-byte loads; thread d then owns channel d of the key
// group (g tokens, per-channel quantization) and writes its g*B/32 packed words, scale and
// zero; the value groups of the same g tokens (per-token quantization, g channels each) are
// handled one group per thread straight from global memory.
// Arithmetic is fp32 with explicit round-to-nearest intrinsics (no FMA contraction) so that
// codes, scales and zeros are reproducible bit for bit.
#include "qp_common.cuh"

namespace qp {

namespace {

struct QParams {
  float zf, sf, inv;     // inv = 1/sf, correctly rounded (0 when sf is 0 or infinite)
  __half z16, s16;
};

__device__ __forceinline__ QParams group_params(float mn, float mx, int qmax) {
  QParams p;
  p.z16 = __float2half_rd(mn);                      // zero: largest fp16 <= min
  p.zf = __half2float(p.z16);
  const float range = __fsub_rn(mx, p.zf);
  p.s16 = __float2half_ru(__fdiv_rn(range, (float)qmax));   // scale: rounded up, so max never clips
  p.sf = __half2float(p.s16);
  p.inv = p.sf != 0.f ? __frcp_rn(p.sf) : 0.f;
  return p;
}

// code = clamp(rint((x - z) / s)) with the true quotient.  The quotient is first estimated as
// (x - z) * (1/s), which is within 2^-22 relative (< 1e-4 absolute for codes up to 255) of it, so the
// rounded integer can only differ when the estimate lies that close to a half-integer; only then is
// the IEEE division done.  The result is the same integer in every case.
__device__ __forceinline__ uint32_t quant_code(float x, const QParams& p, int qmax) {
  if (p.sf == 0.f) return 0u;
  const float d = __fsub_rn(x, p.zf);
  float q = __fmul_rn(d, p.inv);
  float r = rintf(q);
  if (fabsf(q - r) > 0.4995f) r = rintf(__fdiv_rn(d, p.sf));
  // 0 <= r <= qmax already: x >= min >= z, and the scale was rounded up so (max - z)/s <= qmax (1 + 2^-23)
  return min((uint32_t)r, (uint32_t)qmax);
}

template <int BITS>
__global__ void __launch_bounds__(128)
gather_quant_kernel(const uint16_t* __restrict__ K, const uint16_t* __restrict__ V,
                    const int32_t* __restrict__ kept, int L, int D, int n, int g, uint32_t* __restrict__ Kc,
                    __half* __restrict__ Ks, __half* __restrict__ Kz, uint32_t* __restrict__ Vc,
                    __half* __restrict__ Vs, __half* __restrict__ Vz) {
  extern __shared__ __align__(16) uint16_t sK[];   // [g][D] gathered key rows
  __shared__ int sidx[128];
  constexpr int QMAX = (1 << BITS) - 1, PER = 32 / BITS;
  const int u = blockIdx.x, bh = blockIdx.y, tid = threadIdx.x, nthr = blockDim.x;
  const int wpg = g * BITS / 32;

  for (int e = tid; e < g; e += nthr) sidx[e] = kept[(size_t)bh * n + (size_t)u * g + e];
  __syncthreads();
  const uint16_t* Kh = K + (size_t)bh * L * D;
  const uint16_t* Vh = V + (size_t)bh * L * D;
  for (int c = tid; c < g * (D / 8); c += nthr) {
    const int e = c / (D / 8), col = (c % (D / 8)) * 8;
    *reinterpret_cast<uint4*>(sK + e * D + col) =
        *reinterpret_cast<const uint4*>(Kh + (size_t)sidx[e] * D + col);
  }
  __syncthreads();

  // keys: channel d, tokens e = 0..g-1
  for (int d = tid; d < D; d += nthr) {
    float mn = bf16_bits_to_f32(sK[d]), mx = mn;
    for (int e = 1; e < g; ++e) {
      const float x = bf16_bits_to_f32(sK[e * D + d]);
      mn = fminf(mn, x);
      mx = fmaxf(mx, x);
    }
    const QParams p = group_params(mn, mx, QMAX);
    const size_t gi = ((size_t)bh * (n / g) + u) * D + d;
    uint32_t* dst = Kc + gi * wpg;
    for (int wd = 0; wd < wpg; wd += 4) {       // wpg is 2 (B=2,g=32) or a multiple of 4
      uint32_t wv[4] = {0u, 0u, 0u, 0u};
      const int nw = min(4, wpg - wd);
      for (int i = 0; i < nw; ++i)
#pragma unroll
        for (int c = 0; c < PER; ++c)
          wv[i] |= quant_code(bf16_bits_to_f32(sK[((wd + i) * PER + c) * D + d]), p, QMAX) << (c * BITS);
      if (nw == 4) *reinterpret_cast<uint4*>(dst + wd) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
      else *reinterpret_cast<uint2*>(dst + wd) = make_uint2(wv[0], wv[1]);
    }
    Ks[gi] = p.s16;
    Kz[gi] = p.z16;
  }

  // values: token e, channel group v
  const int ngv = D / g;
  for (int it = tid; it < g * ngv; it += nthr) {
    const int e = it / ngv, v = it % ngv;
    const uint16_t* src = Vh + (size_t)sidx[e] * D + (size_t)v * g;
    float mn = INFINITY, mx = -INFINITY;
    for (int c8 = 0; c8 < g; c8 += 8) {
      const uint4 q = *reinterpret_cast<const uint4*>(src + c8);
      const uint32_t ww[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float x0 = bf16lo(ww[i]), x1 = bf16hi(ww[i]);
        mn = fminf(mn, fminf(x0, x1));
        mx = fmaxf(mx, fmaxf(x0, x1));
      }
    }
    const QParams p = group_params(mn, mx, QMAX);
    const size_t gi = ((size_t)bh * n + (size_t)u * g + e) * ngv + v;
    uint32_t* dst = Vc + gi * wpg;
    // second sweep over the group in 16-byte pieces (8 channels); a piece fills 8/PER words
    constexpr int WPP = PER >= 8 ? 1 : 8 / PER;                 // words completed per piece (PER 16: half a word)
    uint32_t word = 0;
    for (int c8 = 0; c8 < g; c8 += 8) {
      const uint4 q = *reinterpret_cast<const uint4*>(src + c8);
      const uint32_t ww[4] = {q.x, q.y, q.z, q.w};
      uint32_t codes[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        codes[2 * i] = quant_code(bf16lo(ww[i]), p, QMAX);
        codes[2 * i + 1] = quant_code(bf16hi(ww[i]), p, QMAX);
      }
      if constexpr (PER == 16) {                                // 2-bit: two pieces per word
        const int sh = (c8 & 8) ? 16 : 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) word |= codes[i] << (sh + i * BITS);
        if (c8 & 8) { dst[c8 / 16] = word; word = 0; }
      } else {
#pragma unroll
        for (int wq = 0; wq < WPP; ++wq) {
          uint32_t wv = 0;
#pragma unroll
          for (int i = 0; i < PER; ++i) wv |= codes[wq * PER + i] << (i * BITS);
          dst[(c8 / 8) * WPP + wq] = wv;
        }
      }
    }
    Vs[gi] = p.s16;
    Vz[gi] = p.z16;
  }
}

// B = 16: plain gather of the kept bf16 rows
__global__ void __launch_bounds__(128)
gather_rows_kernel(const uint16_t* __restrict__ K, const uint16_t* __restrict__ V,
                   const int32_t* __restrict__ kept, int L, int D, int n, uint16_t* __restrict__ Ko,
                   uint16_t* __restrict__ Vo) {
  const int bh = blockIdx.y, cpr = D / 8;            // 16-byte chunks per row
  const int rows_per_blk = blockDim.x / cpr;
  const int t = blockIdx.x * rows_per_blk + threadIdx.x / cpr, c = (threadIdx.x % cpr) * 8;
  if (t >= n || (int)threadIdx.x >= rows_per_blk * cpr) return;
  const size_t src = ((size_t)bh * L + kept[(size_t)bh * n + t]) * D + c;
  const size_t dst = ((size_t)bh * n + t) * D + c;
  *reinterpret_cast<uint4*>(Ko + dst) = *reinterpret_cast<const uint4*>(K + src);
  *reinterpret_cast<uint4*>(Vo + dst) = *reinterpret_cast<const uint4*>(V + src);
}

}  // namespace

cudaError_t launch_gather_quantize(const void* K, const void* V, const int32_t* kept, int L, const qp_cache& c,
                                   cudaStream_t st) {
  const int BH = c.batch * c.n_kv_heads, D = c.head_dim, n = c.n_keep, g = c.group;
  const uint16_t* k = static_cast<const uint16_t*>(K);
  const uint16_t* v = static_cast<const uint16_t*>(V);
  if (c.bits == 16) {
    const int rows_per_blk = 128 / (D / 8);
    gather_rows_kernel<<<dim3((n + rows_per_blk - 1) / rows_per_blk, BH), 128, 0, st>>>(
        k, v, kept, L, D, n, static_cast<uint16_t*>(c.k_codes), static_cast<uint16_t*>(c.v_codes));
    return cudaGetLastError();
  }
  const dim3 grid(n / g, BH);
  const size_t smem = (size_t)g * D * sizeof(uint16_t);
  uint32_t* kc = static_cast<uint32_t*>(c.k_codes);
  uint32_t* vc = static_cast<uint32_t*>(c.v_codes);
  __half *ks = static_cast<__half*>(c.k_scale), *kz = static_cast<__half*>(c.k_zero);
  __half *vs = static_cast<__half*>(c.v_scale), *vz = static_cast<__half*>(c.v_zero);
  switch (c.bits) {
    case 2: gather_quant_kernel<2><<<grid, 128, smem, st>>>(k, v, kept, L, D, n, g, kc, ks, kz, vc, vs, vz); break;
    case 4: gather_quant_kernel<4><<<grid, 128, smem, st>>>(k, v, kept, L, D, n, g, kc, ks, kz, vc, vs, vz); break;
    case 8: gather_quant_kernel<8><<<grid, 128, smem, st>>>(k, v, kept, L, D, n, g, kc, ks, kz, vc, vs, vz); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

}  // namespace qp
