// S3: fused gather + asymmetric min/max group quantization + packing.
//
// Two thread blocks per (batch, KV head, run of g kept tokens): one for the key group, one for the
// value rows.  The g kept key rows are gathered into shared memory with 16-byte loads; thread d then owns channel d of the key
// group (g tokens, per-channel quantization) and writes its g*B/32 packed words, scale and
// zero; the value groups of the same g tokens (per-token quantization, g channels each) are
// handled one group per thread straight from global memory.
// Arithmetic is fp32 with explicit round-to-nearest intrinsics (no FMA contraction) so that
// codes, scales and zeros are reproducible bit for bit.
#include <algorithm>

#include "qp_checked.cuh"
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
  // RN(range / qmax) by the FMA division step with the constant's reciprocal (see quant_word); exact wherever the
  // quotient is a normal fp32 number, and below that every positive quotient rounds up to the same smallest fp16
  const float qm = (float)qmax, y = 1.0f / qm;
  const float q0 = __fmul_rn(range, y);
  const float quot = __fmaf_rn(__fmaf_rn(-q0, qm, range), y, q0);
  p.s16 = __float2half_ru(quot);                    // scale: rounded up, so max never clips
  p.sf = __half2float(p.s16);
  p.inv = p.sf != 0.f ? __frcp_rn(p.sf) : 0.f;
  return p;
}

// code = rint((x - z) / s) with the correctly rounded quotient Q = RN(d / s), d = RN(x - z) >= 0, without a division
// per element: with y = RN(1/s) (once per group), q = RN(d * y) is within an ulp of the quotient, the remainder
// d - q * s comes exactly rounded out of one FMA, and q' = RN(q + rem * y) is the correctly rounded quotient (the
// classical FMA division step; s is an fp16 value, so its significand is never all ones, the one excluded case).
// Exact ties (q' = k + 1/2) are frequent with bf16 inputs and fp16 scales, and they round to even exactly as in the
// division.  Rounding adds 1.5 * 2^23 (a float below 2^22 becomes that constant plus its nearest integer, ties to
// even, in the low mantissa bits), and the codes are packed with integer shift-adds of those bit patterns, the
// constant's contribution taken off once per word.  Six instructions per element, no branch.
// (An earlier form estimated d * y, tested a margin around the half-integers and redid a word with the IEEE division
// when a lane failed the test: with exact ties in about one group in eight that redo ran for a tenth of the warps'
// words and doubled the instruction count, 13 per element under ncu.)
template <int BITS, bool FILTER>
__device__ __forceinline__ uint32_t quant_word(const float (&x)[32 / BITS], const QParams& p, float thr) {
  constexpr int PER = 32 / BITS;
  if (p.inv == 0.f) return 0u;                         // scale 0 (a constant group) or infinite: every code is 0
  constexpr float kMagic = 12582912.f;                 // 1.5 * 2^23
  constexpr uint32_t kMagicBits = 0x4B400000u;
  uint32_t acc = 0, bias = 0;
#pragma unroll
  for (int c = 0; c < PER; ++c) {
    const float d = __fsub_rn(x[c], p.zf);
    const float q = __fmul_rn(d, p.inv);
    const float rem = __fmaf_rn(-q, p.sf, d);
    const float q1 = __fmaf_rn(rem, p.inv, q);         // RN(d / s): 0 <= q1 <= qmax for an inlier
    uint32_t bits = __float_as_uint(__fadd_rn(q1, kMagic));
    if (FILTER && fabsf(x[c]) > thr) bits = kMagicBits;   // an outlier's code is 0
    acc += bits << (c * BITS);
    bias += kMagicBits << (c * BITS);                  // folded at compile time
  }
  return acc - bias;
}

// One layer's arguments.  Sources: K, V rows [BH, L, D]; kept [BH, n_idx] positions of the rows to take
// (null: row u*g + e itself, the case of a full tail).  Destinations: group u0 + u of arrays that have room for
// ns tokens per (batch, KV head).
struct QuantLayer {
  const uint16_t *K, *V;
  const int32_t* kept;
  uint32_t *Kc, *Vc;
  __half *Ks, *Kz, *Vs, *Vz;
  int L, n_idx, ns, u0;
  int k_axis = 0;          // 1: key groups run over g channels of one token, like the values
  float thr = INFINITY;    // |x| > thr: outlier, left out of min/max, code 0
};
template <int NL>
struct QuantTable {
  QuantLayer l[NL];
};

// FILTER: outlier filtering compiled in (the threshold test costs two instructions per element otherwise spent for nothing)
// D is a compile-time constant and the loops over a group run in fully unrolled chunks of 32 elements: with
// run-time extents the address arithmetic and loop control cost more instructions than the quantization itself
// (25 instructions per element under ncu against about 13 of arithmetic).
// GROUP = 32 (the usual group) is compiled with the group's 32 elements held in registers between the min/max sweep
// and the packing, and with vector stores of a group's words; GROUP = 0 takes the group size at run time.
// Twelve blocks of 128 threads per SM (40 registers, a few spilled words): the kernel waits on its gathered rows, so
// resident warps count for more than registers; measured with at least 1 / 10 / 12 / 14 blocks per SM for 8192 kept tokens
// x 64 heads: 96.7 / 93.1 / 89.9 / 96.6 us at 2 bit, 99.0 / 96.5 / 92.7 / 98.7 us at 4 bit, 113.0 / 101.6 / 100.9 / 108.9 us at 8 bit.
#ifndef QP_QUANT_MINB
#define QP_QUANT_MINB 12
#endif
template <int BITS, int NL, int D, int GROUP, bool FILTER = false>
__global__ void __launch_bounds__(128, QP_QUANT_MINB)
gather_quant_kernel(const __grid_constant__ QuantTable<NL> tab, int g_rt) {
  const int g = GROUP > 0 ? GROUP : g_rt;
  extern __shared__ __align__(16) uint16_t sK[];   // [g][D] gathered key rows
  __shared__ int sidx[128];
  constexpr int QMAX = (1 << BITS) - 1, PER = 32 / BITS;
  const QuantLayer& ql = tab.l[blockIdx.z];
  if ((int)(blockIdx.x >> 1) * g >= ql.n_idx) return;   // layers of one launch may keep different numbers of tokens
  const uint16_t* __restrict__ K = ql.K;
  const uint16_t* __restrict__ V = ql.V;
  const int32_t* __restrict__ kept = ql.kept;
  uint32_t* __restrict__ Kc = ql.Kc;
  uint32_t* __restrict__ Vc = ql.Vc;
  __half* __restrict__ Ks = ql.Ks; __half* __restrict__ Kz = ql.Kz;
  __half* __restrict__ Vs = ql.Vs; __half* __restrict__ Vz = ql.Vz;
  const int L = ql.L, n = ql.n_idx, ns = ql.ns;
  const float thr = FILTER ? ql.thr : INFINITY;
  const bool k_rows = ql.k_axis == 1;              // keys token by token: the value loop below, run on K
  // two blocks per run of g kept tokens: an even block quantizes its key group, the odd one its value rows (each has
  // a shorter chain of dependent memory round trips than one block doing both)
  const int u = blockIdx.x >> 1, bh = blockIdx.y, tid = threadIdx.x, nthr = blockDim.x;
  const bool key_part = (blockIdx.x & 1) == 0;
  const int ud = ql.u0 + u;                        // destination group
  const int wpg = g * BITS / 32;

  for (int e = tid; e < g; e += nthr) {
    const int src = kept ? kept[(size_t)bh * n + (size_t)u * g + e] : u * g + e;
    sidx[e] = QP_IN_RANGE(src, L, QP_SITE_GATHER_KEPT) ? src : 0;
  }
  __syncthreads();
  const uint16_t* Kh = K + (size_t)bh * L * D;
  const uint16_t* Vh = V + (size_t)bh * L * D;
  for (int c = tid; key_part && !k_rows && c < g * (D / 8); c += nthr) {
    const int e = c / (D / 8), col = (c % (D / 8)) * 8;
    *reinterpret_cast<uint4*>(sK + e * D + col) =
        *reinterpret_cast<const uint4*>(Kh + (size_t)sidx[e] * D + col);
  }
  __syncthreads();

  // one group of 32 elements held in registers: range, parameters, BITS packed words
  auto quant_group32 = [&](const float (&x)[32], uint32_t* dst, __half* s_out, __half* z_out) {
    float mn = INFINITY, mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      if (FILTER && fabsf(x[j]) > thr) continue;
      mn = fminf(mn, x[j]);
      mx = fmaxf(mx, x[j]);
    }
    if (mn > mx) mn = mx = 0.f;                     // outliers only
    const QParams p = group_params(mn, mx, QMAX);
    uint32_t wv[BITS];                              // 32 * BITS / 32 words
#pragma unroll
    for (int i = 0; i < BITS; ++i) {
      float xs[PER];
#pragma unroll
      for (int c = 0; c < PER; ++c) xs[c] = x[i * PER + c];
      wv[i] = quant_word<BITS, FILTER>(xs, p, thr);
    }
    if constexpr (BITS == 2) {
      *reinterpret_cast<uint2*>(dst) = make_uint2(wv[0], wv[1]);
    } else {
#pragma unroll
      for (int i = 0; i < BITS; i += 4) *reinterpret_cast<uint4*>(dst + i) = make_uint4(wv[i], wv[i + 1], wv[i + 2], wv[i + 3]);
    }
    *s_out = p.s16;
    *z_out = p.z16;
  };

  // keys: channel d, tokens e = 0..g-1
  if constexpr (GROUP == 32) {
    for (int d = tid; key_part && !k_rows && d < D; d += nthr) {
      float x[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) x[j] = bf16_bits_to_f32(sK[j * D + d]);
      const size_t gi = ((size_t)bh * (ns / 32) + ud) * D + d;
      quant_group32(x, Kc + gi * BITS, Ks + gi, Kz + gi);
    }
  }
  for (int d = tid; GROUP != 32 && key_part && !k_rows && d < D; d += nthr) {
    float mn = INFINITY, mx = -INFINITY;
    for (int e0 = 0; e0 < g; e0 += 32) {
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const float x = bf16_bits_to_f32(sK[(e0 + j) * D + d]);
        if (FILTER && fabsf(x) > thr) continue;
        mn = fminf(mn, x);
        mx = fmaxf(mx, x);
      }
    }
    if (mn > mx) mn = mx = 0.f;                     // outliers only
    const QParams p = group_params(mn, mx, QMAX);
    const size_t gi = ((size_t)bh * (ns / g) + ud) * D + d;
    uint32_t* dst = Kc + gi * wpg;
    for (int wd = 0; wd < wpg; wd += 4) {       // wpg is 2 (B=2,g=32) or a multiple of 4
      uint32_t wv[4] = {0u, 0u, 0u, 0u};
      const int nw = min(4, wpg - wd);
      for (int i = 0; i < nw; ++i) {
        float x[PER];
#pragma unroll
        for (int c = 0; c < PER; ++c) x[c] = bf16_bits_to_f32(sK[((wd + i) * PER + c) * D + d]);
        wv[i] = quant_word<BITS, FILTER>(x, p, thr);
      }
      if (nw == 4) *reinterpret_cast<uint4*>(dst + wd) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
      else *reinterpret_cast<uint2*>(dst + wd) = make_uint2(wv[0], wv[1]);
    }
    Ks[gi] = p.s16;
    Kz[gi] = p.z16;
  }

  // values: token e, channel group v
  const int ngv = D / g;
  const uint16_t* Rh = key_part ? Kh : Vh;          // rows quantized token by token by this block
  uint32_t* __restrict__ Rc = key_part ? Kc : Vc;
  __half* __restrict__ Rs = key_part ? Ks : Vs;
  __half* __restrict__ Rz = key_part ? Kz : Vz;
  if constexpr (GROUP == 32) {
    for (int it = tid; (!key_part || k_rows) && it < 32 * (D / 32); it += nthr) {
      const int e = it / (D / 32), v = it % (D / 32);
      const uint4* src = reinterpret_cast<const uint4*>(Rh + (size_t)sidx[e] * D + (size_t)v * 32);
      float x[32];
#pragma unroll
      for (int c8 = 0; c8 < 4; ++c8) {
        const uint4 q = src[c8];
        x[8 * c8 + 0] = bf16lo(q.x); x[8 * c8 + 1] = bf16hi(q.x); x[8 * c8 + 2] = bf16lo(q.y); x[8 * c8 + 3] = bf16hi(q.y);
        x[8 * c8 + 4] = bf16lo(q.z); x[8 * c8 + 5] = bf16hi(q.z); x[8 * c8 + 6] = bf16lo(q.w); x[8 * c8 + 7] = bf16hi(q.w);
      }
      const size_t gi = ((size_t)bh * ns + (size_t)ud * 32 + e) * (D / 32) + v;
      quant_group32(x, Rc + gi * BITS, Rs + gi, Rz + gi);
    }
  }
  for (int it = tid; GROUP != 32 && (!key_part || k_rows) && it < g * ngv; it += nthr) {
    const int e = it / ngv, v = it % ngv;
    const uint16_t* src = Rh + (size_t)sidx[e] * D + (size_t)v * g;
    float mn = INFINITY, mx = -INFINITY;
    for (int c32 = 0; c32 < g; c32 += 32) {
#pragma unroll
      for (int c8 = 0; c8 < 32; c8 += 8) {
        const uint4 q = *reinterpret_cast<const uint4*>(src + c32 + c8);
        const uint32_t ww[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float x0 = bf16lo(ww[i]), x1 = bf16hi(ww[i]);
          if (!FILTER || !(fabsf(x0) > thr)) { mn = fminf(mn, x0); mx = fmaxf(mx, x0); }
          if (!FILTER || !(fabsf(x1) > thr)) { mn = fminf(mn, x1); mx = fmaxf(mx, x1); }
        }
      }
    }
    if (mn > mx) mn = mx = 0.f;                     // outliers only
    const QParams p = group_params(mn, mx, QMAX);
    const size_t gi = ((size_t)bh * ns + (size_t)ud * g + e) * ngv + v;
    uint32_t* dst = Rc + gi * wpg;
    // second sweep over the group, one packed word (32/BITS channels) at a time
    for (int wd = 0; wd < wpg; ++wd) {
      float x[PER];
      const uint16_t* wsrc = src + wd * PER;
      if constexpr (PER >= 8) {
#pragma unroll
        for (int h8 = 0; h8 < PER / 8; ++h8) {
          const uint4 q = *reinterpret_cast<const uint4*>(wsrc + 8 * h8);
          x[8 * h8 + 0] = bf16lo(q.x); x[8 * h8 + 1] = bf16hi(q.x); x[8 * h8 + 2] = bf16lo(q.y); x[8 * h8 + 3] = bf16hi(q.y);
          x[8 * h8 + 4] = bf16lo(q.z); x[8 * h8 + 5] = bf16hi(q.z); x[8 * h8 + 6] = bf16lo(q.w); x[8 * h8 + 7] = bf16hi(q.w);
        }
      } else {                                                  // 8 bit: four channels = 8 bytes
        const uint2 q = *reinterpret_cast<const uint2*>(wsrc);
        x[0] = bf16lo(q.x); x[1] = bf16hi(q.x); x[2] = bf16lo(q.y); x[3] = bf16hi(q.y);
      }
      dst[wd] = quant_word<BITS, FILTER>(x, p, thr);
    }
    Rs[gi] = p.s16;
    Rz[gi] = p.z16;
  }
}

// Side list of one tensor (keys or values) of one (batch, KV head): the elements with |x| > thr of the n kept
// rows, in ascending order of t*D + d, plus the first entry of every 32-token tile.  One block walks the head
// in chunks of blockDim.x * 8 elements and compacts in order (ballot counts, one block-wide prefix per chunk),
// so the list is the same in every run.
constexpr int SL_THREADS = 256;
__global__ void __launch_bounds__(SL_THREADS)
side_list_kernel(const uint16_t* __restrict__ K, const uint16_t* __restrict__ V, const int32_t* __restrict__ kept, int L,
                 int D, int n, float thr, SideList k_out, SideList v_out) {
  __shared__ int s_warp[SL_THREADS / 32];
  __shared__ int s_base;
  const int bh = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint16_t* X = (blockIdx.y == 0 ? K : V) + (size_t)bh * L * D;
  const SideList& o = blockIdx.y == 0 ? k_out : v_out;
  int32_t* idx = const_cast<int32_t*>(o.idx) + (size_t)bh * o.cap;
  uint16_t* val = const_cast<uint16_t*>(o.val) + (size_t)bh * o.cap;
  int32_t* tile_ptr = const_cast<int32_t*>(o.tile_ptr) + (size_t)bh * (o.n_tiles + 1);
  const int32_t* kp = kept ? kept + (size_t)bh * n : nullptr;
  const int total8 = n * D / 8;                                   // 16-byte pieces
  if (tid == 0) s_base = 0;
  __syncthreads();
  for (int c0 = 0; c0 < total8; c0 += SL_THREADS) {
    const int c = c0 + tid;
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    int t = 0, d0 = 0;
    if (c < total8) {
      t = (c * 8) / D; d0 = (c * 8) % D;
      const int pos = kp ? kp[t] : t;
      const uint4 q = *reinterpret_cast<const uint4*>(X + (size_t)(QP_IN_RANGE(pos, L, QP_SITE_SIDE_KEPT) ? pos : 0) * D + d0);
      w[0] = q.x; w[1] = q.y; w[2] = q.z; w[3] = q.w;
    }
    unsigned mask = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (fabsf(bf16lo(w[i])) > thr) mask |= 1u << (2 * i);
      if (fabsf(bf16hi(w[i])) > thr) mask |= 1u << (2 * i + 1);
    }
    if (c >= total8) mask = 0;
    const int mine = __popc(mask);
    int incl = mine;                                              // inclusive prefix within the warp
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, s);
      if (lane >= s) incl += y;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    int before = s_base;
    for (int q = 0; q < warp; ++q) before += s_warp[q];
    int pos = before + incl - mine;
    // a piece that starts a 32-token tile records where the tile's entries begin
    if (c < total8 && d0 == 0 && (t & 31) == 0) tile_ptr[t >> 5] = pos;
#pragma unroll
    for (int e = 0; e < 8; ++e)
      if (mask >> e & 1u) {
        if (pos < o.cap) {
          idx[pos] = t * D + d0 + e;
          val[pos] = (uint16_t)((e & 1) ? w[e >> 1] >> 16 : w[e >> 1] & 0xffffu);
        }
        ++pos;
      }
    __syncthreads();
    if (tid == SL_THREADS - 1) s_base = before + incl;
    __syncthreads();
  }
  if (tid == 0) {
    tile_ptr[o.n_tiles] = s_base;
    const_cast<int32_t*>(o.cnt)[bh] = s_base <= o.cap ? s_base : -1;
  }
}

// B = 16: plain gather of the kept bf16 rows
__global__ void __launch_bounds__(128)
gather_rows_kernel(const uint16_t* __restrict__ K, const uint16_t* __restrict__ V,
                   const int32_t* __restrict__ kept, int L, int D, int n, int ns, uint16_t* __restrict__ Ko,
                   uint16_t* __restrict__ Vo) {
  const int bh = blockIdx.y, cpr = D / 8;            // 16-byte chunks per row
  const int rows_per_blk = blockDim.x / cpr;
  const int t = blockIdx.x * rows_per_blk + threadIdx.x / cpr, c = (threadIdx.x % cpr) * 8;
  if (t >= n || (int)threadIdx.x >= rows_per_blk * cpr) return;
  const int pos = kept[(size_t)bh * n + t];
  const size_t src = ((size_t)bh * L + (QP_IN_RANGE(pos, L, QP_SITE_ROWS_KEPT) ? pos : 0)) * D + c;
  const size_t dst = ((size_t)bh * ns + t) * D + c;   // ns: tokens the destination has room for
  *reinterpret_cast<uint4*>(Ko + dst) = *reinterpret_cast<const uint4*>(K + src);
  *reinterpret_cast<uint4*>(Vo + dst) = *reinterpret_cast<const uint4*>(V + src);
}

template <int BITS, int NL, int D>
cudaError_t launch_quant_bits(const QuantTable<NL>& tab, dim3 grid, int g, cudaStream_t st, bool filter) {
  const size_t smem = (size_t)g * D * sizeof(uint16_t);
  if constexpr (NL == 1) {
    if (filter) {
      if (g == 32) gather_quant_kernel<BITS, NL, D, 32, true><<<grid, 128, smem, st>>>(tab, g);
      else gather_quant_kernel<BITS, NL, D, 0, true><<<grid, 128, smem, st>>>(tab, g);
      return cudaGetLastError();
    }
  }
  if (g == 32) gather_quant_kernel<BITS, NL, D, 32, false><<<grid, 128, smem, st>>>(tab, g);
  else gather_quant_kernel<BITS, NL, D, 0, false><<<grid, 128, smem, st>>>(tab, g);
  return cudaGetLastError();
}
template <int NL>
cudaError_t launch_quant_table(int bits, const QuantTable<NL>& tab, dim3 grid, int D, int g, cudaStream_t st,
                               bool filter = false) {
  if (D != 64 && D != 128) return cudaErrorInvalidValue;
  switch (bits) {
    case 2: return D == 128 ? launch_quant_bits<2, NL, 128>(tab, grid, g, st, filter) : launch_quant_bits<2, NL, 64>(tab, grid, g, st, filter);
    case 4: return D == 128 ? launch_quant_bits<4, NL, 128>(tab, grid, g, st, filter) : launch_quant_bits<4, NL, 64>(tab, grid, g, st, filter);
    case 8: return D == 128 ? launch_quant_bits<8, NL, 128>(tab, grid, g, st, filter) : launch_quant_bits<8, NL, 64>(tab, grid, g, st, filter);
    default: return cudaErrorInvalidValue;
  }
}

// rows of the new token into the tails (or, at 16 bit, into the caches): 16 bytes per thread
struct AppendLayer {
  const uint16_t *k_new, *v_new;   // [BH, D]
  uint16_t *k_dst, *v_dst;         // row of head 0; heads are head_stride elements apart
  size_t head_stride;
};
struct AppendTable {
  AppendLayer l[QP_MAX_LAYERS];
};
__global__ void __launch_bounds__(128)
append_rows_kernel(const __grid_constant__ AppendTable tab, int BH, int D) {
  // This kernel sits between two decode calls of a generation loop and keeps their overlap alive: it passes
  // the launch permission on at once (the next call's attention kernel reads nothing written here), and only
  // then waits for the stream's previous kernel, whose merge step may still be reading the tail rows.
  asm volatile("griddepcontrol.launch_dependents;\n" ::);
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  const AppendLayer& a = tab.l[blockIdx.y];
  const int cpr = D / 8;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;          // 16-byte piece of the layer's [BH, D] rows
  if (i >= BH * cpr) return;
  const int bh = i / cpr, c = (i % cpr) * 8;
  *reinterpret_cast<uint4*>(a.k_dst + bh * a.head_stride + c) = *reinterpret_cast<const uint4*>(a.k_new + (size_t)bh * D + c);
  *reinterpret_cast<uint4*>(a.v_dst + bh * a.head_stride + c) = *reinterpret_cast<const uint4*>(a.v_new + (size_t)bh * D + c);
}

}  // namespace

cudaError_t launch_gather_quantize(const void* K, const void* V, const int32_t* kept, int L, const qp_cache& c,
                                   cudaStream_t st) {
  const int BH = c.batch * c.n_kv_heads, D = c.head_dim, n = c.n_keep, g = c.group, ns = cache_capacity(c);
  const uint16_t* k = static_cast<const uint16_t*>(K);
  const uint16_t* v = static_cast<const uint16_t*>(V);
  if (c.bits == 16) {
    const int rows_per_blk = 128 / (D / 8);
    gather_rows_kernel<<<dim3((n + rows_per_blk - 1) / rows_per_blk, BH), 128, 0, st>>>(
        k, v, kept, L, D, n, ns, static_cast<uint16_t*>(c.k_codes), static_cast<uint16_t*>(c.v_codes));
    return cudaGetLastError();
  }
  QuantTable<1> tab;
  tab.l[0] = QuantLayer{k, v, kept, static_cast<uint32_t*>(c.k_codes), static_cast<uint32_t*>(c.v_codes),
                        static_cast<__half*>(c.k_scale), static_cast<__half*>(c.k_zero),
                        static_cast<__half*>(c.v_scale), static_cast<__half*>(c.v_zero), L, n, ns, 0};
  return launch_quant_table<1>(c.bits, tab, dim3(2 * (n / g), BH, 1), D, g, st);
}

cudaError_t launch_gather_quantize_ex(const void* K, const void* V, const int32_t* kept, int L, const qp_cache& c,
                                      const qp_strategy& s, cudaStream_t st) {
  const int BH = c.batch * c.n_kv_heads, D = c.head_dim, n = c.n_keep, g = c.group, ns = cache_capacity(c);
  const uint16_t* k = static_cast<const uint16_t*>(K);
  const uint16_t* v = static_cast<const uint16_t*>(V);
  const bool filter = s.outlier_threshold > 0.f && s.outlier_threshold < INFINITY;
  QuantTable<1> tab;
  tab.l[0] = QuantLayer{k, v, kept, static_cast<uint32_t*>(c.k_codes), static_cast<uint32_t*>(c.v_codes),
                        static_cast<__half*>(c.k_scale), static_cast<__half*>(c.k_zero),
                        static_cast<__half*>(c.v_scale), static_cast<__half*>(c.v_zero), L, n, ns, 0,
                        s.k_axis, filter ? s.outlier_threshold : INFINITY};
  cudaError_t e = launch_quant_table<1>(c.bits, tab, dim3(2 * (n / g), BH, 1), D, g, st, filter);
  if (e != cudaSuccess || !filter) return e;
  const int n_tiles = (n + 31) / 32;
  auto side = [&](const qp_side& q) {
    return SideList{q.idx, static_cast<const uint16_t*>(q.val), q.cnt, q.tile_ptr, q.cap, n_tiles};
  };
  side_list_kernel<<<dim3(BH, 2), SL_THREADS, 0, st>>>(k, v, kept, L, D, n, s.outlier_threshold, side(s.k_side),
                                                      side(s.v_side));
  return cudaGetLastError();
}

cudaError_t launch_gather_quantize_layers(int n_layers, const void* const* K, const void* const* V,
                                          const int32_t* const* kept, int L, const qp_cache* caches, cudaStream_t st) {
  const qp_cache& c0 = caches[0];
  if (n_layers == 1 || c0.bits == 16) {            // plain row gathers: one launch per layer
    for (int l = 0; l < n_layers; ++l) {
      const cudaError_t e = launch_gather_quantize(K[l], V[l], kept[l], L, caches[l], st);
      if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
  }
  QuantTable<QP_MAX_LAYERS> tab;
  int max_groups = 0;
  for (int l = 0; l < n_layers; ++l) {
    const qp_cache& c = caches[l];
    tab.l[l] = QuantLayer{static_cast<const uint16_t*>(K[l]), static_cast<const uint16_t*>(V[l]), kept[l],
                          static_cast<uint32_t*>(c.k_codes), static_cast<uint32_t*>(c.v_codes),
                          static_cast<__half*>(c.k_scale), static_cast<__half*>(c.k_zero),
                          static_cast<__half*>(c.v_scale), static_cast<__half*>(c.v_zero), L, c.n_keep, cache_capacity(c), 0};
    max_groups = std::max(max_groups, c.n_keep / c.group);
  }
  return launch_quant_table<QP_MAX_LAYERS>(c0.bits, tab, dim3(2 * max_groups, c0.batch * c0.n_kv_heads, n_layers),
                                           c0.head_dim, c0.group, st);
}

cudaError_t launch_append_rows(int n_layers, const void* const* k_new, const void* const* v_new, const qp_cache* caches,
                               const qp_tail* tails, cudaStream_t st) {
  const qp_cache& c0 = caches[0];
  const int BH = c0.batch * c0.n_kv_heads, D = c0.head_dim;
  AppendTable tab;
  for (int l = 0; l < n_layers; ++l) {
    const qp_cache& c = caches[l];
    AppendLayer& a = tab.l[l];
    a.k_new = static_cast<const uint16_t*>(k_new[l]);
    a.v_new = static_cast<const uint16_t*>(v_new[l]);
    if (c.bits == 16) {                                          // token n_keep of the cache itself
      a.head_stride = (size_t)cache_capacity(c) * D;
      a.k_dst = static_cast<uint16_t*>(c.k_codes) + (size_t)c.n_keep * D;
      a.v_dst = static_cast<uint16_t*>(c.v_codes) + (size_t)c.n_keep * D;
    } else {                                                     // slot n_tail of the tail
      a.head_stride = (size_t)c.group * D;
      a.k_dst = static_cast<uint16_t*>(tails[l].k_tail) + (size_t)tails[l].n_tail * D;
      a.v_dst = static_cast<uint16_t*>(tails[l].v_tail) + (size_t)tails[l].n_tail * D;
    }
  }
  const int pieces = BH * (D / 8);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((pieces + 127) / 128, n_layers);
  cfg.blockDim = dim3(128);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, append_rows_kernel, tab, BH, D);
}

// which[0..n_layers): indices into caches / tails of the layers whose tail is full
cudaError_t launch_flush_tails(int n_layers, const int* which, const qp_cache* caches, const qp_tail* tails,
                               cudaStream_t st) {
  const qp_cache& c0 = caches[which[0]];
  const int BH = c0.batch * c0.n_kv_heads, D = c0.head_dim, g = c0.group;
  auto fill = [&](QuantLayer& ql, int l) {
    const qp_cache& c = caches[l];
    ql = QuantLayer{static_cast<const uint16_t*>(tails[l].k_tail), static_cast<const uint16_t*>(tails[l].v_tail), nullptr,
                    static_cast<uint32_t*>(c.k_codes), static_cast<uint32_t*>(c.v_codes),
                    static_cast<__half*>(c.k_scale), static_cast<__half*>(c.k_zero),
                    static_cast<__half*>(c.v_scale), static_cast<__half*>(c.v_zero),
                    g, g, cache_capacity(c), c.n_keep / g};
  };
  if (n_layers == 1) {
    QuantTable<1> tab;
    fill(tab.l[0], which[0]);
    return launch_quant_table<1>(c0.bits, tab, dim3(2, BH, 1), D, g, st);
  }
  QuantTable<QP_MAX_LAYERS> tab;
  for (int i = 0; i < n_layers; ++i) fill(tab.l[i], which[i]);
  return launch_quant_table<QP_MAX_LAYERS>(c0.bits, tab, dim3(2, BH, n_layers), D, g, st);
}

#ifdef QP_CHECKED
cudaError_t quant_check_read(unsigned int (&out)[4]) { return checked::read_and_clear(out); }
#endif

}  // namespace qp
