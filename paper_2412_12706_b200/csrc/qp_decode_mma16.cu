// S4 on tensor cores for 16-bit caches (the gathered bf16 rows, no scale/zero).
//
// Plain flash-decoding on mma.sync bf16: S^T = Q K^T with the query heads of the GQA group as the
// MMA rows (rows 8..15 are unused), so the probabilities come out of the accumulators in exactly
// the register layout the second product O = P V wants for its A operand; K is read with ldmatrix
// (rows = tokens), V with the transposing form.  Same flat-range decomposition and partial records
// as the quantised kernels.  n need not be a multiple of 32: the ragged tail is zero-filled and masked.
#include "qp_mma.cuh"

namespace qp {

namespace {

constexpr int D16_WARPS = 4;
constexpr int D16_THREADS = D16_WARPS * 32;
constexpr int D16_STAGES = 3;
constexpr int D16_MINB = 1;

template <int D>
struct Tile16 {
  static constexpr int KC = 0;                // 32 token rows of 2D bytes, 16-byte chunks XOR-swizzled by token & 7
  static constexpr int VC = KC + 64 * D;
  static constexpr int BYTES = VC + 64 * D;
};

__device__ __forceinline__ void cp_async16_zf(uint32_t saddr, const void* gptr, bool valid) {
  const int n = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(saddr), "l"(gptr), "r"(n));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

template <int D>
__global__ void __launch_bounds__(D16_THREADS, D16_MINB)
decode_mma16_kernel(const __grid_constant__ DecTable tab, const DecDims dm, float* __restrict__ partials) {
  using TL = Tile16<D>;
  constexpr int CPR = D / 8;       // 16-byte chunks per token row
  constexpr int KST = D / 16;      // k-steps of Q K^T
  constexpr int NJ = D / 8;        // channel n-tiles of P V
  extern __shared__ __align__(128) unsigned char smem[];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int G = dm.Hq / dm.Hkv, BH = dm.Bt * dm.Hkv;
  const SkOwner sk{tab.total_tiles, tab.n_workers};
  const int cta = blockIdx.x;
  long long cur = sk.start(cta);
  const long long f_end = sk.start(cta + 1);

  const uint32_t wsm_u = smem_u32(smem + warp * (D16_STAGES * TL::BYTES));
  float* s_acc = reinterpret_cast<float*>(smem);                // [warp][8 heads][D], overlays the idle stages
  float* s_m = s_acc + D16_WARPS * 8 * D;
  float* s_l = s_m + D16_WARPS * 8;
  const float scale_log2 = 1.4426950408889634f * rsqrtf((float)D);

  // ldmatrix row of this lane: token (lane & 7) of an 8-token matrix, chunk select by lane >> 3
  const int lrow = lane & 7, lsel = lane >> 3;

  int li = 0;
  while (li + 1 < tab.n_layers && tab.l[li + 1].tile_base <= cur) ++li;

  while (cur < f_end) {
    const DecLayer& ly = tab.l[li];
    const int n = ly.n, tph = (n + 31) >> 5;
    const int rel = (int)(cur - ly.tile_base), bh = rel / tph, tile_begin = rel % tph;
    const int n_tiles = (int)min((long long)(tph - tile_begin), f_end - cur);
    const int b = bh / dm.Hkv, hk = bh % dm.Hkv;
    const unsigned char* gK = static_cast<const unsigned char*>(ly.kc) + (size_t)bh * ly.ns * D * 2;
    const unsigned char* gV = static_cast<const unsigned char*>(ly.vc) + (size_t)bh * ly.ns * D * 2;

    auto issue_tile = [&](int tile, int stage) {
      const uint32_t sb = wsm_u + stage * TL::BYTES;
      const int tok0 = tile * 32;
#pragma unroll
      for (int i = 0; i < CPR; ++i) {                           // 32 * CPR pieces per matrix, CPR per lane
        const int idx = lane + 32 * i, tau = idx / CPR, ch = idx % CPR;
        const bool ok = tok0 + tau < n;
        const size_t off = ok ? ((size_t)(tok0 + tau) * D * 2 + ch * 16) : 0;
        const uint32_t dst = tau * (2 * D) + ((ch ^ (tau & 7)) << 4);
        cp_async16_zf(sb + TL::KC + dst, gK + off, ok);
        cp_async16_zf(sb + TL::VC + dst, gV + off, ok);
      }
    };

    const int n_my = warp < n_tiles ? (n_tiles - warp + D16_WARPS - 1) / D16_WARPS : 0;
#pragma unroll
    for (int s = 0; s < D16_STAGES - 1; ++s) {
      if (s < n_my) issue_tile(tile_begin + warp + D16_WARPS * s, s);
      cp_async_commit();
    }

    // A fragments of Q: row g = query head g of this KV head (exact bf16; rows >= G and 8..15 are zero)
    uint32_t qa[KST][2];
    {
      const uint16_t* qp = static_cast<const uint16_t*>(ly.q) + ((size_t)(b * dm.Hq + hk * G + g)) * D;
#pragma unroll
      for (int c = 0; c < KST; ++c) {
        qa[c][0] = g < G ? *reinterpret_cast<const uint32_t*>(qp + 16 * c + 2 * t) : 0u;
        qa[c][1] = g < G ? *reinterpret_cast<const uint32_t*>(qp + 16 * c + 8 + 2 * t) : 0u;
      }
    }

    float m_run = -INFINITY, l_run = 0.f;                       // head g (replicated over t)
    float accO[NJ][4];
#pragma unroll
    for (int j = 0; j < NJ; ++j)
#pragma unroll
      for (int x = 0; x < 4; ++x) accO[j][x] = 0.f;

    const bool last_seg = cur + n_tiles >= f_end;
    for (int it = 0; it < n_my; ++it) {
      if (last_seg && it == n_my - 1) pdl_gate();               // see qp_mma.cuh (a warp without tiles leaves it to the others)
      __syncwarp();
      if (it + D16_STAGES - 1 < n_my)
        issue_tile(tile_begin + warp + D16_WARPS * (it + D16_STAGES - 1), (it + D16_STAGES - 1) % D16_STAGES);
      cp_async_commit();
      cp_async_wait<D16_STAGES - 1>();
      __syncwarp();
      const uint32_t sb = wsm_u + (it % D16_STAGES) * TL::BYTES;
      const int tok0 = (tile_begin + warp + D16_WARPS * it) * 32;

      // ---------------- S^T = Q K^T: 4 token n-tiles x KST k-steps
      float sc[4][4];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
        const int tau = 8 * nt + lrow;
#pragma unroll
        for (int c = 0; c < KST; c += 2) {
          // matrices: (k 16c..+7), (k 16c+8..), (k 16c+16..), (k 16c+24..) of tokens 8nt..8nt+7
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4(b0, b1, b2, b3, sb + TL::KC + tau * (2 * D) + (((2 * c + lsel) ^ (tau & 7)) << 4));
          mma_bf16_m16n8k16(sc[nt], {qa[c][0], 0u, qa[c][1], 0u}, b0, b1);
          mma_bf16_m16n8k16(sc[nt], {qa[c + 1][0], 0u, qa[c + 1][1], 0u}, b2, b3);
        }
      }
      // this lane: head g, tokens tok0 + 8nt + 2t (+1)
      float mx = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const int tk = tok0 + 8 * nt + 2 * t;
        sc[nt][0] = tk < n ? sc[nt][0] * scale_log2 : -INFINITY;
        sc[nt][1] = tk + 1 < n ? sc[nt][1] * scale_log2 : -INFINITY;
        mx = fmaxf(mx, fmaxf(sc[nt][0], sc[nt][1]));
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float mnew = fmaxf(m_run, mx);                      // finite: the first token of a tile is < n
      const float corr = ex2(m_run - mnew);
      m_run = mnew;
      float sum = 0.f;
      uint32_t pa[4];                                           // bf16 pairs: tokens 8nt + 2t, +1
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const float p0 = ex2(sc[nt][0] - mnew), p1 = ex2(sc[nt][1] - mnew);
        sum += p0 + p1;
        pa[nt] = pack_bf16x2(p0, p1);
      }
      l_run = fmaf(l_run, corr, sum);
      if (__any_sync(0xffffffffu, corr != 1.f)) {
#pragma unroll
        for (int j = 0; j < NJ; ++j) { accO[j][0] *= corr; accO[j][1] *= corr; }
      }

      // ---------------- O += P V: channel n-tiles x 2 k-steps of 16 tokens
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        const int tau = 8 * lsel + lrow;                        // matrices: tokens 0-7, 8-15, 16-23, 24-31
        uint32_t v0, v1, v2, v3;
        ldmatrix_x4_trans(v0, v1, v2, v3, sb + TL::VC + tau * (2 * D) + ((j ^ (tau & 7)) << 4));
        mma_bf16_m16n8k16(accO[j], {pa[0], 0u, pa[1], 0u}, v0, v1);
        mma_bf16_m16n8k16(accO[j], {pa[2], 0u, pa[3], 0u}, v2, v3);
      }
    }

    // ---------------- per-warp result -> shared memory -> one partial per (head, block) and query head
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    __syncthreads();
    {
      float* o = s_acc + ((warp * 8 + g) * D);
#pragma unroll
      for (int j = 0; j < NJ; ++j)
        *reinterpret_cast<float2*>(o + 8 * j + 2 * t) = make_float2(accO[j][0], accO[j][1]);
      if (t == 0) { s_m[warp * 8 + g] = m_run; s_l[warp * 8 + g] = l_run; }
    }
    __syncthreads();
    const size_t slot = (size_t)li * BH + bh + cta;
    for (int idx = tid; idx < G * D; idx += D16_THREADS) {
      const int h = idx / D, d = idx % D;
      float M = -INFINITY;
#pragma unroll
      for (int wp = 0; wp < D16_WARPS; ++wp) M = fmaxf(M, s_m[wp * 8 + h]);
      float Ls = 0.f, A = 0.f;
#pragma unroll
      for (int wp = 0; wp < D16_WARPS; ++wp) {
        const float mw = s_m[wp * 8 + h];
        if (mw != -INFINITY) {
          const float f = ex2(mw - M);
          Ls = fmaf(s_l[wp * 8 + h], f, Ls);
          A = fmaf(s_acc[(wp * 8 + h) * D + d], f, A);
        }
      }
      float* op = partials + (slot * G + h) * (size_t)(D + 2);
      if (d == 0) { op[0] = M; op[1] = Ls; }
      op[2 + d] = A;
    }
    __syncthreads();

    cur += n_tiles;
    if (bh == BH - 1 && tile_begin + n_tiles == tph) ++li;
  }
}

template <int D>
constexpr size_t mma16_smem_bytes() {
  return (size_t)D16_WARPS * D16_STAGES * Tile16<D>::BYTES;
}

}  // namespace

int decode_mma16_blocks_per_sm() { return D16_MINB; }

cudaError_t launch_decode_mma16(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st,
                                bool overlap_prev) {
  if (d.D == 128) {
    constexpr size_t smem = mma16_smem_bytes<128>();
    static unsigned char done[64] = {};
    const cudaError_t e = allow_smem(decode_mma16_kernel<128>, smem, done);
    if (e != cudaSuccess) return e;
    return launch_attention(decode_mma16_kernel<128>, tab.n_workers, D16_THREADS, smem, st, overlap_prev, tab, d, partials);
  }
  constexpr size_t smem = mma16_smem_bytes<64>();
  static unsigned char done[64] = {};
  const cudaError_t e = allow_smem(decode_mma16_kernel<64>, smem, done);
  if (e != cudaSuccess) return e;
  return launch_attention(decode_mma16_kernel<64>, tab.n_workers, D16_THREADS, smem, st, overlap_prev, tab, d, partials);
}

}  // namespace qp
