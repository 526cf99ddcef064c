// S4 on tensor cores for 8-bit caches (groups of 32, 64 or 128).
//
// Same scheme as the 4-bit kernel: a byte c in the low byte of a 16-bit lane is the f16 number
// c * 2^-24 (255 is still below the end of the first binade), so (word & 0x00ff00ff) and a byte
// permute of the odd bytes are f16 operand pairs.  A 16-bit unit holds two codes, so one 32-token
// key group of a channel is two 16-byte rows (tokens 0-15, 16-31); they are kept in two planes so
// that the transposing loads stay conflict-free.  Rows of an MMA tile: tokens (16 hf + 2g, +1) on
// the key side, channels (16 q + 2g, +1) on the value side.
#include "qp_mma.cuh"

namespace qp {

namespace {

constexpr int D8_WARPS = 4;
constexpr int D8_THREADS = D8_WARPS * 32;
#ifndef QP_D8_STAGES
#define QP_D8_STAGES 2
#endif
constexpr int D8_STAGES = QP_D8_STAGES;
constexpr int D8_MINB = 2;
constexpr int SP8_STRIDE = 80;
constexpr int SP8_BYTES = 8 * SP8_STRIDE;

template <int D>
struct Tile8 {
  static constexpr int KC = 0;                    // 2 planes (tokens 0-15 / 16-31) of D rows of 16 B
  static constexpr int KS = KC + 32 * D;          // D halves, channels >= 64 shifted by 16 B
  static constexpr int KZ = KS + 2 * D + 16;
  static constexpr int VC = KZ + 2 * D + 16;      // 32 token rows of D bytes
  static constexpr int VS = VC + 32 * D;          // 32 x (D/32) halves
  static constexpr int VZ = VS + 2 * D;
  static constexpr int BYTES = VZ + 2 * D;
};
__host__ __device__ constexpr int ksz_off8(int ch) { return ch * 2 + (ch / 64) * 16; }

constexpr uint32_t M8 = 0x00ff00ffu;
constexpr float C24 = 16777216.0f;
__device__ __forceinline__ uint32_t odd_bytes(uint32_t r) { return __byte_perm(r, 0u, 0x4341); }

template <int D, int GROUP>
__global__ void __launch_bounds__(D8_THREADS, D8_MINB)
decode_mma8_kernel(const __grid_constant__ DecTable tab, const DecDims dm, float* __restrict__ partials) {
  using TL = Tile8<D>;
  constexpr int NG = D / GROUP;    // value scale groups per token
  constexpr int GT = GROUP / 32;   // 32-token tiles per key group
  constexpr int NQ = D / 16;       // 16-byte pieces per value row = k-steps over the key channels
  constexpr int NPAIR = D / 8;     // channel pairs owned by one lane on the key side
  extern __shared__ __align__(128) unsigned char smem[];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int G = dm.Hq / dm.Hkv, BH = dm.Bt * dm.Hkv;
  const SkOwner sk{tab.total_tiles, tab.n_workers};
  const int cta = blockIdx.x;
  asm volatile("griddepcontrol.launch_dependents;\n" ::);
  long long cur = sk.start(cta);
  const long long f_end = sk.start(cta + 1);

  unsigned char* wsm = smem + warp * (D8_STAGES * TL::BYTES + SP8_BYTES);
  const uint32_t wsm_u = smem_u32(wsm);
  const uint32_t sP = wsm_u + D8_STAGES * TL::BYTES;
  float* s_acc = reinterpret_cast<float*>(smem);                // [warp][8][D], overlays the idle stages
  float* s_m = s_acc + D8_WARPS * 8 * D;
  float* s_l = s_m + D8_WARPS * 8;

  // sources of the transposing loads
  uint32_t k_plane, k_slot0, v_row, v_sw;
  {
    const int m = lane >> 3, r = lane & 7, tq = r >> 1, p = r & 1;
    const int hf = m >> 1, set = m & 1;                         // matrices: (hf 0, k 0-7), (hf 0, k 8-15), (hf 1, ..)
    k_plane = TL::KC + hf * 16 * D;
    k_slot0 = ((D / 4) * tq + 2 * set + p) ^ (tq << 1);         // k-step c adds channel 4c: slot0 ^ 4c (disjoint bits)
    const int tau = 8 * m + r;                                  // value side: matrix m = tokens 8m .. 8m+7
    v_row = TL::VC + tau * D;
    v_sw = NQ == 8 ? (tau & 7) : ((tau >> 1) & 3);
  }
  constexpr int MCH = D / 8;
  const int mj = lane < MCH ? lane : lane - MCH;
  const uint32_t ksz_dst = (lane < MCH ? TL::KS : TL::KZ) + mj * 16 + (mj / 8) * 16;
  const uint32_t vsz_dst = (lane < MCH ? TL::VS : TL::VZ) + mj * 16;

  int li = 0;
  while (li + 1 < tab.n_layers && tab.l[li + 1].tile_base <= cur) ++li;

  while (cur < f_end) {
    const DecLayer& ly = tab.l[li];
    const int n = ly.n, tph = n >> 5;
    const int rel = (int)(cur - ly.tile_base), bh = rel / tph, tile_begin = rel % tph;
    const int n_tiles = (int)min((long long)(tph - tile_begin), f_end - cur);
    const int b = bh / dm.Hkv, hk = bh % dm.Hkv;

    const unsigned char* gKc = static_cast<const unsigned char*>(ly.kc) + (size_t)bh * tph * D * 32;
    const unsigned char* gKs = reinterpret_cast<const unsigned char*>(ly.ks) + (size_t)bh * (n / GROUP) * D * 2;
    const unsigned char* gKz = reinterpret_cast<const unsigned char*>(ly.kz) + (size_t)bh * (n / GROUP) * D * 2;
    const unsigned char* gVc = static_cast<const unsigned char*>(ly.vc) + (size_t)bh * n * D;
    const unsigned char* gVs = reinterpret_cast<const unsigned char*>(ly.vs) + (size_t)bh * n * NG * 2;
    const unsigned char* gVz = reinterpret_cast<const unsigned char*>(ly.vz) + (size_t)bh * n * NG * 2;
    const unsigned char* gKm = lane < MCH ? gKs : gKz;
    const unsigned char* gVm = lane < MCH ? gVs : gVz;

    auto issue_tile = [&](int tile, int stage) {
      const uint32_t sb = wsm_u + stage * TL::BYTES;
      const int u = tile / GT, sub = tile % GT;                 // a key group is GROUP bytes per channel
      const unsigned char* kc = gKc + (size_t)u * D * GROUP + sub * 32;
      const unsigned char* vc = gVc + (size_t)tile * 32 * D + lane * 16;
#pragma unroll
      for (int i = 0; i < D / 16; ++i) {
        const int pi = lane + 32 * i;                           // key piece: channel pi/2, token half pi&1
        const int c = pi >> 1, hf = pi & 1;
        cp_async16(sb + TL::KC + hf * 16 * D + ((c ^ ((c / (D / 4)) << 1)) << 4), kc + c * GROUP + hf * 16);
        const int tau = pi / NQ, q = pi % NQ;                   // value piece: token tau, channels 16q .. 16q+15
        const int sw = NQ == 8 ? (tau & 7) : ((tau >> 1) & 3);
        cp_async16(sb + TL::VC + tau * D + ((q ^ sw) << 4), vc + i * 512);
      }
      if (lane < 2 * MCH) {
        cp_async16(sb + ksz_dst, gKm + (size_t)u * D * 2 + mj * 16);
        if (mj < 4 * NG) cp_async16(sb + vsz_dst, gVm + (size_t)tile * 64 * NG + mj * 16);
      }
    };

    const int n_my = warp < n_tiles ? (n_tiles - warp + D8_WARPS - 1) / D8_WARPS : 0;
#pragma unroll
    for (int s = 0; s < D8_STAGES - 1; ++s) {
      if (s < n_my) issue_tile(tile_begin + warp + D8_WARPS * s, s);
      cp_async_commit();
    }

    uint32_t qh2[NPAIR];
    {
      const float scale_log2 = 1.4426950408889634f * rsqrtf((float)D);
      const uint16_t* qp = static_cast<const uint16_t*>(ly.q) + ((size_t)(b * dm.Hq + hk * G + g)) * D + (D / 4) * t;
#pragma unroll
      for (int i = 0; i < NPAIR; i += 4) {
        uint4 w4 = make_uint4(0u, 0u, 0u, 0u);
        if (g < G) w4 = *reinterpret_cast<const uint4*>(qp + 2 * i);
        qh2[i + 0] = pack_half2(bf16lo(w4.x) * scale_log2, bf16hi(w4.x) * scale_log2);
        qh2[i + 1] = pack_half2(bf16lo(w4.y) * scale_log2, bf16hi(w4.y) * scale_log2);
        qh2[i + 2] = pack_half2(bf16lo(w4.z) * scale_log2, bf16hi(w4.z) * scale_log2);
        qh2[i + 3] = pack_half2(bf16lo(w4.w) * scale_log2, bf16hi(w4.w) * scale_log2);
      }
    }

    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    float accO[NQ][4], accPZ[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int q = 0; q < NQ; ++q)
#pragma unroll
      for (int x = 0; x < 4; ++x) accO[q][x] = 0.f;

    for (int it = 0; it < n_my; ++it) {
      __syncwarp();
      if (it + D8_STAGES - 1 < n_my)
        issue_tile(tile_begin + warp + D8_WARPS * (it + D8_STAGES - 1), (it + D8_STAGES - 1) % D8_STAGES);
      cp_async_commit();
      cp_async_wait<D8_STAGES - 1>();
      __syncwarp();
      const uint32_t sb = wsm_u + (it % D8_STAGES) * TL::BYTES;

      // ---------------- keys: m-tile hf holds tokens 16hf + 2g (rows g) and 16hf + 2g + 1 (rows g+8)
      float accK[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}}, accZ[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c2 = 0; c2 < NQ / 2; ++c2) {                     // two k-steps (8 channels of this lane) per round
        const uint4 s4 = lds128(sb + TL::KS + ksz_off8((D / 4) * t + 8 * c2));
        const uint4 z4 = lds128(sb + TL::KZ + ksz_off8((D / 4) * t + 8 * c2));
        const uint32_t sv[4] = {s4.x, s4.y, s4.z, s4.w}, zv[4] = {z4.x, z4.y, z4.z, z4.w};
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          const int c = 2 * c2 + cc;
          const uint32_t b0 = hmul2_u32(qh2[2 * c], sv[2 * cc]), b1 = hmul2_u32(qh2[2 * c + 1], sv[2 * cc + 1]);
          uint32_t R0, R1, R2, R3;
          ldmatrix_x4_trans(R0, R1, R2, R3, sb + k_plane + ((k_slot0 ^ (4 * c)) << 4));
          mma_f16_m16n8k16(accK[0], R0 & M8, odd_bytes(R0), R1 & M8, odd_bytes(R1), b0, b1);
          mma_f16_m16n8k16(accK[1], R2 & M8, odd_bytes(R2), R3 & M8, odd_bytes(R3), b0, b1);
          mma_f16_m16n8k16(accZ, zv[2 * cc], zv[2 * cc], zv[2 * cc + 1], zv[2 * cc + 1], qh2[2 * c], qh2[2 * c + 1]);
        }
      }
      // lg[j][x]: tokens {2g, 2g+1, 16+2g, 17+2g}[j], column 2t + x
      float lg[4][2];
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        lg[2 * hf][0] = fmaf(accK[hf][0], C24, accZ[0]);
        lg[2 * hf][1] = fmaf(accK[hf][1], C24, accZ[1]);
        lg[2 * hf + 1][0] = fmaf(accK[hf][2], C24, accZ[0]);
        lg[2 * hf + 1][1] = fmaf(accK[hf][3], C24, accZ[1]);
      }

      float corr[2];
#pragma unroll
      for (int x = 0; x < 2; ++x) {
        float mx = fmaxf(fmaxf(lg[0][x], lg[1][x]), fmaxf(lg[2][x], lg[3][x]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
        const float mnew = fmaxf(m_run[x], mx);
        corr[x] = ex2(m_run[x] - mnew);
        m_run[x] = mnew;
        float sum = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          lg[j][x] = ex2(lg[j][x] - mnew);
          sum += lg[j][x];
        }
        l_run[x] = fmaf(l_run[x], corr[x], sum);
      }
      if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
          accO[q][0] *= corr[0]; accO[q][1] *= corr[1];
          accO[q][2] *= corr[0]; accO[q][3] *= corr[1];
        }
        accPZ[0] *= corr[0]; accPZ[1] *= corr[1];
      }

      // ---------------- P through shared memory: [column][token] f16
#pragma unroll
      for (int x = 0; x < 2; ++x) {
        const uint32_t row = sP + (2 * t + x) * SP8_STRIDE + 4 * g;
        asm volatile("st.shared.u32 [%0], %1;\n" ::"r"(row), "r"(pack_half2(lg[0][x], lg[1][x])));
        asm volatile("st.shared.u32 [%0], %1;\n" ::"r"(row + 32), "r"(pack_half2(lg[2][x], lg[3][x])));
      }
      __syncwarp();
      uint32_t p2[4];
#pragma unroll
      for (int pr = 0; pr < 4; ++pr) p2[pr] = lds32(sP + g * SP8_STRIDE + 4 * t + 16 * pr);

      // ---------------- values
      uint32_t ps[4][NG], zp[4];                                // ps[pair][scale group], zero-point rows: group g
#pragma unroll
      for (int pr = 0; pr < 4; ++pr) {
        const int a = 8 * pr + 2 * t;
        zp[pr] = 0u;
        if constexpr (NG == 4) {
          const uint4 x = lds128(sb + TL::VS + a * 8);
          ps[pr][0] = hmul2_u32(p2[pr], __byte_perm(x.x, x.z, 0x5410));
          ps[pr][1] = hmul2_u32(p2[pr], __byte_perm(x.x, x.z, 0x7632));
          ps[pr][2] = hmul2_u32(p2[pr], __byte_perm(x.y, x.w, 0x5410));
          ps[pr][3] = hmul2_u32(p2[pr], __byte_perm(x.y, x.w, 0x7632));
          if (g < NG) {
            const uint32_t ya = lds32(sb + TL::VZ + a * 8 + (g & 2) * 2);
            const uint32_t yb = lds32(sb + TL::VZ + a * 8 + 8 + (g & 2) * 2);
            zp[pr] = __byte_perm(ya, yb, (g & 1) ? 0x7632 : 0x5410);
          }
        } else if constexpr (NG == 2) {
          const uint2 x = lds64(sb + TL::VS + a * 4);
          ps[pr][0] = hmul2_u32(p2[pr], __byte_perm(x.x, x.y, 0x5410));
          ps[pr][1] = hmul2_u32(p2[pr], __byte_perm(x.x, x.y, 0x7632));
          if (g < NG) {
            const uint2 y = lds64(sb + TL::VZ + a * 4);
            zp[pr] = __byte_perm(y.x, y.y, (g & 1) ? 0x7632 : 0x5410);
          }
        } else {                                                // one scale per token: the pair is one word
          ps[pr][0] = hmul2_u32(p2[pr], lds32(sb + TL::VS + a * 2));
          if (g == 0) zp[pr] = lds32(sb + TL::VZ + a * 2);
        }
      }
      mma_f16_m16n8k16(accPZ, zp[0], 0u, zp[1], 0u, p2[0], p2[1]);
      mma_f16_m16n8k16(accPZ, zp[2], 0u, zp[3], 0u, p2[2], p2[3]);
#pragma unroll
      for (int q = 0; q < NQ; ++q) {                            // rows: channels 16q + 2g (g) and 16q + 2g + 1 (g+8)
        uint32_t R0, R1, R2, R3;
        ldmatrix_x4_trans(R0, R1, R2, R3, sb + v_row + ((q ^ v_sw) << 4));
        mma_f16_m16n8k16(accO[q], R0 & M8, odd_bytes(R0), R1 & M8, odd_bytes(R1), ps[0][q * NG / NQ], ps[1][q * NG / NQ]);
        mma_f16_m16n8k16(accO[q], R2 & M8, odd_bytes(R2), R3 & M8, odd_bytes(R3), ps[2][q * NG / NQ], ps[3][q * NG / NQ]);
      }
    }

    // ---------------- per-warp result -> shared memory -> one partial per (head, block) and query head
#pragma unroll
    for (int x = 0; x < 2; ++x) {
      l_run[x] += __shfl_xor_sync(0xffffffffu, l_run[x], 4);
      l_run[x] += __shfl_xor_sync(0xffffffffu, l_run[x], 8);
      l_run[x] += __shfl_xor_sync(0xffffffffu, l_run[x], 16);
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
      const int v = q * NG / NQ;                                // scale group of channels 16q ..
      const float pz0 = __shfl_sync(0xffffffffu, accPZ[0], 4 * v + t);
      const float pz1 = __shfl_sync(0xffffffffu, accPZ[1], 4 * v + t);
      const int ch = 16 * q + 2 * g;
      float* o0 = s_acc + ((warp * 8 + 2 * t) * D);
      float* o1 = o0 + D;
      *reinterpret_cast<float2*>(o0 + ch) = make_float2(fmaf(accO[q][0], C24, pz0), fmaf(accO[q][2], C24, pz0));
      *reinterpret_cast<float2*>(o1 + ch) = make_float2(fmaf(accO[q][1], C24, pz1), fmaf(accO[q][3], C24, pz1));
    }
    if (g == 0) {
      s_m[warp * 8 + 2 * t] = m_run[0]; s_m[warp * 8 + 2 * t + 1] = m_run[1];
      s_l[warp * 8 + 2 * t] = l_run[0]; s_l[warp * 8 + 2 * t + 1] = l_run[1];
    }
    __syncthreads();
    const size_t slot = (size_t)li * BH + bh + cta;
    for (int idx = tid; idx < G * D; idx += D8_THREADS) {
      const int h = idx / D, d = idx % D;
      float M = -INFINITY;
#pragma unroll
      for (int wp = 0; wp < D8_WARPS; ++wp) M = fmaxf(M, s_m[wp * 8 + h]);
      float Ls = 0.f, A = 0.f;
#pragma unroll
      for (int wp = 0; wp < D8_WARPS; ++wp) {
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
  // (see the 4-bit kernel: a call may start before the previous call's merge kernel has ended; the call after it
  // relies on this grid not ending before that kernel has)
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
}

template <int D>
constexpr size_t mma8_smem_bytes() {
  constexpr size_t stages = (size_t)D8_WARPS * (D8_STAGES * Tile8<D>::BYTES + SP8_BYTES);
  constexpr size_t combine = (size_t)D8_WARPS * 8 * D * 4 + 2 * D8_WARPS * 8 * 4;
  return stages > combine ? stages : combine;
}

}  // namespace

int decode_mma8_blocks_per_sm() { return D8_MINB; }

namespace {
template <int D, int GROUP>
cudaError_t launch_mma8(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st, bool overlap_prev) {
  constexpr size_t smem = mma8_smem_bytes<D>();
  static unsigned char done[64] = {};
  const cudaError_t e = allow_smem(decode_mma8_kernel<D, GROUP>, smem, done);
  if (e != cudaSuccess) return e;
  return launch_attention(decode_mma8_kernel<D, GROUP>, tab.n_workers, D8_THREADS, smem, st, overlap_prev, tab, d,
                          partials);
}
}  // namespace

cudaError_t launch_decode_mma8(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st,
                               bool overlap_prev) {
  if (d.D == 128) {
    if (d.group == 32) return launch_mma8<128, 32>(tab, d, partials, st, overlap_prev);
    if (d.group == 64) return launch_mma8<128, 64>(tab, d, partials, st, overlap_prev);
    return launch_mma8<128, 128>(tab, d, partials, st, overlap_prev);
  }
  if (d.group == 32) return launch_mma8<64, 32>(tab, d, partials, st, overlap_prev);
  return launch_mma8<64, 64>(tab, d, partials, st, overlap_prev);
}

}  // namespace qp
