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
#ifndef QP_D8_MINB
#define QP_D8_MINB 2
#endif
constexpr int D8_MINB = QP_D8_MINB;
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

  const int tid = threadIdx.x, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);       // provably warp-uniform
  const int G = dm.Hq / dm.Hkv, BH = dm.Bt * dm.Hkv;
  // every warp is a worker of its own (see the 4-bit kernel): contiguous tile range, private copy ring
  const int wk = blockIdx.x * D8_WARPS + warp;
  if (wk >= tab.n_workers) return;
  const SkOwner sk{tab.total_tiles, tab.n_workers};
  const long long f0 = sk.start(wk);
  const int total = (int)(sk.start(wk + 1) - f0);
  if (total <= 0) return;

  const uint32_t wsm_u = smem_u32(smem + warp * (D8_STAGES * TL::BYTES + SP8_BYTES));
  const uint32_t sP = wsm_u + D8_STAGES * TL::BYTES;

  // destinations of the asynchronous copies: key piece pi = lane + 32i is channel pi/2, token half pi&1; value
  // piece pi is token pi/NQ, channels 16(pi%NQ) ..
  uint32_t kdst[D / 16], vdst[D / 16];
#pragma unroll
  for (int i = 0; i < D / 16; ++i) {
    const int pi = lane + 32 * i, c = pi >> 1, hf = pi & 1;
    kdst[i] = TL::KC + hf * 16 * D + ((c ^ ((c / (D / 4)) << 1)) << 4);
    const int tau = pi / NQ, q = pi % NQ;
    const int sw = NQ == 8 ? (tau & 7) : ((tau >> 1) & 3);
    vdst[i] = TL::VC + tau * D + ((q ^ sw) << 4);
  }
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

  // copy cursor (p_*) and compute cursor (c_*)
  int p_li = 0;
  while (p_li + 1 < tab.n_layers && (long long)tab.l[p_li + 1].tile_base <= f0) ++p_li;
  int p_tph = tab.l[p_li].n >> 5;
  int p_bh = (int)(f0 - tab.l[p_li].tile_base) / p_tph, p_tile = (int)(f0 - tab.l[p_li].tile_base) % p_tph;
  int c_li = p_li, c_bh = p_bh, c_tile = p_tile, c_tph = p_tph;

  const unsigned char *gKc, *gKm, *gVc, *gVm;                   // per-lane sources of the tile under the copy cursor
  auto set_head = [&]() {
    const DecLayer& ly = tab.l[p_li];
    const size_t n = (size_t)ly.ns, bh = (size_t)p_bh;   // head stride: the arrays' capacity
    const int u = p_tile / GT, sub = p_tile % GT;
    // (a key group of GROUP tokens is GROUP bytes per channel: a tile's 32 tokens are 32 of them, two pieces)
    gKc = static_cast<const unsigned char*>(ly.kc) + bh * n * D + (size_t)u * D * GROUP + sub * 32 +
          (lane >> 1) * GROUP + (lane & 1) * 16;
    gVc = static_cast<const unsigned char*>(ly.vc) + bh * n * D + (size_t)p_tile * 32 * D + lane * 16;
    gKm = reinterpret_cast<const unsigned char*>(lane < MCH ? ly.ks : ly.kz) + (bh * (n / GROUP) + u) * D * 2 + mj * 16;
    gVm = reinterpret_cast<const unsigned char*>(lane < MCH ? ly.vs : ly.vz) + (bh * n + (size_t)p_tile * 32) * NG * 2 +
          mj * 16;
  };
  set_head();
  auto issue_tile = [&](uint32_t sb) {
#pragma unroll
    for (int i = 0; i < D / 16; ++i) {
      cp_async16(sb + kdst[i], gKc + i * 16 * GROUP);
      cp_async16(sb + vdst[i], gVc + i * 512);
    }
    if (2 * MCH == 32 || lane < 2 * MCH) {
      cp_async16(sb + ksz_dst, gKm);
      if (NG == 4 || mj < 4 * NG) cp_async16(sb + vsz_dst, gVm);
    }
    if (++p_tile == p_tph) {
      p_tile = 0;
      if (++p_bh == BH) {
        p_bh = 0;
        if (++p_li < tab.n_layers) p_tph = tab.l[p_li].n >> 5;
      }
      if (p_li < tab.n_layers) set_head();
    } else {
      gVc += 32 * D;
      gVm += 64 * NG;
      if (GT == 1 || p_tile % GT == 0) {
        gKc += D * GROUP - (GT - 1) * 32;
        gKm += D * 2;
      } else {
        gKc += 32;
      }
    }
  };
#pragma unroll
  for (int s = 0; s < D8_STAGES - 1; ++s) {
    if (s < total) issue_tile(wsm_u + s * TL::BYTES);
    cp_async_commit();
  }
  uint32_t sb = wsm_u, sb_copy = wsm_u + (D8_STAGES - 1) * TL::BYTES;

  uint32_t qh2[NPAIR];
  float m_run[2], accO[NQ][4], accPZ[4];
  auto clear_state = [&]() {
    m_run[0] = m_run[1] = -INFINITY;
#pragma unroll
    for (int x = 0; x < 4; ++x) accPZ[x] = 0.f;
#pragma unroll
    for (int q = 0; q < NQ; ++q)
#pragma unroll
      for (int x = 0; x < 4; ++x) accO[q][x] = 0.f;
  };
  clear_state();
  bool fresh = true;
  const int gate = gate_tile(total);

  for (int it = 0; it < total; ++it) {
    if (it == gate) pdl_gate();                                 // see qp_mma.cuh
    if (fresh) {
      fresh = false;
      const DecLayer& ly = tab.l[c_li];
      const int b = c_bh / dm.Hkv, hk = c_bh % dm.Hkv;
      const float scale_log2 = 1.4426950408889634f * rsqrtf((float)D);
      const uint16_t* qp = static_cast<const uint16_t*>(ly.q) + ((size_t)(b * dm.Hq + hk * G + g)) * D + (D / 4) * t;
#pragma unroll
      for (int i = 0; i < NPAIR; i += 4) {
        uint4 w4 = make_uint4(0u, 0u, 0u, 0u);
        if (g < G) w4 = *reinterpret_cast<const uint4*>(qp + 2 * i);
        qh2[i + 0] = pack_half2(bf16lo(w4.x) * scale_log2, bf16hi(w4.x) * scale_log2);
        qh2[i + 2] = pack_half2(bf16lo(w4.y) * scale_log2, bf16hi(w4.y) * scale_log2);   // order (0, 2, 1, 3): see
        qh2[i + 1] = pack_half2(bf16lo(w4.z) * scale_log2, bf16hi(w4.z) * scale_log2);   // the zero-point MMAs
        qh2[i + 3] = pack_half2(bf16lo(w4.w) * scale_log2, bf16hi(w4.w) * scale_log2);
      }
    }

    {
      __syncwarp();
      if (it + D8_STAGES - 1 < total) issue_tile(sb_copy);
      cp_async_commit();
      cp_async_wait<D8_STAGES - 1>();
      __syncwarp();

      // ---------------- keys: m-tile hf holds tokens 16hf + 2g (rows g) and 16hf + 2g + 1 (rows g+8)
      // zero-point term with swapped roles (A = query pairs as they sit in registers, B = zero-point pairs as
      // loaded; rows g of the first, rows g+8 of the second MMA are read), as in the 4-bit kernel
      float accK[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
      float accK2[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};   // second k-step of a round: a chain of its own
      float accZa[4] = {0.f, 0.f, 0.f, 0.f}, accZb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c2 = 0; c2 < NQ / 2; ++c2) {                     // two k-steps (8 channels of this lane) per round
        const uint4 s4 = lds128(sb + TL::KS + ksz_off8((D / 4) * t + 8 * c2));
        const uint4 z4 = lds128(sb + TL::KZ + ksz_off8((D / 4) * t + 8 * c2));
        // qh2[4 c2 + (0, 1, 2, 3)] hold the channel pairs (0, 2, 1, 3) of these eight channels
        const uint32_t b00 = hmul2_u32(qh2[4 * c2 + 0], s4.x), b01 = hmul2_u32(qh2[4 * c2 + 2], s4.y);
        const uint32_t b10 = hmul2_u32(qh2[4 * c2 + 1], s4.z), b11 = hmul2_u32(qh2[4 * c2 + 3], s4.w);
        uint32_t R0, R1, R2, R3;
        ldmatrix_x4_trans(R0, R1, R2, R3, sb + k_plane + ((k_slot0 ^ (8 * c2)) << 4));
        mma_f16_m16n8k16(accK[0], R0 & M8, odd_bytes(R0), R1 & M8, odd_bytes(R1), b00, b01);
        mma_f16_m16n8k16(accK[1], R2 & M8, odd_bytes(R2), R3 & M8, odd_bytes(R3), b00, b01);
        mma_f16_m16n8k16(accZa, qh2[4 * c2 + 0], qh2[4 * c2 + 1], qh2[4 * c2 + 2], qh2[4 * c2 + 3], z4.x, z4.y);
        ldmatrix_x4_trans(R0, R1, R2, R3, sb + k_plane + ((k_slot0 ^ (8 * c2 + 4)) << 4));
        mma_f16_m16n8k16(accK2[0], R0 & M8, odd_bytes(R0), R1 & M8, odd_bytes(R1), b10, b11);
        mma_f16_m16n8k16(accK2[1], R2 & M8, odd_bytes(R2), R3 & M8, odd_bytes(R3), b10, b11);
        mma_f16_m16n8k16(accZb, qh2[4 * c2 + 0], qh2[4 * c2 + 1], qh2[4 * c2 + 2], qh2[4 * c2 + 3], z4.z, z4.w);
      }
#pragma unroll
      for (int hf = 0; hf < 2; ++hf)
#pragma unroll
        for (int x = 0; x < 4; ++x) accK[hf][x] += accK2[hf][x];
      const float zq = accZa[0] + accZb[2];                     // of head g; this lane needs columns 2t, 2t+1
      const float zq_e[2] = {__shfl_sync(0xffffffffu, zq, 8 * t), __shfl_sync(0xffffffffu, zq, 8 * t + 4)};

      // ---------------- running softmax (log2 domain), reference renewed lazily as in the 4-bit kernel
      //   lg[j][x]: tokens {2g, 2g+1, 16+2g, 17+2g}[j], column 2t + x, minus the column's reference
      constexpr float kSlack = 4.f;
      float lg[4][2];
#pragma unroll
      for (int x = 0; x < 2; ++x) {
        const float zm = zq_e[x] - m_run[x];                    // +inf on the first tile of a head
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          lg[2 * hf][x] = fmaf(accK[hf][x], C24, zm);
          lg[2 * hf + 1][x] = fmaf(accK[hf][2 + x], C24, zm);
        }
      }
      const float over = fmaxf(fmaxf(fmaxf(lg[0][0], lg[1][0]), fmaxf(lg[2][0], lg[3][0])),
                               fmaxf(fmaxf(lg[0][1], lg[1][1]), fmaxf(lg[2][1], lg[3][1])));
      if (__any_sync(0xffffffffu, over > kSlack)) {             // rare: renew the references, rescale
        float corr[2];
#pragma unroll
        for (int x = 0; x < 2; ++x) {
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            lg[2 * hf][x] = fmaf(accK[hf][x], C24, zq_e[x]);
            lg[2 * hf + 1][x] = fmaf(accK[hf][2 + x], C24, zq_e[x]);
          }
          float mx = fmaxf(fmaxf(lg[0][x], lg[1][x]), fmaxf(lg[2][x], lg[3][x]));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
          const float mnew = fmaxf(m_run[x], mx);
          corr[x] = ex2(m_run[x] - mnew);
          m_run[x] = mnew;
#pragma unroll
          for (int j = 0; j < 4; ++j) lg[j][x] -= mnew;
        }
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
          accO[q][0] *= corr[0]; accO[q][1] *= corr[1];
          accO[q][2] *= corr[0]; accO[q][3] *= corr[1];
        }
        accPZ[0] *= corr[0]; accPZ[1] *= corr[1];
      }
#pragma unroll
      for (int x = 0; x < 2; ++x)
#pragma unroll
        for (int j = 0; j < 4; ++j) lg[j][x] = ex2(lg[j][x]);    // p; its sum over the tokens: row NG of accPZ

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

      // ---------------- values; zero-point MMA: row g < NG = zero points of scale group g, row NG = ones
      uint32_t ps[4][NG], zp[4];                                // ps[pair][scale group]
#pragma unroll
      for (int pr = 0; pr < 4; ++pr) {
        const int a = 8 * pr + 2 * t;
        zp[pr] = g == NG ? 0x3c003c00u : 0u;
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
      sb_copy = sb;
      sb = sb + TL::BYTES == sP ? wsm_u : sb + TL::BYTES;
    }

    // ---------------- end of this head's part of the range: one partial record per query head, from registers
    if (++c_tile == c_tph || it == total - 1) {
      const float l0 = __shfl_sync(0xffffffffu, accPZ[0], 4 * NG + t), l1 = __shfl_sync(0xffffffffu, accPZ[1], 4 * NG + t);
      const size_t slot = (size_t)c_li * BH + c_bh + wk;
      float* r0 = partials + (slot * G + 2 * t) * (size_t)(D + 2);      // record of column 2t; column 2t+1 follows
      float* r1 = r0 + (D + 2);
      const bool h0 = 2 * t < G, h1 = 2 * t + 1 < G;
#pragma unroll
      for (int q = 0; q < NQ; ++q) {
        const int v = q * NG / NQ;                              // scale group of channels 16q ..
        const float pz0 = __shfl_sync(0xffffffffu, accPZ[0], 4 * v + t);
        const float pz1 = __shfl_sync(0xffffffffu, accPZ[1], 4 * v + t);
        const int ch = 16 * q + 2 * g;
        if (h0) *reinterpret_cast<float2*>(r0 + 2 + ch) = make_float2(fmaf(accO[q][0], C24, pz0), fmaf(accO[q][2], C24, pz0));
        if (h1) *reinterpret_cast<float2*>(r1 + 2 + ch) = make_float2(fmaf(accO[q][1], C24, pz1), fmaf(accO[q][3], C24, pz1));
      }
      if (g == 0) {
        if (h0) *reinterpret_cast<float2*>(r0) = make_float2(m_run[0], l0);
        if (h1) *reinterpret_cast<float2*>(r1) = make_float2(m_run[1], l1);
      }
      clear_state();
      c_tile = 0;
      fresh = true;
      if (++c_bh == BH) {
        c_bh = 0;
        if (++c_li < tab.n_layers) c_tph = tab.l[c_li].n >> 5;
      }
    }
  }
}

template <int D>
constexpr size_t mma8_smem_bytes() { return (size_t)D8_WARPS * (D8_STAGES * Tile8<D>::BYTES + SP8_BYTES); }

}  // namespace

int decode_mma8_blocks_per_sm() { return D8_MINB; }
int decode_mma8_warps() { return D8_WARPS; }

namespace {
template <int D, int GROUP>
cudaError_t launch_mma8(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st, bool overlap_prev) {
  constexpr size_t smem = mma8_smem_bytes<D>();
  static unsigned char done[64] = {};
  const cudaError_t e = allow_smem(decode_mma8_kernel<D, GROUP>, smem, done);
  if (e != cudaSuccess) return e;
  return launch_attention(decode_mma8_kernel<D, GROUP>, (tab.n_workers + D8_WARPS - 1) / D8_WARPS, D8_THREADS, smem, st,
                          overlap_prev, tab, d, partials);
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
