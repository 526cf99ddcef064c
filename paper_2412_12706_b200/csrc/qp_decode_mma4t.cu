// S4 on tensor cores for 4-bit caches whose KEYS are quantized token by token like the values (the FlexGen
// arrangement of Sec. 5.3, also what the head-level budgets use): k_codes [n, D/g, wpg], k_scale, k_zero [n, D/g].
//
// Same decomposition, copy ring, softmax bookkeeping and value side as the per-channel kernel (qp_decode_mma.cu);
// only the key side differs.  With the codes of a token lying along the channels, a 16-byte piece of a key row is 32
// channels of one token, and a plain (non-transposing) ldmatrix hands lane (g, t) the word with channels 8t..8t+7 of
// token g (+8, +16, +24 for the other three matrices).  The eight 4-bit codes of that word become MMA operands by
// masking alone (a 16-bit lane holding a small integer c is the f16 number c * 2^-24):
//     word & 0x000f000f        -> channels (8t+0, 8t+4)          word & 0x00f000f0        -> (8t+1, 8t+5) x 16
//     (word >> 8) & 0x000f000f -> channels (8t+2, 8t+6)          (word >> 8) & 0x00f000f0 -> (8t+3, 8t+7) x 16
// so two MMAs (k = 16 each) cover the 32 channels of a piece: the contraction index is just a permutation of the
// channels, which the query operand follows (and which also carries the factors 1/16).
// The scale of a key group depends on the token (the MMA's row) and on the channel group, so it cannot be folded
// into the query operand: every 32-channel piece accumulates on its own and is scaled afterwards in fp32,
//     logit[tok][h] = sum_pieces s[tok][group] * (sum_d code * q'[h][d]) + z[tok][group] * (sum_d q'[h][d]).
#include <algorithm>

#include "qp_mma.cuh"

namespace qp {

namespace {

constexpr int DT_WARPS = 4;
constexpr int DT_THREADS = DT_WARPS * 32;
constexpr int DT_STAGES = 3, DT_MINB = 3;
constexpr int SPT_STRIDE = 80;           // bytes per column of the per-warp P buffer (8 columns x 32 tokens f16 + pad)
constexpr int SPT_BYTES = 8 * SPT_STRIDE;

// byte offsets of one 32-token tile in shared memory (both code areas: 32 token rows of D/2 bytes)
template <int D>
struct Tile4T {
  static constexpr int KC = 0;
  static constexpr int KS = KC + 16 * D;          // 32 x (D/32) halves at most (g = 32)
  static constexpr int KZ = KS + 2 * D;
  static constexpr int VC = KZ + 2 * D;
  static constexpr int VS = VC + 16 * D;
  static constexpr int VZ = VS + 2 * D;
  static constexpr int BYTES = VZ + 2 * D;
};

constexpr uint32_t M0 = 0x000f000fu, M1 = 0x00f000f0u;
constexpr float C24 = 16777216.0f, C20 = 1048576.0f;

template <int D, int GROUP>
__global__ void __launch_bounds__(DT_THREADS, DT_MINB)
decode_mma4t_kernel(const __grid_constant__ DecTable tab, const DecDims dm, float* __restrict__ partials) {
  using TL = Tile4T<D>;
  constexpr int NC = D / 32;       // 32-channel pieces of a row
  constexpr int NG = D / GROUP;    // scale groups per token (keys and values alike)
  extern __shared__ __align__(128) unsigned char smem[];

  const int tid = threadIdx.x, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  const int G = dm.Hq / dm.Hkv, BH = dm.Bt * dm.Hkv;
  const int wk = blockIdx.x * DT_WARPS + warp;
  if (wk >= tab.n_workers) return;
  const SkOwner sk{tab.total_tiles, tab.n_workers};
  const long long f0 = sk.start(wk);
  const int total = (int)(sk.start(wk + 1) - f0);
  if (total <= 0) return;

  const uint32_t wsm_u = smem_u32(smem + warp * (DT_STAGES * TL::BYTES + SPT_BYTES));
  const uint32_t sP = wsm_u + DT_STAGES * TL::BYTES;

  // a 16-byte piece (token tau, 32 channels v) of either code area sits at tau * D/2 + ((v ^ sw(tau)) << 4): conflict-free
  // for the row-wise loads of the key side and for the transposing loads of the value side
  auto piece_off = [](int tau, int v) {
    const int sw = NC == 4 ? (tau >> 1) & 3 : (tau >> 2) & 1;
    return tau * (D / 2) + ((v ^ sw) << 4);
  };
  uint32_t cdst[D / 32], kr_off[NC], v_off[NC];
#pragma unroll
  for (int i = 0; i < D / 32; ++i) {
    const int c = lane + 32 * i;                                // 16-byte piece of the 32 x D/2 byte code block
    cdst[i] = piece_off(c / NC, c % NC);
  }
  {
    const int tau = 8 * (lane >> 3) + (lane & 7);               // matrix m = lane >> 3 holds tokens 8m .. 8m+7
#pragma unroll
    for (int v = 0; v < NC; ++v) {
      kr_off[v] = TL::KC + piece_off(tau, v);
      v_off[v] = TL::VC + piece_off(tau, v);
    }
  }
  constexpr int MP = 4 * NG;                                    // 16-byte pieces of a tile's scale (or zero) array
  const int arr = lane / MP, mj = lane % MP;                    // lanes < 2 MP: array (0 scale, 1 zero) and piece

  int p_li = 0;
  while (p_li + 1 < tab.n_layers && (long long)tab.l[p_li + 1].tile_base <= f0) ++p_li;
  int p_tph = tab.l[p_li].n >> 5;
  int p_bh = (int)(f0 - tab.l[p_li].tile_base) / p_tph, p_tile = (int)(f0 - tab.l[p_li].tile_base) % p_tph;
  int c_li = p_li, c_bh = p_bh, c_tile = p_tile, c_tph = p_tph;

  const unsigned char *gKc, *gVc, *gKm, *gVm;
  const uint32_t km_dst = (arr == 0 ? TL::KS : TL::KZ) + mj * 16, vm_dst = (arr == 0 ? TL::VS : TL::VZ) + mj * 16;
  auto set_head = [&]() {
    const DecLayer& ly = tab.l[p_li];
    const size_t row0 = (size_t)p_bh * ly.ns + (size_t)p_tile * 32;      // first token row of the tile
    gKc = static_cast<const unsigned char*>(ly.kc) + row0 * (D / 2) + lane * 16;
    gVc = static_cast<const unsigned char*>(ly.vc) + row0 * (D / 2) + lane * 16;
    gKm = reinterpret_cast<const unsigned char*>(arr == 0 ? ly.ks : ly.kz) + row0 * NG * 2 + mj * 16;
    gVm = reinterpret_cast<const unsigned char*>(arr == 0 ? ly.vs : ly.vz) + row0 * NG * 2 + mj * 16;
  };
  set_head();
  auto issue_tile = [&](uint32_t sb) {
#pragma unroll
    for (int i = 0; i < D / 32; ++i) {
      cp_async16(sb + TL::KC + cdst[i], gKc + i * 512);
      cp_async16(sb + TL::VC + cdst[i], gVc + i * 512);
    }
    if (2 * MP == 32 || lane < 2 * MP) {
      cp_async16(sb + km_dst, gKm);
      cp_async16(sb + vm_dst, gVm);
    }
    if (++p_tile == p_tph) {
      p_tile = 0;
      if (++p_bh == BH) {
        p_bh = 0;
        if (++p_li < tab.n_layers) p_tph = tab.l[p_li].n >> 5;
      }
      if (p_li < tab.n_layers) set_head();
    } else {
      gKc += 16 * D;
      gVc += 16 * D;
      gKm += 64 * NG;
      gVm += 64 * NG;
    }
  };
#pragma unroll
  for (int s = 0; s < DT_STAGES - 1; ++s) {
    if (s < total) issue_tile(wsm_u + s * TL::BYTES);
    cp_async_commit();
  }
  uint32_t sb = wsm_u, sb_copy = wsm_u + (DT_STAGES - 1) * TL::BYTES;

  // query operands of the key MMAs, per 32-channel piece: (q0,q4), (q1,q5)/16, (q2,q6), (q3,q7)/16 of this lane's eight
  // channels 32v + 8t .. of head g; and the piece sums of q' for this lane's two columns (heads 2t, 2t+1)
  uint32_t qb[NC][4];
  float qsum[NC][2];
  float m_run[2], accO[NC][2][4], accPZ[4];
  auto clear_state = [&]() {
    m_run[0] = m_run[1] = -INFINITY;
#pragma unroll
    for (int e = 0; e < 4; ++e) accPZ[e] = 0.f;
#pragma unroll
    for (int v = 0; v < NC; ++v)
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int e = 0; e < 4; ++e) accO[v][mt][e] = 0.f;
  };
  clear_state();
  bool fresh = true;
  const int gate = gate_tile(total);

  for (int it = 0; it < total; ++it) {
    if (it == gate) pdl_gate();
    if (fresh) {
      fresh = false;
      const DecLayer& ly = tab.l[c_li];
      const int b = c_bh / dm.Hkv, hk = c_bh % dm.Hkv;
      const float scale_log2 = 1.4426950408889634f * rsqrtf((float)D);
      const uint16_t* qp = static_cast<const uint16_t*>(ly.q) + ((size_t)(b * dm.Hq + hk * G + g)) * D + 8 * t;
#pragma unroll
      for (int v = 0; v < NC; ++v) {
        uint4 w4 = make_uint4(0u, 0u, 0u, 0u);
        if (g < G) w4 = *reinterpret_cast<const uint4*>(qp + 32 * v);
        const float q0 = bf16lo(w4.x) * scale_log2, q1 = bf16hi(w4.x) * scale_log2, q2 = bf16lo(w4.y) * scale_log2,
                    q3 = bf16hi(w4.y) * scale_log2, q4 = bf16lo(w4.z) * scale_log2, q5 = bf16hi(w4.z) * scale_log2,
                    q6 = bf16lo(w4.w) * scale_log2, q7 = bf16hi(w4.w) * scale_log2;
        qb[v][0] = pack_half2(q0, q4);
        qb[v][1] = pack_half2(q1 * 0.0625f, q5 * 0.0625f);
        qb[v][2] = pack_half2(q2, q6);
        qb[v][3] = pack_half2(q3 * 0.0625f, q7 * 0.0625f);
        // piece sum of the f16-rounded q' of head g (what the MMA really multiplies), over the four lanes t
        const __half2 h0 = *reinterpret_cast<const __half2*>(&qb[v][0]), h2 = *reinterpret_cast<const __half2*>(&qb[v][2]);
        float sq = __low2float(h0) + __high2float(h0) + __low2float(h2) + __high2float(h2) +
                   16.f * (__low2float(*reinterpret_cast<const __half2*>(&qb[v][1])) +
                           __high2float(*reinterpret_cast<const __half2*>(&qb[v][1])) +
                           __low2float(*reinterpret_cast<const __half2*>(&qb[v][3])) +
                           __high2float(*reinterpret_cast<const __half2*>(&qb[v][3])));
        sq += __shfl_xor_sync(0xffffffffu, sq, 1);
        sq += __shfl_xor_sync(0xffffffffu, sq, 2);               // every lane (g, *) now has the sum of head g
        qsum[v][0] = __shfl_sync(0xffffffffu, sq, 8 * t);       // head 2t sits in lanes (2t, *)
        qsum[v][1] = __shfl_sync(0xffffffffu, sq, 8 * t + 4);
      }
    }

    __syncwarp();
    if (it + DT_STAGES - 1 < total) issue_tile(sb_copy);
    cp_async_commit();
    cp_async_wait<DT_STAGES - 1>();
    __syncwarp();

    // ---------------- keys: this lane ends up with tokens g, g+8, g+16, g+24 and columns 2t, 2t+1
    //   lg[j][e]: logit of token g + 8j, head 2t + e (log2 domain)
    float lg[4][2] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};
    __half ksh[4][NG], kzh[4][NG];                              // scale and zero of this lane's four tokens
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t so = sb + TL::KS + (g + 8 * j) * NG * 2, zo = sb + TL::KZ + (g + 8 * j) * NG * 2;
      if constexpr (NG == 4) {
        const uint2 a = lds64(so), b = lds64(zo);
        *reinterpret_cast<uint2*>(ksh[j]) = a;
        *reinterpret_cast<uint2*>(kzh[j]) = b;
      } else if constexpr (NG == 2) {
        *reinterpret_cast<uint32_t*>(ksh[j]) = lds32(so);
        *reinterpret_cast<uint32_t*>(kzh[j]) = lds32(zo);
      } else {
        unsigned short a, b;
        asm volatile("ld.shared.u16 %0, [%1];\n" : "=h"(a) : "r"(so));
        asm volatile("ld.shared.u16 %0, [%1];\n" : "=h"(b) : "r"(zo));
        ksh[j][0] = *reinterpret_cast<const __half*>(&a);
        kzh[j][0] = *reinterpret_cast<const __half*>(&b);
      }
    }
#pragma unroll
    for (int v = 0; v < NC; ++v) {
      uint32_t R0, R1, R2, R3;                                  // tokens g, g+8, g+16, g+24: channels 32v + 8t ..
      ldmatrix_x4(R0, R1, R2, R3, sb + kr_off[v]);
      float a0[4] = {0.f, 0.f, 0.f, 0.f}, a1[4] = {0.f, 0.f, 0.f, 0.f};
      mma_f16_m16n8k16(a0, R0 & M0, R1 & M0, R0 & M1, R1 & M1, qb[v][0], qb[v][1]);
      mma_f16_m16n8k16(a1, R2 & M0, R3 & M0, R2 & M1, R3 & M1, qb[v][0], qb[v][1]);
      const uint32_t S0 = R0 >> 8, S1 = R1 >> 8, S2 = R2 >> 8, S3 = R3 >> 8;
      mma_f16_m16n8k16(a0, S0 & M0, S1 & M0, S0 & M1, S1 & M1, qb[v][2], qb[v][3]);
      mma_f16_m16n8k16(a1, S2 & M0, S3 & M0, S2 & M1, S3 & M1, qb[v][2], qb[v][3]);
      // a0: rows g, g+8 of tokens 0..15; a1: the same of tokens 16..31
      const int grp = v * NG / NC;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float sc = __half2float(ksh[j][grp]), zr = __half2float(kzh[j][grp]);
        const float c0 = (j < 2 ? a0 : a1)[2 * (j & 1)], c1 = (j < 2 ? a0 : a1)[2 * (j & 1) + 1];
        lg[j][0] = fmaf(sc * C24, c0, fmaf(zr, qsum[v][0], lg[j][0]));
        lg[j][1] = fmaf(sc * C24, c1, fmaf(zr, qsum[v][1], lg[j][1]));
      }
    }

    // ---------------- running softmax (log2 domain); the reference is renewed only when a logit exceeds it by
    // more than kSlack (see the per-channel kernel)
    constexpr float kSlack = 4.f;
    float over = -INFINITY;
#pragma unroll
    for (int j = 0; j < 4; ++j) over = fmaxf(over, fmaxf(lg[j][0] - m_run[0], lg[j][1] - m_run[1]));
    if (__any_sync(0xffffffffu, over > kSlack)) {
      float corr[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        float mx = fmaxf(fmaxf(lg[0][e], lg[1][e]), fmaxf(lg[2][e], lg[3][e]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
        const float mnew = fmaxf(m_run[e], mx);
        corr[e] = ex2(m_run[e] - mnew);
        m_run[e] = mnew;
      }
#pragma unroll
      for (int v = 0; v < NC; ++v)
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          accO[v][mt][0] *= corr[0]; accO[v][mt][1] *= corr[1];
          accO[v][mt][2] *= corr[0]; accO[v][mt][3] *= corr[1];
        }
      accPZ[0] *= corr[0]; accPZ[1] *= corr[1];
    }
#pragma unroll
    for (int e = 0; e < 2; ++e)
#pragma unroll
      for (int j = 0; j < 4; ++j) lg[j][e] = ex2(lg[j][e] - m_run[e]);

    // ---------------- P through shared memory: [column][token] f16 (this lane's tokens are 8 apart)
#pragma unroll
    for (int e = 0; e < 2; ++e)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const __half hv = __float2half_rn(lg[j][e]);
        asm volatile("st.shared.u16 [%0], %1;\n" ::"r"(sP + (2 * t + e) * SPT_STRIDE + (g + 8 * j) * 2),
                     "h"(*reinterpret_cast<const unsigned short*>(&hv)));
      }
    __syncwarp();
    uint32_t p2[4];                                             // tokens (2t, 2t+1) + {0, 8, 16, 24} of column g
#pragma unroll
    for (int pr = 0; pr < 4; ++pr) p2[pr] = lds32(sP + g * SPT_STRIDE + 4 * t + 16 * pr);

    // ---------------- values: exactly the per-channel kernel's value side
    uint32_t ps[4][NG], zp[4];
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
      } else {
        ps[pr][0] = hmul2_u32(p2[pr], lds32(sb + TL::VS + a * 2));
        if (g == 0) zp[pr] = lds32(sb + TL::VZ + a * 2);
      }
    }
    mma_f16_m16n8k16(accPZ, zp[0], 0u, zp[1], 0u, p2[0], p2[1]);
    mma_f16_m16n8k16(accPZ, zp[2], 0u, zp[3], 0u, p2[2], p2[3]);
#pragma unroll
    for (int v = 0; v < NC; ++v) {
      uint32_t R0, R1, R2, R3;
      ldmatrix_x4_trans(R0, R1, R2, R3, sb + v_off[v]);
      mma_f16_m16n8k16(accO[v][0], R0 & M0, R0 & M1, R1 & M0, R1 & M1, ps[0][v * NG / NC], ps[1][v * NG / NC]);
      const uint32_t S0 = R0 >> 8, S1 = R1 >> 8;
      mma_f16_m16n8k16(accO[v][1], S0 & M0, S0 & M1, S1 & M0, S1 & M1, ps[0][v * NG / NC], ps[1][v * NG / NC]);
      mma_f16_m16n8k16(accO[v][0], R2 & M0, R2 & M1, R3 & M0, R3 & M1, ps[2][v * NG / NC], ps[3][v * NG / NC]);
      const uint32_t S2 = R2 >> 8, S3 = R3 >> 8;
      mma_f16_m16n8k16(accO[v][1], S2 & M0, S2 & M1, S3 & M0, S3 & M1, ps[2][v * NG / NC], ps[3][v * NG / NC]);
    }
    sb_copy = sb;
    sb = sb + TL::BYTES == sP ? wsm_u : sb + TL::BYTES;

    // ---------------- end of this head's part of the range: one partial record per query head
    if (++c_tile == c_tph || it == total - 1) {
      const float l0 = __shfl_sync(0xffffffffu, accPZ[0], 4 * NG + t), l1 = __shfl_sync(0xffffffffu, accPZ[1], 4 * NG + t);
      const size_t slot = (size_t)c_li * BH + c_bh + wk;
      float* r0 = partials + (slot * G + 2 * t) * (size_t)(D + 2);
      float* r1 = r0 + (D + 2);
      const bool h0 = 2 * t < G, h1 = 2 * t + 1 < G;
#pragma unroll
      for (int v = 0; v < NC; ++v) {
        const float pz0 = __shfl_sync(0xffffffffu, accPZ[0], 4 * (v * NG / NC) + t);
        const float pz1 = __shfl_sync(0xffffffffu, accPZ[1], 4 * (v * NG / NC) + t);
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          const int ch = 32 * v + 4 * g + 2 * mt;
          if (h0) *reinterpret_cast<float2*>(r0 + 2 + ch) =
                      make_float2(fmaf(accO[v][mt][0], C24, pz0), fmaf(accO[v][mt][2], C20, pz0));
          if (h1) *reinterpret_cast<float2*>(r1 + 2 + ch) =
                      make_float2(fmaf(accO[v][mt][1], C24, pz1), fmaf(accO[v][mt][3], C20, pz1));
        }
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
constexpr size_t mma4t_smem_bytes() { return (size_t)DT_WARPS * (DT_STAGES * Tile4T<D>::BYTES + SPT_BYTES); }

template <int D, int GROUP>
cudaError_t launch_t(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st) {
  constexpr size_t smem = mma4t_smem_bytes<D>();
  static unsigned char done[64] = {};
  const cudaError_t e = allow_smem(decode_mma4t_kernel<D, GROUP>, smem, done);
  if (e != cudaSuccess) return e;
  return launch_attention(decode_mma4t_kernel<D, GROUP>, (tab.n_workers + DT_WARPS - 1) / DT_WARPS, DT_THREADS, smem, st,
                          false, tab, d, partials);
}

}  // namespace

bool decode_mma4t_supported(const DecDims& d) {
  return d.bits == 4 && (d.D == 128 || d.D == 64) && d.D % d.group == 0 && d.Hq / d.Hkv <= 8;
}
int decode_mma4t_workers_per_sm() { return DT_MINB * DT_WARPS; }

// attention kernel only; the caller launches the flat-range merge
cudaError_t launch_decode_mma4t(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st) {
  if (d.D == 128) {
    if (d.group == 32) return launch_t<128, 32>(tab, d, partials, st);
    if (d.group == 64) return launch_t<128, 64>(tab, d, partials, st);
    return launch_t<128, 128>(tab, d, partials, st);
  }
  if (d.group == 32) return launch_t<64, 32>(tab, d, partials, st);
  return launch_t<64, 64>(tab, d, partials, st);
}

}  // namespace qp
