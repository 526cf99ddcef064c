// S4 on tensor cores for 2-bit caches (group 32, at most 4 query heads per KV head).
//
// Same idea as the 4-bit kernel (codes used as f16 subnormals, transposing ldmatrix, scale folded
// into the B operand, flat-range decomposition), with one extra twist forced by the layout: at
// 2 bits a quantisation group of 32 elements is only 8 bytes, but ldmatrix moves 16-byte rows.
// A shared-memory row is therefore built from two 8-byte halves that belong to two different
// problems, and the 8 MMA columns are used as 2 variants x 4 heads:
//   keys    row = [channel c of tile A | channel c of tile B]   (two consecutive 32-token tiles);
//           MMA rows with lane bit e = g>>2 hold tokens of tile e, columns (e', h) hold q'[h] * scale
//           of tile e'; the e = e' blocks are the logits, the other blocks are ignored.
//   values  row = [token, channel group v | token, channel group v + NC/2];
//           MMA rows with bit e hold channels of group v + e*NC/2, columns (e', h) hold
//           p[h] * scale of group v + e'*NC/2; again only e = e' is used.
// A 16-bit unit holds 8 codes; code j sits at bits 2j, and (word & (0x00030003 << 2j)) is an f16
// pair worth c * 4^j * 2^-24 as long as the pattern stays below 2^11 (j <= 4); j = 5..7 use the
// word shifted right by 10.  The powers of two are undone on the f32 accumulators.
// Decomposition, softmax bookkeeping and the zero-point MMAs follow the 4-bit kernel: every warp is a worker of
// its own over a contiguous range of 32-token tiles, which it walks in pairs (the last tile before a head
// boundary or the end of the range may be single).
#include "qp_mma.cuh"

namespace qp {

namespace {

constexpr int D2_WARPS = 4;
constexpr int D2_THREADS = D2_WARPS * 32;
#ifndef QP_D2_STAGES
#define QP_D2_STAGES 2
#endif
#ifndef QP_D2_MINB
#define QP_D2_MINB 3
#endif
constexpr int D2_STAGES = QP_D2_STAGES;
constexpr int SP2_STRIDE = 144;          // bytes per head row of the per-warp P buffer (64 tokens + pad)
constexpr int SP2_BYTES = 4 * SP2_STRIDE;

// byte offsets of one double tile (2 x 32 tokens) in shared memory
template <int D>
struct Tile2 {
  static constexpr int KMETA = 2 * D + 16;        // D halves, channels >= 64 shifted by 16 B
  static constexpr int KC = 0;                    // D rows of 16 B: [tile A channel c | tile B channel c]
  static constexpr int KS0 = KC + 16 * D;         // KS(e) = KS0 + e * 2 * KMETA, KZ(e) = KS(e) + KMETA
  static constexpr int VC = KS0 + 4 * KMETA;      // 64 tokens x NC/2 rows of 16 B
  static constexpr int VS = VC + 16 * D;          // 64 tokens x NC halves
  static constexpr int VZ = VS + 4 * D;
  static constexpr int BYTES = VZ + 4 * D;
};

__host__ __device__ constexpr int ksz_off2(int ch) { return ch * 2 + (ch / 64) * 16; }

__device__ __forceinline__ void cp_async8_zfill(uint32_t saddr, const void* gptr, bool valid) {
  const int n = valid ? 8 : 0;
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;\n" ::"r"(saddr), "l"(gptr), "r"(n));
}
__device__ __forceinline__ void cp_async16_zfill(uint32_t saddr, const void* gptr, bool valid) {
  const int n = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(saddr), "l"(gptr), "r"(n));
}
__device__ __forceinline__ void sts128(uint32_t a, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(a), "r"(x), "r"(y), "r"(z), "r"(w));
}

constexpr uint32_t MJ0 = 0x00030003u, MJ1 = MJ0 << 2, MJ2 = MJ0 << 4, MJ3 = MJ0 << 6, MJ4 = MJ0 << 8;
// accumulator scale of code position j: rows g of m-tile mt use j = 2mt, rows g+8 use j = 2mt+1
__device__ __forceinline__ constexpr float cfac(int j) {
  return j == 0 ? 16777216.f : j == 1 ? 4194304.f : j == 2 ? 1048576.f : j == 3 ? 262144.f : j == 4 ? 65536.f
       : j == 5 ? 16777216.f : j == 6 ? 4194304.f : 1048576.f;
}

// the four m-tiles of one k-step: A registers from the two transposed words, shared B
__device__ __forceinline__ void mma_unit8(float (&acc)[4][4], uint32_t Ra, uint32_t Rb, uint32_t b0, uint32_t b1) {
  mma_f16_m16n8k16(acc[0], Ra & MJ0, Ra & MJ1, Rb & MJ0, Rb & MJ1, b0, b1);
  mma_f16_m16n8k16(acc[1], Ra & MJ2, Ra & MJ3, Rb & MJ2, Rb & MJ3, b0, b1);
  const uint32_t Sa = Ra >> 10, Sb = Rb >> 10;
  mma_f16_m16n8k16(acc[2], Ra & MJ4, Sa & MJ0, Rb & MJ4, Sb & MJ0, b0, b1);
  mma_f16_m16n8k16(acc[3], Sa & MJ1, Sa & MJ2, Sb & MJ1, Sb & MJ2, b0, b1);
}

template <int D>
__global__ void __launch_bounds__(D2_THREADS, QP_D2_MINB)
decode_mma2_kernel(const __grid_constant__ DecTable tab, const DecDims dm, float* __restrict__ partials) {
  using TL = Tile2<D>;
  constexpr int NC = D / 32;       // value groups per token; also ldmatrix.x4 calls over a key tile's channels
  constexpr int NCH = NC / 2;      // value-group pairs (v, v + NCH)
  constexpr int NPAIR = D / 8;     // channel pairs owned by one lane on the key side
  extern __shared__ __align__(128) unsigned char smem[];

  const int tid = threadIdx.x, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);       // provably warp-uniform
  const int e = g >> 2, o = g & 3;                              // variant bit and unit index of this lane's MMA rows
  const bool lane_valid = e == (t >> 1);                        // this lane's accumulator entries are an e = e' block
  const int G = dm.Hq / dm.Hkv, BH = dm.Bt * dm.Hkv;
  const int wk = blockIdx.x * D2_WARPS + warp;
  if (wk >= tab.n_workers) return;
  const SkOwner sk{tab.total_tiles, tab.n_workers};
  const long long f0 = sk.start(wk);
  const int total = (int)(sk.start(wk + 1) - f0);
  if (total <= 0) return;

  const uint32_t wsm_u = smem_u32(smem + warp * (D2_STAGES * TL::BYTES + SP2_BYTES));
  const uint32_t sP = wsm_u + D2_STAGES * TL::BYTES;

  // destinations of the asynchronous copies (8-byte pieces of the codes: tile te of the pair goes to half te of
  // a key row; a value piece (token, group vv) goes to half vv / NCH of row (token, vv % NCH))
  uint32_t kdst[D / 32], vdst[2][D / 32];
#pragma unroll
  for (int i = 0; i < D / 32; ++i) {
    const int c = lane + 32 * i;
    kdst[i] = TL::KC + (c ^ ((c / (D / 4)) << 1)) * 16;
#pragma unroll
    for (int te = 0; te < 2; ++te) {
      const int tau = 32 * te + c / NC, vv = c % NC;
      const int rho = tau * NCH + vv % NCH;
      vdst[te][i] = TL::VC + (NCH == 2 ? rho ^ ((tau >> 2) & 1) : rho) * 16 + (vv / NCH) * 8;
    }
  }
  constexpr int MCH = D / 8;                                    // 16-byte pieces of a key scale or zero array
  constexpr int VCH = D / 4;                                    // 16-byte pieces of the value scales of a pair
  const int k_arr = lane / MCH, k_j = lane % MCH;               // lanes < 2 MCH: array (0 scale, 1 zero) and piece
  const uint32_t kmeta_dst = TL::KS0 + k_arr * TL::KMETA + k_j * 16 + (k_j / 8) * 16;   // + 2 te KMETA

  // sources of the transposing loads
  uint32_t k_off, v_off[NCH];
  {
    const int m = lane >> 3, r = lane & 7, tq = r >> 1, p = r & 1;
    const int ch = (D / 4) * tq + 2 * m + p;                    // + 8 per ldmatrix call
    k_off = TL::KC + ((ch ^ (tq << 1)) << 4);
    const int tau = 8 * m + r;                                  // + 32 for the second tile
#pragma unroll
    for (int v = 0; v < NCH; ++v) {
      const int rho = tau * NCH + v;
      v_off[v] = TL::VC + ((NCH == 2 ? rho ^ ((tau >> 2) & 1) : rho) << 4);
    }
  }

  // copy cursor (p_*) and compute cursor (c_*): both walk the range in the same pairs
  int p_li = 0;
  while (p_li + 1 < tab.n_layers && (long long)tab.l[p_li + 1].tile_base <= f0) ++p_li;
  int p_tph = tab.l[p_li].n >> 5;
  int p_bh = (int)(f0 - tab.l[p_li].tile_base) / p_tph, p_tile = (int)(f0 - tab.l[p_li].tile_base) % p_tph;
  int c_li = p_li, c_bh = p_bh, c_tile = p_tile, c_tph = p_tph;
  int p_left = total, c_left = total;

  const unsigned char *gKc, *gKm, *gVc, *gVs, *gVz;             // per-lane sources of the tile under the copy cursor
  auto set_head = [&]() {
    const DecLayer& ly = tab.l[p_li];
    const size_t n = (size_t)ly.ns, bh = (size_t)p_bh, tile = (size_t)p_tile;   // head stride: capacity
    gKc = static_cast<const unsigned char*>(ly.kc) + bh * n * (D / 4) + tile * D * 8 + lane * 8;
    gVc = static_cast<const unsigned char*>(ly.vc) + bh * n * (D / 4) + tile * 8 * D + lane * 8;
    gKm = reinterpret_cast<const unsigned char*>(k_arr ? ly.kz : ly.ks) + (bh * (n >> 5) + tile) * D * 2 + k_j * 16;
    gVs = reinterpret_cast<const unsigned char*>(ly.vs) + (bh * n + tile * 32) * (D / 16) + lane * 16;
    gVz = reinterpret_cast<const unsigned char*>(ly.vz) + (bh * n + tile * 32) * (D / 16) + lane * 16;
  };
  set_head();
  // stage the pair of tiles under the copy cursor (a missing second tile is zero-filled), advance the cursor
  auto issue_pair = [&](uint32_t sb) {
    const bool two = p_tile + 1 < p_tph && p_left >= 2;
#pragma unroll
    for (int te = 0; te < 2; ++te) {
      const bool ok = te == 0 || two;
      const unsigned char* kc = gKc + (ok ? te : 0) * (D * 8);
      const unsigned char* vc = gVc + (ok ? te : 0) * (8 * D);
#pragma unroll
      for (int i = 0; i < D / 32; ++i) {
        cp_async8_zfill(sb + kdst[i] + te * 8, kc + i * 256, ok);
        cp_async8_zfill(sb + vdst[te][i], vc + i * 256, ok);
      }
      if (2 * MCH == 32 || lane < 2 * MCH)
        cp_async16_zfill(sb + kmeta_dst + 2 * te * TL::KMETA, gKm + (ok ? te : 0) * (D * 2), ok);
    }
    if (VCH == 32 || lane < VCH) {                              // the two tiles' value scales are contiguous
      const bool ok = lane < VCH / 2 || two;
      const int back = ok ? 0 : (VCH / 2) * 16;                 // keep the address inside the array
      cp_async16_zfill(sb + TL::VS + lane * 16, gVs - back, ok);
      cp_async16_zfill(sb + TL::VZ + lane * 16, gVz - back, ok);
    }
    const int adv = two ? 2 : 1;
    p_left -= adv;
    p_tile += adv;
    if (p_tile == p_tph) {
      p_tile = 0;
      if (++p_bh == BH) {
        p_bh = 0;
        if (++p_li < tab.n_layers) p_tph = tab.l[p_li].n >> 5;
      }
      if (p_li < tab.n_layers) set_head();
    } else {
      gKc += adv * (D * 8);
      gVc += adv * (8 * D);
      gKm += adv * (D * 2);
      gVs += adv * (2 * D);
      gVz += adv * (2 * D);
    }
  };
#pragma unroll
  for (int s = 0; s < D2_STAGES - 1; ++s) {
    if (p_left > 0) issue_pair(wsm_u + s * TL::BYTES);
    cp_async_commit();
  }
  uint32_t sb = wsm_u, sb_copy = wsm_u + (D2_STAGES - 1) * TL::BYTES;

  uint32_t qh2[NPAIR];
  // softmax reference of heads 2(t&1), 2(t&1)+1 (identical in all lanes with the same t&1) and accumulators
  float m_run[2], accO[NCH][4][4], accPZ[4];
  auto clear_state = [&]() {
    m_run[0] = m_run[1] = -INFINITY;
#pragma unroll
    for (int x = 0; x < 4; ++x) accPZ[x] = 0.f;
#pragma unroll
    for (int v = 0; v < NCH; ++v)
#pragma unroll
      for (int mt = 0; mt < 4; ++mt)
#pragma unroll
        for (int x = 0; x < 4; ++x) accO[v][mt][x] = 0.f;
  };
  clear_state();
  bool fresh = true, gated = false;

  while (c_left > 0) {
    if (!gated && c_left <= total - gate_tile(total)) {
      gated = true;
      pdl_gate();
    }
    if (fresh) {
      fresh = false;
      const DecLayer& ly = tab.l[c_li];
      const int b = c_bh / dm.Hkv, hk = c_bh % dm.Hkv;
      // query fragments: column g of the MMAs = (variant g>>2, head g&3); both variants carry the same q'
      const float scale_log2 = 1.4426950408889634f * rsqrtf((float)D);
      const uint16_t* qp = static_cast<const uint16_t*>(ly.q) + ((size_t)(b * dm.Hq + hk * G + o)) * D + (D / 4) * t;
#pragma unroll
      for (int i = 0; i < NPAIR; i += 4) {
        uint4 w4 = make_uint4(0u, 0u, 0u, 0u);
        if (o < G) w4 = *reinterpret_cast<const uint4*>(qp + 2 * i);
        qh2[i + 0] = pack_half2(bf16lo(w4.x) * scale_log2, bf16hi(w4.x) * scale_log2);
        qh2[i + 2] = pack_half2(bf16lo(w4.y) * scale_log2, bf16hi(w4.y) * scale_log2);   // order (0, 2, 1, 3): see
        qh2[i + 1] = pack_half2(bf16lo(w4.z) * scale_log2, bf16hi(w4.z) * scale_log2);   // the zero-point MMAs
        qh2[i + 3] = pack_half2(bf16lo(w4.w) * scale_log2, bf16hi(w4.w) * scale_log2);
      }
    }
    const bool two = c_tile + 1 < c_tph && c_left >= 2;         // the same pairing as the copy cursor's
    {
      __syncwarp();
      if (p_left > 0) issue_pair(sb_copy);
      cp_async_commit();
      cp_async_wait<D2_STAGES - 1>();
      __syncwarp();
      const bool tile_present = e == 0 || two;                  // is this lane's tile real?

      // ---------------- keys: rows (e, o) = tokens 8o..8o+7 of tile e; columns (e', h)
      // zero-point term with swapped roles (A = query pairs as they sit in registers, B = zero-point pairs of the
      // tile of this lane's column variant; rows g of the first, rows g+8 of the second MMA are read)
      float accK[4][4], accZa[4] = {0.f, 0.f, 0.f, 0.f}, accZb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int mt = 0; mt < 4; ++mt)
#pragma unroll
        for (int x = 0; x < 4; ++x) accK[mt][x] = 0.f;
      const uint32_t ks_e = sb + TL::KS0 + 2 * e * TL::KMETA, kz_e = ks_e + TL::KMETA;
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const uint4 s4 = lds128(ks_e + ksz_off2((D / 4) * t + 8 * c));
        const uint4 z4 = lds128(kz_e + ksz_off2((D / 4) * t + 8 * c));
        uint32_t R0, R1, R2, R3;
        ldmatrix_x4_trans(R0, R1, R2, R3, sb + k_off + c * 128);
        // qh2[4c + (0, 1, 2, 3)] hold the channel pairs (0, 2, 1, 3) of this lane's eight channels
        mma_unit8(accK, R0, R1, hmul2_u32(qh2[4 * c + 0], s4.x), hmul2_u32(qh2[4 * c + 2], s4.y));
        mma_f16_m16n8k16(accZa, qh2[4 * c + 0], qh2[4 * c + 1], qh2[4 * c + 2], qh2[4 * c + 3], z4.x, z4.y);
        mma_unit8(accK, R2, R3, hmul2_u32(qh2[4 * c + 1], s4.z), hmul2_u32(qh2[4 * c + 3], s4.w));
        mma_f16_m16n8k16(accZb, qh2[4 * c + 0], qh2[4 * c + 1], qh2[4 * c + 2], qh2[4 * c + 3], z4.z, z4.w);
      }
      // lanes (g, t) hold the term of head g&3 and the tile of column variant t>>1; this lane needs heads
      // 2(t&1), 2(t&1)+1 of variant t>>1
      const float zq = accZa[0] + accZb[2];
      const float zq_c[2] = {__shfl_sync(0xffffffffu, zq, 8 * (t & 1) + t),
                             __shfl_sync(0xffffffffu, zq, 8 * (t & 1) + 4 + t)};

      // ---------------- running softmax over the 64 tokens (log2 domain), reference renewed lazily
      //   lg[2mt + rh][c]: token 8o + 2mt + rh of tile e, head 2(t&1) + c, minus the head's reference
      constexpr float kSlack = 4.f;
      const bool use = lane_valid && tile_present;
      float lg[8][2];
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const float zm = zq_c[c] - m_run[c];                    // +inf on the first pair of a head
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
          lg[2 * mt][c] = use ? fmaf(accK[mt][c], cfac(2 * mt), zm) : -INFINITY;
          lg[2 * mt + 1][c] = use ? fmaf(accK[mt][2 + c], cfac(2 * mt + 1), zm) : -INFINITY;
        }
      }
      float over = fmaxf(lg[0][0], lg[0][1]);
#pragma unroll
      for (int j = 1; j < 8; ++j) over = fmaxf(over, fmaxf(lg[j][0], lg[j][1]));
      if (__any_sync(0xffffffffu, over > kSlack)) {             // rare: renew the references, rescale
        float corr[2];
#pragma unroll
        for (int c = 0; c < 2; ++c) {
#pragma unroll
          for (int mt = 0; mt < 4; ++mt) {
            lg[2 * mt][c] = use ? fmaf(accK[mt][c], cfac(2 * mt), zq_c[c]) : -INFINITY;
            lg[2 * mt + 1][c] = use ? fmaf(accK[mt][2 + c], cfac(2 * mt + 1), zq_c[c]) : -INFINITY;
          }
          float mx = lg[0][c];
#pragma unroll
          for (int j = 1; j < 8; ++j) mx = fmaxf(mx, lg[j][c]);
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));    // lanes with the same t&1 share the two heads
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
          const float mnew = fmaxf(m_run[c], mx);
          corr[c] = ex2(m_run[c] - mnew);
          m_run[c] = mnew;
#pragma unroll
          for (int j = 0; j < 8; ++j) lg[j][c] -= mnew;
        }
#pragma unroll
        for (int v = 0; v < NCH; ++v)
#pragma unroll
          for (int mt = 0; mt < 4; ++mt) {
            accO[v][mt][0] *= corr[0]; accO[v][mt][1] *= corr[1];
            accO[v][mt][2] *= corr[0]; accO[v][mt][3] *= corr[1];
          }
        accPZ[0] *= corr[0]; accPZ[1] *= corr[1];
      }
#pragma unroll
      for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int j = 0; j < 8; ++j) lg[j][c] = ex2(lg[j][c]);    // p (0 for entries that are not logits)

      // ---------------- P through shared memory: [head][64 tokens] f16
      if (lane_valid) {
#pragma unroll
        for (int c = 0; c < 2; ++c)
          sts128(sP + (2 * (t & 1) + c) * SP2_STRIDE + (32 * e + 8 * o) * 2,
                 pack_half2(lg[0][c], lg[1][c]), pack_half2(lg[2][c], lg[3][c]),
                 pack_half2(lg[4][c], lg[5][c]), pack_half2(lg[6][c], lg[7][c]));
      }
      __syncwarp();

      // ---------------- values: rows (e, o) = channels 8o..8o+7 of group v + e*NCH; columns (e', h)
      // zero-point MMA: row g < NC = zero points of value group g, row NC = ones (softmax denominators)
#pragma unroll
      for (int kp = 0; kp < 2; ++kp) {                          // 32 tokens = two k-steps per transposed load
        uint32_t p2[2][2], ps[2][2][NCH], zp[2][2];             // [k-step][token-pair half]
#pragma unroll
        for (int kk = 0; kk < 2; ++kk)
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            const int a = 32 * kp + 16 * kk + 8 * hf + 2 * t;   // first token of the pair
            p2[kk][hf] = lds32(sP + o * SP2_STRIDE + a * 2);
            // scales of tokens a, a+1 for the groups of this lane's column variant e
            if constexpr (NC == 4) {
              const uint32_t wa = lds32(sb + TL::VS + a * 8 + 4 * e);
              const uint32_t wb = lds32(sb + TL::VS + a * 8 + 8 + 4 * e);
              ps[kk][hf][0] = hmul2_u32(p2[kk][hf], __byte_perm(wa, wb, 0x5410));
              ps[kk][hf][1] = hmul2_u32(p2[kk][hf], __byte_perm(wa, wb, 0x7632));
            } else {
              const uint2 x = lds64(sb + TL::VS + a * 4);
              ps[kk][hf][0] = hmul2_u32(p2[kk][hf], __byte_perm(x.x, x.y, e ? 0x7632 : 0x5410));
            }
            zp[kk][hf] = g == NC ? 0x3c003c00u : 0u;
            if (g < NC) {
              if constexpr (NC == 4) {
                const uint32_t ya = lds32(sb + TL::VZ + a * 8 + (g & 2) * 2);
                const uint32_t yb = lds32(sb + TL::VZ + a * 8 + 8 + (g & 2) * 2);
                zp[kk][hf] = __byte_perm(ya, yb, (g & 1) ? 0x7632 : 0x5410);
              } else {
                const uint2 y = lds64(sb + TL::VZ + a * 4);
                zp[kk][hf] = __byte_perm(y.x, y.y, (g & 1) ? 0x7632 : 0x5410);
              }
            }
          }
        mma_f16_m16n8k16(accPZ, zp[0][0], 0u, zp[0][1], 0u, p2[0][0], p2[0][1]);
        mma_f16_m16n8k16(accPZ, zp[1][0], 0u, zp[1][1], 0u, p2[1][0], p2[1][1]);
#pragma unroll
        for (int v = 0; v < NCH; ++v) {
          uint32_t R0, R1, R2, R3;                              // tokens 0-7, 8-15, 16-23, 24-31 of this half
          ldmatrix_x4_trans(R0, R1, R2, R3, sb + v_off[v] + kp * (32 * NCH * 16));
          mma_unit8(accO[v], R0, R1, ps[0][0][v], ps[0][1][v]);
          mma_unit8(accO[v], R2, R3, ps[1][0][v], ps[1][1][v]);
        }
      }
      sb_copy = sb;
      sb = sb + TL::BYTES == sP ? wsm_u : sb + TL::BYTES;
    }

    // ---------------- end of this head's part of the range: one partial record per query head, from registers
    const int adv = two ? 2 : 1;
    c_left -= adv;
    c_tile += adv;
    if (c_tile == c_tph || c_left == 0) {
      // softmax denominators of heads 2(t&1), +1: row NC of the zero-point accumulator, columns (0, h)
      const float l0 = __shfl_sync(0xffffffffu, accPZ[0], 4 * NC + (t & 1));
      const float l1 = __shfl_sync(0xffffffffu, accPZ[1], 4 * NC + (t & 1));
      const size_t slot = (size_t)c_li * BH + c_bh + wk;
      const int h0i = 2 * (t & 1);
      float* r0 = partials + (slot * G + h0i) * (size_t)(D + 2);
      float* r1 = r0 + (D + 2);
      const bool h0 = lane_valid && h0i < G, h1 = lane_valid && h0i + 1 < G;
#pragma unroll
      for (int v = 0; v < NCH; ++v) {
        // zero-point term of group vv = v + e*NCH for heads 2(t&1), +1: row vv of accPZ, columns (0, h)
        const int vv = v + e * NCH;
        const float pz0 = __shfl_sync(0xffffffffu, accPZ[0], 4 * vv + (t & 1));
        const float pz1 = __shfl_sync(0xffffffffu, accPZ[1], 4 * vv + (t & 1));
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
          const int ch = 32 * vv + 8 * o + 2 * mt;
          if (h0) *reinterpret_cast<float2*>(r0 + 2 + ch) =
                      make_float2(fmaf(accO[v][mt][0], cfac(2 * mt), pz0), fmaf(accO[v][mt][2], cfac(2 * mt + 1), pz0));
          if (h1) *reinterpret_cast<float2*>(r1 + 2 + ch) =
                      make_float2(fmaf(accO[v][mt][1], cfac(2 * mt), pz1), fmaf(accO[v][mt][3], cfac(2 * mt + 1), pz1));
        }
      }
      if (g == 0 && t < 2) {                                    // lanes (0, 0) and (0, 1): e = 0 = t>>1
        if (h0) *reinterpret_cast<float2*>(r0) = make_float2(m_run[0], l0);
        if (h1) *reinterpret_cast<float2*>(r1) = make_float2(m_run[1], l1);
      }
      clear_state();
      fresh = true;
      if (c_tile == c_tph) {
        c_tile = 0;
        if (++c_bh == BH) {
          c_bh = 0;
          if (++c_li < tab.n_layers) c_tph = tab.l[c_li].n >> 5;
        }
      }
    }
  }
}

template <int D>
constexpr size_t mma2_smem_bytes() { return (size_t)D2_WARPS * (D2_STAGES * Tile2<D>::BYTES + SP2_BYTES); }

}  // namespace

bool decode_mma2_supported(const DecDims& d) {
  return d.bits == 2 && d.group == 32 && (d.D == 128 || d.D == 64) && d.Hq / d.Hkv <= 4;
}
int decode_mma2_workers_per_sm() { return QP_D2_MINB * D2_WARPS; }

cudaError_t launch_decode_mma2(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st,
                               bool overlap_prev) {
  const int blocks = (tab.n_workers + D2_WARPS - 1) / D2_WARPS;
  if (d.D == 128) {
    constexpr size_t smem = mma2_smem_bytes<128>();
    static unsigned char done[64] = {};
    const cudaError_t e = allow_smem(decode_mma2_kernel<128>, smem, done);
    if (e != cudaSuccess) return e;
    return launch_attention(decode_mma2_kernel<128>, blocks, D2_THREADS, smem, st, overlap_prev, tab, d, partials);
  }
  constexpr size_t smem = mma2_smem_bytes<64>();
  static unsigned char done[64] = {};
  const cudaError_t e = allow_smem(decode_mma2_kernel<64>, smem, done);
  if (e != cudaSuccess) return e;
  return launch_attention(decode_mma2_kernel<64>, blocks, D2_THREADS, smem, st, overlap_prev, tab, d, partials);
}

}  // namespace qp
