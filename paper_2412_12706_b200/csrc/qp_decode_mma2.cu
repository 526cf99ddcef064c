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

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int e = g >> 2, o = g & 3;                              // variant bit and unit index of this lane's MMA rows
  const bool lane_valid = e == (t >> 1);                        // this lane's accumulator entries are an e = e' block
  const int G = dm.Hq / dm.Hkv, BH = dm.Bt * dm.Hkv;
  const SkOwner sk{tab.total_tiles, tab.n_workers};
  const int cta = blockIdx.x;
  asm volatile("griddepcontrol.launch_dependents;\n" ::);
  long long cur = sk.start(cta);
  const long long f_end = sk.start(cta + 1);

  unsigned char* wsm = smem + warp * (D2_STAGES * TL::BYTES + SP2_BYTES);
  const uint32_t wsm_u = smem_u32(wsm);
  const uint32_t sP = wsm_u + D2_STAGES * TL::BYTES;
  float* s_acc = reinterpret_cast<float*>(smem);                // [warp][4 heads][D], overlays the idle stages
  float* s_m = s_acc + D2_WARPS * 4 * D;                        // [warp][4]
  float* s_l = s_m + D2_WARPS * 4;

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

  int li = 0;
  while (li + 1 < tab.n_layers && tab.l[li + 1].tile_base <= cur) ++li;

  while (cur < f_end) {
    const DecLayer& ly = tab.l[li];
    const int n = ly.n, tph = n >> 5;
    const int rel = (int)(cur - ly.tile_base), bh = rel / tph, tile_begin = rel % tph;
    const int n_tiles = (int)min((long long)(tph - tile_begin), f_end - cur);
    const int n_dt = (n_tiles + 1) >> 1;                        // double tiles of this segment
    const int b = bh / dm.Hkv, hk = bh % dm.Hkv;

    const unsigned char* gKc = static_cast<const unsigned char*>(ly.kc) + (size_t)bh * tph * D * 8;
    const unsigned char* gKs = reinterpret_cast<const unsigned char*>(ly.ks) + (size_t)bh * tph * D * 2;
    const unsigned char* gKz = reinterpret_cast<const unsigned char*>(ly.kz) + (size_t)bh * tph * D * 2;
    const unsigned char* gVc = static_cast<const unsigned char*>(ly.vc) + (size_t)bh * n * (D / 4);
    const unsigned char* gVs = reinterpret_cast<const unsigned char*>(ly.vs) + (size_t)bh * n * (D / 16);
    const unsigned char* gVz = reinterpret_cast<const unsigned char*>(ly.vz) + (size_t)bh * n * (D / 16);

    // stage double tile `dt` (tiles tile_begin + 2dt and, if inside the segment, + 1); a missing second tile is zero
    auto issue_dt = [&](int dt, int stage) {
      const uint32_t sb = wsm_u + stage * TL::BYTES;
      const int tile = tile_begin + 2 * dt;
      const bool two = 2 * dt + 1 < n_tiles;
      // key codes: per tile D pieces of 8 B (channel c), into half `te` of row slot(c)
#pragma unroll
      for (int te = 0; te < 2; ++te) {
        const unsigned char* src = gKc + (size_t)(tile + (two ? te : 0)) * D * 8 + lane * 8;
#pragma unroll
        for (int i = 0; i < D / 32; ++i) {
          const int c = lane + 32 * i;
          const int slot = c ^ ((c / (D / 4)) << 1);
          cp_async8_zfill(sb + TL::KC + slot * 16 + te * 8, src + i * 256, te == 0 || two);
        }
      }
      // value codes: per tile 32 tokens x NC pieces of 8 B (token tau, group vv)
#pragma unroll
      for (int te = 0; te < 2; ++te) {
        const unsigned char* src = gVc + (size_t)(tile + (two ? te : 0)) * 8 * D + lane * 8;
#pragma unroll
        for (int i = 0; i < D / 32; ++i) {
          const int idx = lane + 32 * i, tau = 32 * te + idx / NC, vv = idx % NC;
          const int rho = tau * NCH + vv % NCH;
          const int row = NCH == 2 ? rho ^ ((tau >> 2) & 1) : rho;
          cp_async8_zfill(sb + TL::VC + row * 16 + (vv / NCH) * 8, src + i * 256, te == 0 || two);
        }
      }
      // key scale / zero: per tile and array D/8 pieces of 16 B
      constexpr int MCH = D / 8;
#pragma unroll
      for (int te = 0; te < 2; ++te) {
        if (lane < 2 * MCH) {
          const int arr = lane / MCH, j = lane % MCH;           // 0 = scale, 1 = zero
          const unsigned char* src = (arr ? gKz : gKs) + (size_t)(tile + (two ? te : 0)) * D * 2 + j * 16;
          cp_async16_zfill(sb + TL::KS0 + (2 * te + arr) * TL::KMETA + j * 16 + (j / 8) * 16, src, te == 0 || two);
        }
      }
      // value scale / zero: the two tiles are contiguous, D/4 pieces of 16 B per array
      constexpr int VCH = D / 4;
      if (lane < VCH) {
        const bool ok = lane < VCH / 2 || two;
        const size_t off = (size_t)tile * 2 * D + (ok ? lane * 16 : 0);
        cp_async16_zfill(sb + TL::VS + lane * 16, gVs + off, ok);
        cp_async16_zfill(sb + TL::VZ + lane * 16, gVz + off, ok);
      }
    };

    const int n_my = warp < n_dt ? (n_dt - warp + D2_WARPS - 1) / D2_WARPS : 0;
#pragma unroll
    for (int s = 0; s < D2_STAGES - 1; ++s) {
      if (s < n_my) issue_dt(warp + D2_WARPS * s, s);
      cp_async_commit();
    }

    // query fragments: column g of the MMAs = (variant g>>2, head g&3); both variants carry the same q'
    uint32_t qh2[NPAIR];
    {
      const float scale_log2 = 1.4426950408889634f * rsqrtf((float)D);
      const uint16_t* qp = static_cast<const uint16_t*>(ly.q) + ((size_t)(b * dm.Hq + hk * G + o)) * D + (D / 4) * t;
#pragma unroll
      for (int i = 0; i < NPAIR; i += 4) {
        uint4 w4 = make_uint4(0u, 0u, 0u, 0u);
        if (o < G) w4 = *reinterpret_cast<const uint4*>(qp + 2 * i);
        qh2[i + 0] = pack_half2(bf16lo(w4.x) * scale_log2, bf16hi(w4.x) * scale_log2);
        qh2[i + 1] = pack_half2(bf16lo(w4.y) * scale_log2, bf16hi(w4.y) * scale_log2);
        qh2[i + 2] = pack_half2(bf16lo(w4.z) * scale_log2, bf16hi(w4.z) * scale_log2);
        qh2[i + 3] = pack_half2(bf16lo(w4.w) * scale_log2, bf16hi(w4.w) * scale_log2);
      }
    }

    // softmax state of heads 2(t&1), 2(t&1)+1 (identical in all lanes with the same t&1) and accumulators
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    float accO[NCH][4][4], accPZ[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int v = 0; v < NCH; ++v)
#pragma unroll
      for (int mt = 0; mt < 4; ++mt)
#pragma unroll
        for (int x = 0; x < 4; ++x) accO[v][mt][x] = 0.f;

    for (int it = 0; it < n_my; ++it) {
      __syncwarp();
      if (it + D2_STAGES - 1 < n_my) issue_dt(warp + D2_WARPS * (it + D2_STAGES - 1), (it + D2_STAGES - 1) % D2_STAGES);
      cp_async_commit();
      cp_async_wait<D2_STAGES - 1>();
      __syncwarp();
      const uint32_t sb = wsm_u + (it % D2_STAGES) * TL::BYTES;
      const bool tile_present = e == 0 || 2 * (warp + D2_WARPS * it) + 1 < n_tiles;   // is this lane's tile real?

      // ---------------- keys: rows (e, o) = tokens 8o..8o+7 of tile e; columns (e', h)
      float accK[4][4], accZ[4] = {0.f, 0.f, 0.f, 0.f};
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
        mma_unit8(accK, R0, R1, hmul2_u32(qh2[4 * c + 0], s4.x), hmul2_u32(qh2[4 * c + 1], s4.y));
        mma_f16_m16n8k16(accZ, z4.x, z4.x, z4.y, z4.y, qh2[4 * c + 0], qh2[4 * c + 1]);
        mma_unit8(accK, R2, R3, hmul2_u32(qh2[4 * c + 2], s4.z), hmul2_u32(qh2[4 * c + 3], s4.w));
        mma_f16_m16n8k16(accZ, z4.z, z4.z, z4.w, z4.w, qh2[4 * c + 2], qh2[4 * c + 3]);
      }
      // lg[2mt + rh][c]: token 8o + 2mt + rh of tile e, head 2(t&1) + c
      float lg[8][2];
      const bool use = lane_valid && tile_present;
#pragma unroll
      for (int mt = 0; mt < 4; ++mt) {
        lg[2 * mt][0] = use ? fmaf(accK[mt][0], cfac(2 * mt), accZ[0]) : -INFINITY;
        lg[2 * mt][1] = use ? fmaf(accK[mt][1], cfac(2 * mt), accZ[1]) : -INFINITY;
        lg[2 * mt + 1][0] = use ? fmaf(accK[mt][2], cfac(2 * mt + 1), accZ[0]) : -INFINITY;
        lg[2 * mt + 1][1] = use ? fmaf(accK[mt][3], cfac(2 * mt + 1), accZ[1]) : -INFINITY;
      }

      // ---------------- running softmax over the 64 tokens (log2 domain)
      float corr[2];
#pragma unroll
      for (int c = 0; c < 2; ++c) {
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
        float sum = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          lg[j][c] = ex2(lg[j][c] - mnew);                      // 0 for entries that are not logits
          sum += lg[j][c];
        }
        l_run[c] = fmaf(l_run[c], corr[c], sum);
      }
      if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {
#pragma unroll
        for (int v = 0; v < NCH; ++v)
#pragma unroll
          for (int mt = 0; mt < 4; ++mt) {
            accO[v][mt][0] *= corr[0]; accO[v][mt][1] *= corr[1];
            accO[v][mt][2] *= corr[0]; accO[v][mt][3] *= corr[1];
          }
        accPZ[0] *= corr[0]; accPZ[1] *= corr[1];
      }

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
            zp[kk][hf] = 0u;
            if (g < NC) {                                       // zero-point MMA: row g = value group g
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
    }

    // ---------------- per-warp result -> shared memory -> one partial per (head, block) and query head
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      l_run[c] += __shfl_xor_sync(0xffffffffu, l_run[c], 2);
      l_run[c] += __shfl_xor_sync(0xffffffffu, l_run[c], 4);
      l_run[c] += __shfl_xor_sync(0xffffffffu, l_run[c], 8);
      l_run[c] += __shfl_xor_sync(0xffffffffu, l_run[c], 16);
    }
    __syncthreads();                                            // every warp has consumed its last stage
#pragma unroll
    for (int v = 0; v < NCH; ++v) {
      // zero-point term of group vv = v + e*NCH for heads 2(t&1), +1: row vv of accPZ, columns (0, h)
      const int vv = v + e * NCH;
      const float pz0 = __shfl_sync(0xffffffffu, accPZ[0], 4 * vv + (t & 1));
      const float pz1 = __shfl_sync(0xffffffffu, accPZ[1], 4 * vv + (t & 1));
      if (lane_valid) {
        float* o0 = s_acc + ((warp * 4 + 2 * (t & 1)) * D);
        float* o1 = o0 + D;
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
          const int ch = 32 * vv + 8 * o + 2 * mt;
          *reinterpret_cast<float2*>(o0 + ch) =
              make_float2(fmaf(accO[v][mt][0], cfac(2 * mt), pz0), fmaf(accO[v][mt][2], cfac(2 * mt + 1), pz0));
          *reinterpret_cast<float2*>(o1 + ch) =
              make_float2(fmaf(accO[v][mt][1], cfac(2 * mt), pz1), fmaf(accO[v][mt][3], cfac(2 * mt + 1), pz1));
        }
      }
    }
    if (g == 0 && t < 2) {
      s_m[warp * 4 + 2 * t] = m_run[0]; s_m[warp * 4 + 2 * t + 1] = m_run[1];
      s_l[warp * 4 + 2 * t] = l_run[0]; s_l[warp * 4 + 2 * t + 1] = l_run[1];
    }
    __syncthreads();
    const size_t slot = (size_t)li * BH + bh + cta;
    for (int idx = tid; idx < G * D; idx += D2_THREADS) {
      const int h = idx / D, d = idx % D;
      float M = -INFINITY;
#pragma unroll
      for (int wp = 0; wp < D2_WARPS; ++wp) M = fmaxf(M, s_m[wp * 4 + h]);
      float Ls = 0.f, A = 0.f;
#pragma unroll
      for (int wp = 0; wp < D2_WARPS; ++wp) {
        const float mw = s_m[wp * 4 + h];
        if (mw != -INFINITY) {
          const float f = ex2(mw - M);
          Ls = fmaf(s_l[wp * 4 + h], f, Ls);
          A = fmaf(s_acc[(wp * 4 + h) * D + d], f, A);
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
constexpr size_t mma2_smem_bytes() {
  constexpr size_t stages = (size_t)D2_WARPS * (D2_STAGES * Tile2<D>::BYTES + SP2_BYTES);
  constexpr size_t combine = (size_t)D2_WARPS * 4 * D * 4 + 2 * D2_WARPS * 4 * 4;
  return stages > combine ? stages : combine;
}

}  // namespace

bool decode_mma2_supported(const DecDims& d) {
  return d.bits == 2 && d.group == 32 && (d.D == 128 || d.D == 64) && d.Hq / d.Hkv <= 4;
}

cudaError_t launch_decode_mma2(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st,
                               bool overlap_prev) {
  if (d.D == 128) {
    constexpr size_t smem = mma2_smem_bytes<128>();
    static unsigned char done[64] = {};
    const cudaError_t e = allow_smem(decode_mma2_kernel<128>, smem, done);
    if (e != cudaSuccess) return e;
    return launch_attention(decode_mma2_kernel<128>, tab.n_workers, D2_THREADS, smem, st, overlap_prev, tab, d, partials);
  }
  constexpr size_t smem = mma2_smem_bytes<64>();
  static unsigned char done[64] = {};
  const cudaError_t e = allow_smem(decode_mma2_kernel<64>, smem, done);
  if (e != cudaSuccess) return e;
  return launch_attention(decode_mma2_kernel<64>, tab.n_workers, D2_THREADS, smem, st, overlap_prev, tab, d, partials);
}

}  // namespace qp
