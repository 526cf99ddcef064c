// S4 on tensor cores: split-K decode attention that keeps the packed codes packed until they
// sit in MMA operand registers.
//
// Why tensor cores on an HBM-bound kernel: per byte of 4-bit cache there are 1.6 codes and each
// code needs one FMA per query head of the GQA group on the key side (and again on the value
// side).  On the fp32 pipes that is more issue slots than the SM has per byte it can fetch, so a
// scalar kernel is instruction-bound far below the memory roofline.  Here the multiply-adds go
// through mma.sync (m16n8k16, f16 operands, f32 accumulate, operands straight from registers);
// what is left per code on the integer pipe is about 0.6 instructions of mask/shift.
//
// Mapping (group g = 32, so one tile = 32 tokens = one key group):
//   keys   logit2[tok][h] = sum_d code[tok][d] * (q'[h][d] * s[d])  +  sum_d q'[h][d] * z[d]
//          A = codes, rows = tokens, k = channels;  B = q' * scale folded per tile (f16);
//          the zero-point term is a second small MMA whose A rows all hold z.
//   values out[h][d] = sum_tok code[tok][d] * (p[h][tok] * s[tok][v])  +  sum_tok p[h][tok] * z[tok][v]
//          A = codes, rows = channels, k = tokens;  B = p * scale per channel group v (f16);
//          zero-point term: A rows = v, one MMA per 16 tokens.
// q' = q * log2(e)/sqrt(D), softmax in the log2 domain.
//
// Codes become f16 operands without any conversion: a 16-bit lane holding a small integer c is
// the f16 number c * 2^-24 (subnormals and the first binade are equally spaced), so
// (word & 0x000f000f) is already a pair of f16 values; (word & 0x00f000f0) is the same scaled by
// 16.  The power-of-two factors are undone once, on the f32 accumulators.
// The packed layout stores a group's codes along the quantisation group (tokens for keys,
// channels for values) while an MMA register pairs two elements along the contraction; the
// transposing ldmatrix fetches 16-bit units of two different rows into one register, which is
// exactly that pairing.  Shared-memory rows are XOR-swizzled so these loads are conflict-free.
#include <algorithm>

#include "qp_mma.cuh"

namespace qp {

namespace {

#ifndef QP_DM_WARPS
#define QP_DM_WARPS 4
#endif
constexpr int DM_WARPS = QP_DM_WARPS;
constexpr int DM_THREADS = DM_WARPS * 32;
// Two builds of the kernel.  "Deep": three copy stages, three blocks (12 warps) per SM: a warp keeps two tiles in
// flight, which is what short ranges need (a worker with a handful of tiles is bound by the latency of its own
// copies).  "Wide": two stages, four blocks (16 warps) per SM and at most 128 registers: with long ranges the
// extra warps fill more issue slots than the shallower ring loses.  Measured, deep -> wide: 5.37 -> 5.60 TB/s on
// 336 MB launches of 8k-context caches, 5.87 -> 6.02 TB/s on 336 MB launches of 128k-context caches, but
// 20 -> 30 us on 84 MB launches, 5.11 -> 4.15 TB/s on a 168 MB launch whose merge grid is small enough to sit
// beside the attention blocks (the wide build leaves it no registers), and 5.18 -> 5.06 TB/s with 8 query heads
// per KV head.  The launch therefore takes the wide build only for 20 or more tiles per worker, at most 4 query
// heads per KV head and a merge grid of the large kind; five blocks per SM (96 registers) were slower again.
constexpr int DM_DEEP_STAGES = 3, DM_DEEP_MINB = 3, DM_WIDE_STAGES = 2, DM_WIDE_MINB = 4;
constexpr int DM_WIDE_MIN_TILES = 20;    // tiles per worker from which the wide build is used
constexpr int SP_STRIDE = 80;            // bytes per column of the per-warp P buffer (8 columns)
constexpr int SP_BYTES = 8 * SP_STRIDE;

// byte offsets of one 32-token tile in shared memory, 4-bit codes (value scale/zero regions sized for g = 32)
template <int D>
struct Tile4 {
  static constexpr int KC = 0;                    // D rows of 16 B: one channel, 32 tokens
  static constexpr int KS = KC + D * 16;          // D halves; channels >= 64 shifted by 16 B (bank spread)
  static constexpr int KZ = KS + D * 2 + 16;
  static constexpr int VC = KZ + D * 2 + 16;      // 32 token rows of D/2 bytes
  static constexpr int VS = VC + 16 * D;          // 32 x (D/32) halves
  static constexpr int VZ = VS + 2 * D;
  static constexpr int BYTES = VZ + 2 * D;
};
// key scale/zero of channel ch: the four lanes t read 16 B at channel (D/4)*t + 8c; the extra 16 B
// after channel 63 keeps lanes t and t+2 out of each other's banks
__host__ __device__ constexpr int ksz_off(int ch) { return ch * 2 + (ch / 64) * 16; }

constexpr uint32_t M0 = 0x000f000fu;   // code in bits 0..3 of each half: value c * 2^-24
constexpr uint32_t M1 = 0x00f000f0u;   // code in bits 4..7 of each half: value c * 2^-20
constexpr float C24 = 16777216.0f, C20 = 1048576.0f;

template <int D, int GROUP, int DM_STAGES, int DM_MINB>
__global__ void __launch_bounds__(DM_THREADS, DM_MINB)
decode_mma4_kernel(const __grid_constant__ DecTable tab, const DecDims dm, float* __restrict__ partials) {
  using TL = Tile4<D>;
  constexpr int NC = D / 32;       // ldmatrix.x4 calls over the channels of a key tile = value groups per token
  constexpr int NPAIR = D / 8;     // channel pairs owned by one lane on the key side (D/4 channels)
  constexpr int NG = D / GROUP;    // value scale groups per token
  constexpr int GT = GROUP / 32;   // 32-token tiles per key group
  extern __shared__ __align__(128) unsigned char smem[];

  const int tid = threadIdx.x, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);       // provably warp-uniform: cursors stay in uniform registers
  const int G = dm.Hq / dm.Hkv, BH = dm.Bt * dm.Hkv;
  // Every warp is a worker of its own: a contiguous range of the flat tile sequence, a private copy ring,
  // one partial record per head it touches.  Warps of a block share nothing and never synchronise.
  const int wk = blockIdx.x * DM_WARPS + warp;
  if (wk >= tab.n_workers) return;
  const SkOwner sk{tab.total_tiles, tab.n_workers};
  const long long f0 = sk.start(wk);
  const int total = (int)(sk.start(wk + 1) - f0);
  if (total <= 0) return;

  const uint32_t wsm_u = smem_u32(smem + warp * (DM_STAGES * TL::BYTES + SP_BYTES));
  const uint32_t sP = wsm_u + DM_STAGES * TL::BYTES;

  // per-lane shared-memory offsets: destinations of the asynchronous copies, sources of the transposing loads
  uint32_t kdst[D / 32], vdst[D / 32], k_off, v_off[NC];
#pragma unroll
  for (int i = 0; i < D / 32; ++i) {
    const int c = lane + 32 * i;                                // key channel
    kdst[i] = TL::KC + ((c ^ ((c / (D / 4)) << 1)) << 4);
    const int tau = c / NC, v = c % NC;                         // 16-byte piece of the value codes
    const int sw = NC == 4 ? (tau >> 1) & 3 : (tau >> 2) & 1;
    vdst[i] = TL::VC + tau * (D / 2) + ((v ^ sw) << 4);
  }
  {
    const int m = lane >> 3, r = lane & 7, tq = r >> 1, p = r & 1;
    const int ch = (D / 4) * tq + 2 * m + p;                    // + 8 per ldmatrix call
    k_off = TL::KC + ((ch ^ (tq << 1)) << 4);
    const int tau = 8 * m + r;                                  // matrix m = tokens 8m .. 8m+7
    const int sw = NC == 4 ? (tau >> 1) & 3 : (tau >> 2) & 1;
#pragma unroll
    for (int v = 0; v < NC; ++v) v_off[v] = TL::VC + tau * (D / 2) + ((v ^ sw) << 4);
  }
  constexpr int MCH = D / 8;                                    // 16-byte pieces of each scale / zero array
  const int mj = lane < MCH ? lane : lane - MCH;                // piece handled by this lane
  const uint32_t ksz_dst = (lane < MCH ? TL::KS : TL::KZ) + mj * 16 + (mj / 8) * 16;
  const uint32_t vsz_dst = (lane < MCH ? TL::VS : TL::VZ) + mj * 16;

  // Two cursors walk the range: the copy cursor (p_*) runs DM_STAGES - 1 tiles ahead of the compute cursor
  // (c_*) and crosses head and layer boundaries without draining the ring.
  int p_li = 0;
  while (p_li + 1 < tab.n_layers && (long long)tab.l[p_li + 1].tile_base <= f0) ++p_li;
  int p_tph = tab.l[p_li].n >> 5;
  int p_bh = (int)(f0 - tab.l[p_li].tile_base) / p_tph, p_tile = (int)(f0 - tab.l[p_li].tile_base) % p_tph;
  int c_li = p_li, c_bh = p_bh, c_tile = p_tile, c_tph = p_tph;

  // per-lane sources of the tile under the copy cursor; *m: scale or zero array by lane
  const unsigned char *gKc, *gKm, *gVc, *gVm;
  auto set_head = [&]() {
    const DecLayer& ly = tab.l[p_li];
    const size_t n = (size_t)ly.ns, bh = (size_t)p_bh;   // head stride: the arrays' capacity
    const int u = p_tile / GT, sub = p_tile % GT;
    // (a key group of GROUP tokens is GROUP/2 bytes per channel: a tile's 32 tokens are 16 of them)
    gKc = static_cast<const unsigned char*>(ly.kc) + bh * n * (D / 2) + (size_t)u * D * (GROUP / 2) + sub * 16 +
          lane * (GROUP / 2);
    gVc = static_cast<const unsigned char*>(ly.vc) + bh * n * (D / 2) + (size_t)p_tile * 16 * D + lane * 16;
    gKm = reinterpret_cast<const unsigned char*>(lane < MCH ? ly.ks : ly.kz) + (bh * (n / GROUP) + u) * D * 2 + mj * 16;
    gVm = reinterpret_cast<const unsigned char*>(lane < MCH ? ly.vs : ly.vz) + (bh * n + (size_t)p_tile * 32) * NG * 2 +
          mj * 16;
  };
  set_head();
  // stage the tile under the copy cursor (16-byte asynchronous copies, destinations swizzled for the
  // transposing loads), then advance the cursor
  auto issue_tile = [&](uint32_t sb) {
#pragma unroll
    for (int i = 0; i < D / 32; ++i) {
      cp_async16(sb + kdst[i], gKc + i * 32 * (GROUP / 2));
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
      gVc += 16 * D;
      gVm += 64 * NG;
      if (GT == 1 || p_tile % GT == 0) {
        gKc += D * (GROUP / 2) - (GT - 1) * 16;
        gKm += D * 2;
      } else {
        gKc += 16;
      }
    }
  };
#pragma unroll
  for (int s = 0; s < DM_STAGES - 1; ++s) {
    if (s < total) issue_tile(wsm_u + s * TL::BYTES);
    cp_async_commit();
  }
  uint32_t sb = wsm_u, sb_copy = wsm_u + (DM_STAGES - 1) * TL::BYTES;   // stage computed on / stage refilled

  uint32_t qh2[NPAIR];
  // running softmax reference of columns 2t, 2t+1 and the accumulators (cleared again after every record)
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
    if (it == gate) pdl_gate();                                 // see qp_mma.cuh: wait, then let the merge grid in
    if (fresh) {
      fresh = false;
      const DecLayer& ly = tab.l[c_li];
      const int b = c_bh / dm.Hkv, hk = c_bh % dm.Hkv;
      // B-side query fragments: column g of the MMAs is query head g of this KV head (columns >= G are 0);
      // this lane holds the D/4 channels [t*D/4, (t+1)*D/4) as f16 pairs
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
      __syncwarp();                                             // everyone is done with the stage refilled below
      if (it + DM_STAGES - 1 < total) issue_tile(sb_copy);
      cp_async_commit();
      cp_async_wait<DM_STAGES - 1>();
      __syncwarp();

      // ---------------- keys: logits of 32 tokens x 8 columns
      // Zero-point term sum_d q'[h][d] z[d]: the roles are swapped (A = this lane's query pairs as they sit in
      // registers, B = zero-point pairs as loaded), so no operand has to be copied into place.  With
      // A = (qa, qc, qb, qd) and B = (z_a, z_b) rows g of the result hold qa z_a + qb z_b of head g, with
      // B = (z_c, z_d) rows g+8 hold qc z_c + qd z_d; the other rows are never read.
      float accK[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
      float accZa[4] = {0.f, 0.f, 0.f, 0.f}, accZb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const uint4 s4 = lds128(sb + TL::KS + ksz_off((D / 4) * t + 8 * c));
        const uint4 z4 = lds128(sb + TL::KZ + ksz_off((D / 4) * t + 8 * c));
        // qh2[4c + (0, 1, 2, 3)] hold the channel pairs (0, 2, 1, 3) of this lane's eight channels
        const uint32_t qs0 = hmul2_u32(qh2[4 * c + 0], s4.x), qs1 = hmul2_u32(qh2[4 * c + 2], s4.y);
        const uint32_t qs2 = hmul2_u32(qh2[4 * c + 1], s4.z), qs3 = hmul2_u32(qh2[4 * c + 3], s4.w);
        uint32_t R0, R1, R2, R3;
        ldmatrix_x4_trans(R0, R1, R2, R3, sb + k_off + c * 128);
        mma_f16_m16n8k16(accK[0], R0 & M0, R0 & M1, R1 & M0, R1 & M1, qs0, qs1);
        const uint32_t S0 = R0 >> 8, S1 = R1 >> 8;
        mma_f16_m16n8k16(accK[1], S0 & M0, S0 & M1, S1 & M0, S1 & M1, qs0, qs1);
        mma_f16_m16n8k16(accZa, qh2[4 * c + 0], qh2[4 * c + 1], qh2[4 * c + 2], qh2[4 * c + 3], z4.x, z4.y);
        mma_f16_m16n8k16(accK[0], R2 & M0, R2 & M1, R3 & M0, R3 & M1, qs2, qs3);
        const uint32_t S2 = R2 >> 8, S3 = R3 >> 8;
        mma_f16_m16n8k16(accK[1], S2 & M0, S2 & M1, S3 & M0, S3 & M1, qs2, qs3);
        mma_f16_m16n8k16(accZb, qh2[4 * c + 0], qh2[4 * c + 1], qh2[4 * c + 2], qh2[4 * c + 3], z4.z, z4.w);
      }
      // the term of head g sits in lanes (g, *); this lane needs those of columns 2t and 2t+1
      const float zq = accZa[0] + accZb[2];
      const float zq0 = __shfl_sync(0xffffffffu, zq, 8 * t), zq1 = __shfl_sync(0xffffffffu, zq, 8 * t + 4);
      // this lane: tokens 4g .. 4g+3 of the tile, columns 2t and 2t+1
      //   lg[j][e]: logit of token 4g + j, column 2t + e, minus the column's reference maximum
      //
      // ---------------- running softmax (log2 domain)
      // m_run is a reference, not the exact running maximum: it is renewed only when a logit exceeds it by more
      // than kSlack, so p = 2^(logit - m_run) stays below 2^kSlack (the f16 products p * scale keep 12 binades
      // of headroom) and the accumulators are rescaled on a few tiles per head, found without any shuffle.
      constexpr float kSlack = 4.f;
      const float zq_e[2] = {zq0, zq1};
      float lg[4][2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const float zm = zq_e[e] - m_run[e];                    // +inf on the first tile of a head
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          lg[2 * mt][e] = fmaf(accK[mt][e], C24, zm);
          lg[2 * mt + 1][e] = fmaf(accK[mt][2 + e], C20, zm);
        }
      }
      const float over = fmaxf(fmaxf(fmaxf(lg[0][0], lg[1][0]), fmaxf(lg[2][0], lg[3][0])),
                               fmaxf(fmaxf(lg[0][1], lg[1][1]), fmaxf(lg[2][1], lg[3][1])));
      if (__any_sync(0xffffffffu, over > kSlack)) {             // rare: renew the references, rescale
        float corr[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            lg[2 * mt][e] = fmaf(accK[mt][e], C24, zq_e[e]);
            lg[2 * mt + 1][e] = fmaf(accK[mt][2 + e], C20, zq_e[e]);
          }
          float mx = fmaxf(fmaxf(lg[0][e], lg[1][e]), fmaxf(lg[2][e], lg[3][e]));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
          const float mnew = fmaxf(m_run[e], mx);
          corr[e] = ex2(m_run[e] - mnew);
          m_run[e] = mnew;
#pragma unroll
          for (int j = 0; j < 4; ++j) lg[j][e] -= mnew;
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
        for (int j = 0; j < 4; ++j) lg[j][e] = ex2(lg[j][e]);    // p; its sum over the tokens: row NG of accPZ

      // ---------------- P through shared memory: [column][token] f16, then token pairs of column g
      sts64(sP + (2 * t) * SP_STRIDE + g * 8, pack_half2(lg[0][0], lg[1][0]), pack_half2(lg[2][0], lg[3][0]));
      sts64(sP + (2 * t + 1) * SP_STRIDE + g * 8, pack_half2(lg[0][1], lg[1][1]), pack_half2(lg[2][1], lg[3][1]));
      __syncwarp();
      uint32_t p2[4];                                           // tokens (2t,2t+1) + {0, 8, 16, 24}
#pragma unroll
      for (int pr = 0; pr < 4; ++pr) p2[pr] = lds32(sP + g * SP_STRIDE + 4 * t + 16 * pr);

      // ---------------- values: B = p * scale of the token's channel group, zero-point rows
      // zero-point MMA: row g < NG holds the zero points of scale group g, row NG holds ones (the softmax
      // denominator comes out of the same MMA, summed over the tokens in f32)
      uint32_t ps[4][NG], zp[4];                                // ps[pair][scale group]
#pragma unroll
      for (int pr = 0; pr < 4; ++pr) {
        const int a = 8 * pr + 2 * t;                           // first token of the pair
        zp[pr] = g == NG ? 0x3c003c00u : 0u;
        if constexpr (NG == 4) {
          const uint4 x = lds128(sb + TL::VS + a * 8);
          ps[pr][0] = hmul2_u32(p2[pr], __byte_perm(x.x, x.z, 0x5410));
          ps[pr][1] = hmul2_u32(p2[pr], __byte_perm(x.x, x.z, 0x7632));
          ps[pr][2] = hmul2_u32(p2[pr], __byte_perm(x.y, x.w, 0x5410));
          ps[pr][3] = hmul2_u32(p2[pr], __byte_perm(x.y, x.w, 0x7632));
          if (g < NG) {                                         // rows of the zero-point MMA: scale group g
            const uint32_t ya = lds32(sb + TL::VZ + a * 8 + (g & 2) * 2);       // z[a][g & ~1], z[a][g | 1]
            const uint32_t yb = lds32(sb + TL::VZ + a * 8 + 8 + (g & 2) * 2);   // same of token a + 1
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
    }

    // ---------------- end of this head's part of the range: one partial record per query head, from registers
    if (++c_tile == c_tph || it == total - 1) {
      // softmax denominators of columns 2t, 2t+1: row NG of the zero-point accumulator, lane (NG, t)
      const float l0 = __shfl_sync(0xffffffffu, accPZ[0], 4 * NG + t), l1 = __shfl_sync(0xffffffffu, accPZ[1], 4 * NG + t);
      const size_t slot = (size_t)c_li * BH + c_bh + wk;
      float* r0 = partials + (slot * G + 2 * t) * (size_t)(D + 2);      // record of column 2t; column 2t+1 follows
      float* r1 = r0 + (D + 2);
      const bool h0 = 2 * t < G, h1 = 2 * t + 1 < G;
#pragma unroll
      for (int v = 0; v < NC; ++v) {
        // zero-point term of the scale group of channels 32v.. for columns 2t, 2t+1 sits in lane (g = group, t)
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
  // This kernel may have started while the previous call's merge kernel was still reading its records: alternate
  // calls use alternate halves of the workspace, and the call before the previous one had ended before this
  // kernel could start (pdl_gate), so no record store had to wait.
}

// S5 for the decomposition above: head (layer, batch, KV head) was touched by the blocks
// owner(first tile) .. owner(last tile); their records sit at slots head + block.
// One warp per (layer, batch, query head), a lane per four channels.  The kernel is launched as a
// programmatic dependent of the attention kernel: its blocks may become resident while that kernel
// drains and wait at griddepcontrol.wait until its records are complete and visible.  It passes the
// permission on at once, so that the next call's attention kernel can fill the machine while this
// one runs; that kernel reads none of this one's outputs and writes the other half of the workspace.
constexpr int MG_WARPS = 4;
// At most 32 registers per thread, so that a block fits beside the resident blocks of the attention kernel.  A
// small launch (up to two blocks of work per SM) uses at most one block per SM: the whole grid is then resident
// and has passed the launch permission on long before the attention kernel ends, the next call's attention
// kernel fills the SMs as this call's drains, and this kernel runs in that kernel's shadow.  A large launch
// would take too long that way; it uses a warp per output row and overlaps the next call's ramp only.
// The same merge with plain loads (two records in flight per warp).
template <int RUN, int MINB>
__global__ void __launch_bounds__(MG_WARPS * 32, MINB)
decode_merge_direct_kernel(const __grid_constant__ DecTable tab, const DecDims dm, const float* __restrict__ partials) {
  const int D = dm.D, G = dm.Hq / dm.Hkv, BH = dm.Bt * dm.Hkv, n_bq = dm.Bt * dm.Hq;
  const int lane = threadIdx.x & 31, n_items = n_bq * tab.n_layers;
  const unsigned T = (unsigned)tab.total_tiles, W = (unsigned)tab.n_workers;   // T * W < 2^31 (host-checked)
  const size_t stride = (size_t)G * (D + 2);
  asm volatile("griddepcontrol.launch_dependents;\n" ::);
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  for (int item = blockIdx.x * MG_WARPS + (threadIdx.x >> 5); item < n_items; item += gridDim.x * MG_WARPS) {
    const int layer = item / n_bq, bq = item % n_bq;
    const DecLayer& ly = tab.l[layer];
    const int b = bq / dm.Hq, h = bq % dm.Hq, bh = b * dm.Hkv + h / G, hl = h % G;
    const int tph = (ly.n + 31) >> 5;
    const unsigned first = (unsigned)ly.tile_base + (unsigned)bh * tph;
    const int w_lo = (int)(((first + 1u) * W - 1u) / T), w_hi = (int)(((first + tph) * W - 1u) / T);
    const size_t head = (size_t)layer * BH + bh;
    const float* base = partials + (head * G + hl) * (size_t)(D + 2);
    // reference maxima of the records: a lane per record, then across the warp
    float M = -INFINITY;
    for (int w = w_lo + lane; w <= w_hi; w += 32) M = fmaxf(M, base[w * stride]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    if (4 * lane >= D) continue;
    float Ls = 0.f, A0 = 0.f, A1 = 0.f, A2 = 0.f, A3 = 0.f;
    // RUN records' loads are in flight together (past the row's end the last record again, with weight 0)
    for (int w0 = w_lo; w0 <= w_hi; w0 += RUN) {
      float2 ml[RUN], a01[RUN], a23[RUN];
#pragma unroll
      for (int i = 0; i < RUN; ++i) {
        const float* r = base + min(w0 + i, w_hi) * stride;
        ml[i] = *reinterpret_cast<const float2*>(r);
        a01[i] = *reinterpret_cast<const float2*>(r + 2 + 4 * lane);
        a23[i] = *reinterpret_cast<const float2*>(r + 4 + 4 * lane);
      }
#pragma unroll
      for (int i = 0; i < RUN; ++i) {
        const float f = w0 + i <= w_hi ? ex2(ml[i].x - M) : 0.f;
        Ls = fmaf(ml[i].y, f, Ls);
        A0 = fmaf(a01[i].x, f, A0); A1 = fmaf(a01[i].y, f, A1);
        A2 = fmaf(a23[i].x, f, A2); A3 = fmaf(a23[i].y, f, A3);
      }
    }
    const float inv = __fdiv_rn(1.0f, Ls);
    __nv_bfloat162 o01 = __floats2bfloat162_rn(A0 * inv, A1 * inv), o23 = __floats2bfloat162_rn(A2 * inv, A3 * inv);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t*>(&o01);
    packed.y = *reinterpret_cast<uint32_t*>(&o23);
    *reinterpret_cast<uint2*>(static_cast<bf16*>(ly.out) + (size_t)bq * D + 4 * lane) = packed;
  }
}

constexpr int MG_BATCH = 8;              // records staged per warp at a time
__device__ __forceinline__ void cp_async8(uint32_t saddr, const void* gptr) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(saddr), "l"(gptr));
}
__global__ void __launch_bounds__(MG_WARPS * 32, 16)
decode_merge_sk_kernel(const __grid_constant__ DecTable tab, const DecDims dm, const float* __restrict__ partials) {
  // A row's records are fetched MG_BATCH at a time with asynchronous copies into shared memory (no registers are
  // held by loads in flight, which the 32-register budget could not afford): one memory round trip per batch
  // instead of one per record.
  // a staged record: (max, sum) at floats 0, 1, the D accumulators from float 4 on (16-byte aligned rows of 132)
  __shared__ __align__(16) float s_rec[MG_WARPS][MG_BATCH][132];
  const int D = dm.D, G = dm.Hq / dm.Hkv, BH = dm.Bt * dm.Hkv, n_bq = dm.Bt * dm.Hq;
  const int lane = threadIdx.x & 31, wq = threadIdx.x >> 5, n_items = n_bq * tab.n_layers;
  const unsigned T = (unsigned)tab.total_tiles, W = (unsigned)tab.n_workers;   // T * W < 2^31 (host-checked)
  const size_t stride = (size_t)G * (D + 2);
  const int pieces = (D + 2) / 2;                                // 8-byte pieces of a record (records are 8-byte aligned)
  float (*rec)[132] = s_rec[wq];
  const uint32_t rec_u = smem_u32(&rec[0][0]);
  asm volatile("griddepcontrol.launch_dependents;\n" ::);
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  for (int item = blockIdx.x * MG_WARPS + wq; item < n_items; item += gridDim.x * MG_WARPS) {
    const int layer = item / n_bq, bq = item % n_bq;
    const DecLayer& ly = tab.l[layer];
    const int b = bq / dm.Hq, h = bq % dm.Hq, bh = b * dm.Hkv + h / G, hl = h % G;
    const int tph = (ly.n + 31) >> 5;
    const unsigned first = (unsigned)ly.tile_base + (unsigned)bh * tph;
    const int w_lo = (int)(((first + 1u) * W - 1u) / T), w_hi = (int)(((first + tph) * W - 1u) / T);
    const size_t head = (size_t)layer * BH + bh;
    const float* base = partials + ((head + w_lo) * G + hl) * (size_t)(D + 2);
    const int count = w_hi - w_lo + 1;
    // running reference maximum over the batches (a single batch in all but very finely split launches)
    float M = -INFINITY, Ls = 0.f, A0 = 0.f, A1 = 0.f, A2 = 0.f, A3 = 0.f;
    for (int r0 = 0; r0 < count; r0 += MG_BATCH) {
      const int nb = min(MG_BATCH, count - r0);
      __syncwarp();                                              // the previous batch has been consumed
      for (int p = lane; p < nb * pieces; p += 32) {
        const int j = p / pieces, o = p % pieces;
        cp_async8(rec_u + (j * 132 + (o ? 2 + 2 * o : 0)) * 4, base + (size_t)(r0 + j) * stride + 2 * o);
      }
      cp_async_commit();
      cp_async_wait<0>();
      __syncwarp();
      float mb = lane < nb ? rec[lane][0] : -INFINITY;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, o));
      const float Mn = fmaxf(M, mb), corr = ex2(M - Mn);         // corr = 0 on the first batch (M = -inf)
      M = Mn;
      Ls *= corr; A0 *= corr; A1 *= corr; A2 *= corr; A3 *= corr;
      if (4 * lane < D)
        for (int j = 0; j < nb; ++j) {
          const float f = ex2(rec[j][0] - M);
          const float4 a = *reinterpret_cast<const float4*>(&rec[j][4 + 4 * lane]);
          Ls = fmaf(rec[j][1], f, Ls);
          A0 = fmaf(a.x, f, A0); A1 = fmaf(a.y, f, A1);
          A2 = fmaf(a.z, f, A2); A3 = fmaf(a.w, f, A3);
        }
    }
    if (4 * lane >= D) continue;
    const float inv = __fdiv_rn(1.0f, Ls);
    __nv_bfloat162 o01 = __floats2bfloat162_rn(A0 * inv, A1 * inv), o23 = __floats2bfloat162_rn(A2 * inv, A3 * inv);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t*>(&o01);
    packed.y = *reinterpret_cast<uint32_t*>(&o23);
    *reinterpret_cast<uint2*>(static_cast<bf16*>(ly.out) + (size_t)bq * D + 4 * lane) = packed;
  }
}

// S5 for launches with few output rows (at most one per SM): one block per (layer, batch, query head), its four
// warps share the head's records (warp q takes records q, q + 4, ...), so a row's chain of dependent reads is a
// quarter as long; the four partial sums are combined through shared memory in a fixed order.  Same launch
// protocol as decode_merge_sk_kernel.
constexpr int MR_RUN = 8;
#ifndef QP_MERGE_ROWS_PER_SM
#define QP_MERGE_ROWS_PER_SM 8
#endif
__global__ void __launch_bounds__(MG_WARPS * 32, 8)
decode_merge_rows_kernel(const __grid_constant__ DecTable tab, const DecDims dm, const float* __restrict__ partials) {
  __shared__ float s_max[MG_WARPS];
  __shared__ float s_part[MG_WARPS][5 * 32];                      // per warp: lane's (A0..A3, Ls)
  const int D = dm.D, G = dm.Hq / dm.Hkv, BH = dm.Bt * dm.Hkv, n_bq = dm.Bt * dm.Hq;
  const int lane = threadIdx.x & 31, wq = threadIdx.x >> 5;
  const unsigned T = (unsigned)tab.total_tiles, W = (unsigned)tab.n_workers;
  const size_t stride = (size_t)G * (D + 2);
  asm volatile("griddepcontrol.launch_dependents;\n" ::);
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  const int layer = blockIdx.x / n_bq, bq = blockIdx.x % n_bq;
  const DecLayer& ly = tab.l[layer];
  const int b = bq / dm.Hq, h = bq % dm.Hq, bh = b * dm.Hkv + h / G, hl = h % G;
  const int tph = (ly.n + 31) >> 5;
  const unsigned first = (unsigned)ly.tile_base + (unsigned)bh * tph;
  const int w_lo = (int)(((first + 1u) * W - 1u) / T), w_hi = (int)(((first + tph) * W - 1u) / T);
  const float* base = partials + (((size_t)layer * BH + bh) * G + hl) * (size_t)(D + 2);
  // the records' reference maxima: a thread per record, then across the block
  float M = -INFINITY;
  for (int w = w_lo + (int)threadIdx.x; w <= w_hi; w += MG_WARPS * 32) M = fmaxf(M, base[w * stride]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  if (lane == 0) s_max[wq] = M;
  __syncthreads();
  M = fmaxf(fmaxf(s_max[0], s_max[1]), fmaxf(s_max[2], s_max[3]));
  float Ls = 0.f, A0 = 0.f, A1 = 0.f, A2 = 0.f, A3 = 0.f;
  // a warp takes runs of MR_RUN consecutive records and has all of a run's loads in flight before it folds them: a long
  // row (a single layer with thousands of kept tokens leaves a hundred records per row) is a chain of dependent
  // round trips otherwise (measured for 128 records per row: 20 us with one record at a time)
  if (4 * lane < D)
    for (int w0 = w_lo + wq * MR_RUN; w0 <= w_hi; w0 += MG_WARPS * MR_RUN) {
      float2 ml[MR_RUN], a01[MR_RUN], a23[MR_RUN];
#pragma unroll
      for (int i = 0; i < MR_RUN; ++i) {
        const float* r = base + min(w0 + i, w_hi) * stride;     // past the end: the last record again, weight 0 below
        ml[i] = *reinterpret_cast<const float2*>(r);
        a01[i] = *reinterpret_cast<const float2*>(r + 2 + 4 * lane);
        a23[i] = *reinterpret_cast<const float2*>(r + 4 + 4 * lane);
      }
#pragma unroll
      for (int i = 0; i < MR_RUN; ++i) {
        const float f = w0 + i <= w_hi ? ex2(ml[i].x - M) : 0.f;
        Ls = fmaf(ml[i].y, f, Ls);
        A0 = fmaf(a01[i].x, f, A0); A1 = fmaf(a01[i].y, f, A1);
        A2 = fmaf(a23[i].x, f, A2); A3 = fmaf(a23[i].y, f, A3);
      }
    }
  float* mine = s_part[wq] + 5 * lane;
  mine[0] = A0; mine[1] = A1; mine[2] = A2; mine[3] = A3; mine[4] = Ls;
  __syncthreads();
  if (wq != 0 || 4 * lane >= D) return;
  Ls = A0 = A1 = A2 = A3 = 0.f;
#pragma unroll
  for (int q = 0; q < MG_WARPS; ++q) {
    const float* o = s_part[q] + 5 * lane;
    A0 += o[0]; A1 += o[1]; A2 += o[2]; A3 += o[3]; Ls += o[4];
  }
  const float inv = __fdiv_rn(1.0f, Ls);
  __nv_bfloat162 o01 = __floats2bfloat162_rn(A0 * inv, A1 * inv), o23 = __floats2bfloat162_rn(A2 * inv, A3 * inv);
  uint2 packed;
  packed.x = *reinterpret_cast<uint32_t*>(&o01);
  packed.y = *reinterpret_cast<uint32_t*>(&o23);
  *reinterpret_cast<uint2*>(static_cast<bf16*>(ly.out) + (size_t)bq * D + 4 * lane) = packed;
}

template <int D, int STAGES>
constexpr size_t mma4_smem_bytes() { return (size_t)DM_WARPS * (STAGES * Tile4<D>::BYTES + SP_BYTES); }

}  // namespace

bool decode_mma_supported(const DecDims& d) {
  if (d.D != 128 && d.D != 64) return false;
  if (d.bits == 16) return true;
  if (d.bits == 4 || d.bits == 8) return d.D % d.group == 0;   // groups of 32, 64, 128
  return d.group == 32 && decode_mma2_supported(d);
}

// The quantized kernels' workers are warps; the 16-bit kernel's workers are blocks of four warps.
int decode_mma_workers_per_sm(const DecDims& d) {
  return d.bits == 4 ? DM_DEEP_MINB * DM_WARPS : d.bits == 8 ? decode_mma8_blocks_per_sm() * decode_mma8_warps()
         : d.bits == 16 ? decode_mma16_blocks_per_sm() : decode_mma2_workers_per_sm();
}
// Launches that do not fill every worker slot with a long range use fewer workers, not emptier ones: a worker's
// ramp and its partial record (which the merge step has to read) are costs per worker.  On a stream whose calls
// overlap, two calls share the GPU most of the time, so a call wants about half of the resident worker slots:
// measured for the 4- and 8-bit kernels with at least 12 / 16 / 20 / 24 / 32 tiles per worker (us per call, calls
// overlapping): 84 MB 4-bit 28.2 / 20.2 / 22.1 / 23.5 / 22.3, 168 MB 4-bit 35.9 / 35.8 / 40.8 / 38.1 / 34.2, 151 MB 8-bit
// 34.9 / 33.0 / 35.1 / 38.7 / 36.6, 75 MB 8-bit 23.1 / 22.3 / 25.0 / 26.4 / 24.0, 42 MB 4-bit 16.9 / 16.3 / 16.6 / 17.4 / 18.6.
// A call that runs alone (plain stream order) takes as many workers as it can give four tiles each: per-layer calls
// replayed from a CUDA graph 10.2 / 8.4 / 8.4 / 10.2 us with at least 1 / 2 / 4 / 8 tiles per worker.  Beyond 2048 tiles
// (a layer of a whole batch, or one long sequence) eight tiles each pay, because the merge reads fewer records: from a
// graph with at least 4 / 8 / 16 tiles, one layer of 8 heads x 16384 tokens 12.8 / 11.8 / 15.6 us, one layer of the 70B
// shapes at batch 4 (42 MB) 20.8 / 17.7 / 17.8 us, 8 heads x 2048 tokens 7.7 / 10.1 / 15.1 us.  The 2-bit and 16-bit
// kernels showed no gain from fewer workers on overlapping streams and use four tiles there.
#ifndef QP_TMIN_BIG
#define QP_TMIN_BIG 16
#endif
#ifndef QP_TMIN_SMALL
#define QP_TMIN_SMALL 16
#endif
#ifndef QP_TMIN_SOLO
#define QP_TMIN_SOLO 4
#endif
int decode_mma_tiles_per_worker_min(const DecDims& d, long long total_tiles, bool paired) {
  if (!paired) return total_tiles > 2048 ? 2 * QP_TMIN_SOLO : QP_TMIN_SOLO;
  if (d.bits != 4 && d.bits != 8) return 4;
  return total_tiles / QP_TMIN_BIG >= 256 ? QP_TMIN_BIG : QP_TMIN_SMALL;
}
// Workers per SM of the wider build of this shape's kernel and the tiles per worker from which it pays
// (0: the shape has one build only).
int decode_mma_wide_workers_per_sm(const DecDims& d, int* min_tiles) {
  if (d.bits != 4 || d.Hq / d.Hkv > 4) return 0;              // (with 8 query heads per KV head the deep build wins)
  *min_tiles = DM_WIDE_MIN_TILES;
  return DM_WIDE_MINB * DM_WARPS;
}

namespace {
template <int D, int GROUP, int STAGES, int MINB>
cudaError_t launch_mma4_build(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st, bool overlap_prev) {
  constexpr size_t smem = mma4_smem_bytes<D, STAGES>();
  static unsigned char done[64] = {};
  const cudaError_t e = allow_smem(decode_mma4_kernel<D, GROUP, STAGES, MINB>, smem, done);
  if (e != cudaSuccess) return e;
  return launch_attention(decode_mma4_kernel<D, GROUP, STAGES, MINB>, (tab.n_workers + DM_WARPS - 1) / DM_WARPS,
                          DM_THREADS, smem, st, overlap_prev, tab, d, partials);
}
template <int D, int GROUP>
cudaError_t launch_mma4(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st, bool overlap_prev) {
  if (tab.wide) return launch_mma4_build<D, GROUP, DM_WIDE_STAGES, DM_WIDE_MINB>(tab, d, partials, st, overlap_prev);
  return launch_mma4_build<D, GROUP, DM_DEEP_STAGES, DM_DEEP_MINB>(tab, d, partials, st, overlap_prev);
}
}  // namespace

cudaError_t launch_decode_mma4(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st,
                               bool overlap_prev) {
  if (d.D == 128) {
    if (d.group == 32) return launch_mma4<128, 32>(tab, d, partials, st, overlap_prev);
    if (d.group == 64) return launch_mma4<128, 64>(tab, d, partials, st, overlap_prev);
    return launch_mma4<128, 128>(tab, d, partials, st, overlap_prev);
  }
  if (d.group == 32) return launch_mma4<64, 32>(tab, d, partials, st, overlap_prev);
  return launch_mma4<64, 64>(tab, d, partials, st, overlap_prev);
}

cudaError_t launch_decode_mma(const DecTable& tab, const DecDims& d, float* partials, cudaStream_t st,
                              bool overlap_prev, const TailTable* tails) {
  cudaError_t e = d.bits == 4   ? launch_decode_mma4(tab, d, partials, st, overlap_prev)
                  : d.bits == 8 ? launch_decode_mma8(tab, d, partials, st, overlap_prev)
                  : d.bits == 16 ? launch_decode_mma16(tab, d, partials, st, overlap_prev)
                                : launch_decode_mma2(tab, d, partials, st, overlap_prev);
  if (e != cudaSuccess) return e;
  if (tails) return launch_merge_tail(tab, d, partials, *tails, st, true);
  return launch_merge_flat(tab, d, partials, st);
}

cudaError_t launch_merge_flat(const DecTable& tab, const DecDims& d, const float* partials, cudaStream_t st) {
  const int items = d.Bt * d.Hq * tab.n_layers;
  cudaLaunchConfig_t cfg = {};
  const int row_blocks = (items + MG_WARPS - 1) / MG_WARPS;
  cfg.gridDim = dim3(row_blocks <= 2 * sm_count() ? std::min(row_blocks, sm_count()) : row_blocks);
  cfg.blockDim = dim3(MG_WARPS * 32);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // few rows: a block per row, whose four warps share the row's records (one layer of a batch: 256 rows of 33 records
  // took 9.4 us with a warp per row on 64 SMs; graph replay of such calls 17.7 -> 15.1 us; up to 8 rows per SM also the
  // 32-layer calls of one sequence gain in plain order, 84 MB 25.8 -> 24.5 us, 336 MB 67.8 -> 65.6 us).  On overlapping
  // streams only up to a block per SM, so that the grid fits beside the next call's attention blocks.
  if (items <= (tab.paired ? 1 : QP_MERGE_ROWS_PER_SM) * sm_count()) {
    cfg.gridDim = dim3(items);
    return cudaLaunchKernelEx(&cfg, decode_merge_rows_kernel, tab, d, (const float*)partials);
  }
  // Measured: on 134-201 MB launches whose merge grid is of the small kind (a block per SM at most) the staged
  // form is the faster one beside the next call's attention blocks (overlapping calls; 168 MB 4-bit calls 52 -> 34 us
  // per call), while alone on the GPU the plain loads are (60 -> 45 us); on GB-sized launches, whose rows have one
  // or two records each, the plain loads win in both modes (2.1 GB calls: 422 -> 362 us).
  if (!tab.paired || row_blocks > 2 * sm_count()) {
    // rows with a few records: two loads in flight and 32 registers, so the grid fits beside attention blocks; longer
    // rows (one layer of a batch leaves dozens of records per row): eight in flight
    const long long heads = (long long)tab.n_layers * d.Bt * d.Hkv;
    if (tab.n_workers / heads + 1 <= 4)
      return cudaLaunchKernelEx(&cfg, decode_merge_direct_kernel<2, 16>, tab, d, (const float*)partials);
    return cudaLaunchKernelEx(&cfg, decode_merge_direct_kernel<8, 8>, tab, d, (const float*)partials);
  }
  return cudaLaunchKernelEx(&cfg, decode_merge_sk_kernel, tab, d, (const float*)partials);
}

}  // namespace qp
