/*
 * qp_oracle.c — plain CPU oracle for the quantized-pruning KV-cache path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement
 * of what the GPU library computes.  It shares no code, header, table or helper
 * with the CUDA path and must never be linked into or called from it.
 *
 * What it follows (paper sections / equations):
 *   - decode attention: Methods, "Decoding Phase", Eq. (3)  h_O = Softmax(h_Q X_K^T) X_V
 *   - quantization:     Methods, "KV Quantization", Eq. (4)  Q(G) = round((G - z)/s),
 *                       s = (m - z)/(2^B - 1)
 *   - dequantization:   Methods, "KV Quantization", Eq. (5)  G' = Q(G)*s + z
 *   - pruning:          Methods, "KV Pruning" (keep s < n tokens per head)
 *   - composition:      Methods, "Quantized Pruning" (prune first, then quantize
 *                       the kept states; decode on the dequantized result)
 *   - grouping axes:    Related Work "KV Quantization" / Sec. 5.3: keys per-channel,
 *                       values per-token (KIVI)
 *   - window / budgets: Appendix B (last 32 tokens kept; memory budget = tokens x bits)
 * The paper names its pruning method (SnapKV) without defining it; the scoring
 * rule implemented here is the reading stated next to qpo_scores().
 *
 * Precision: everything is fp64 except the quantizer, whose stored outputs
 * (codes, fp16 scale, fp16 zero) are defined in fp32 IEEE arithmetic in a fixed
 * operation order so that they can be compared bit for bit.
 *
 * Pin status: every function below is pinned by tests that do not call it to
 * produce the expected value (closed forms, brute force, numpy's float16, dense
 * attention written with numpy).  The *choices* among readings the paper cannot
 * decide (sum over the GQA group, zero padding with divisor = pool, round-up of
 * the stored scale, ascending order of kept tokens) are "parity unpinned,
 * reading stated".
 *
 * Threading: only the outermost independent loop (batch x KV head) is
 * parallelised (OpenMP), nothing is blocked, fused or reordered.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---------- number formats ------------------------------------------------ */

static inline float bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

static inline float f16_to_f32(uint16_t h) {
  uint32_t sign = (uint32_t)(h >> 15) & 1u;
  int32_t e = (h >> 10) & 0x1f;
  uint32_t m = h & 0x3ffu;
  double v;
  if (e == 0) v = ldexp((double)m, -24);                 /* zero / subnormal */
  else if (e == 31) v = m ? NAN : INFINITY;
  else v = ldexp((double)(m | 0x400u), e - 25);          /* (1 + m/1024) * 2^(e-15) */
  return (float)(sign ? -v : v);
}

/* fp32 -> fp16 with a directed rounding: dir < 0 rounds toward -inf (largest
 * fp16 <= x), dir > 0 toward +inf (smallest fp16 >= x).  NaN is returned as a
 * quiet NaN.  Magnitudes beyond the largest finite fp16 go to +-65504 or +-inf
 * according to the direction, as IEEE directed rounding prescribes. */
static uint16_t f32_to_f16_dir(float x, int dir) {
  uint32_t u;
  memcpy(&u, &x, 4);
  uint32_t sign = u >> 31;
  uint32_t a = u & 0x7fffffffu;
  if (a > 0x7f800000u) return 0x7e00;
  if (a == 0) return (uint16_t)(sign << 15);
  /* round the magnitude away from zero iff the direction points away from zero */
  int away = (dir > 0 && !sign) || (dir < 0 && sign);
  int32_t e = (int32_t)(a >> 23) - 127;
  uint32_t mant = a & 0x7fffffu;
  uint32_t hm;      /* magnitude bits, truncated */
  int inexact;
  if (a == 0x7f800000u) { hm = 0x7c00; inexact = 0; }
  else if (e > 15) { hm = 0x7bff; inexact = 1; }
  else if (e >= -14) {
    hm = ((uint32_t)(e + 15) << 10) | (mant >> 13);
    inexact = (mant & 0x1fffu) != 0;
  } else {
    uint32_t M = mant | 0x800000u;       /* value = M * 2^(e-23); unit = 2^-24 */
    int shift = -e - 1;                  /* hm = floor(M * 2^(e+1)) */
    if (e == -127) { M = mant; shift = 125; } /* fp32 subnormal input */
    if (shift >= 32) { hm = 0; inexact = 1; }
    else { hm = M >> shift; inexact = (M & ((1u << shift) - 1u)) != 0; }
  }
  if (inexact && away) hm += 1;          /* carries into the exponent, up to inf */
  return (uint16_t)((sign << 15) | hm);
}

uint16_t qpo_f32_to_f16_down(float x) { return f32_to_f16_dir(x, -1); }
uint16_t qpo_f32_to_f16_up(float x) { return f32_to_f16_dir(x, +1); }
float qpo_f16_to_f32(uint16_t h) { return f16_to_f32(h); }

int qpo_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ---------- budget (Appendix B "Memory Budgets"; Fig. 2 caption) ---------- */

/* tokens x bits is held constant: n = budget_bits / bits, capped at L.  The
 * kept tokens include the w observation-window tokens.  Returns -1 when the
 * budget cannot be met (n <= w, or n not a whole number of quantization
 * groups). */
int64_t qpo_n_keep(int64_t budget_bits, int bits, int group, int L, int w) {
  if (bits != 2 && bits != 4 && bits != 8 && bits != 16) return -1;
  int64_t n = budget_bits / bits;
  if (n > L) n = L;
  if (n <= w) return -1;
  if (bits < 16 && n % group != 0) return -1;
  return n;
}

/* ---------- S1: observation-window scores --------------------------------- */
/*
 * Reading of "SnapKV" used by this build (the paper only names the method,
 * Sec. 4 "Setup" and Appendix B):
 *   for every query head h of the KV head's group and every window row i
 *   (absolute position p = P + i, P = L - w):
 *       S[j]  = (sum_d Q[h,i,d] * K[j,d]) / sqrt(D),  j = 0..p   (causal)
 *       Pr[j] = softmax over j = 0..p
 *   vote[j]   = sum_h sum_i Pr_{h,i}[j]            for prefix columns j < P
 *   pooled[j] = (sum_{|t| <= r} vote[j+t] [0 <= j+t < P]) / pool,  r = (pool-1)/2
 *
 * Layouts: Qwin [Bt,Hq,w,D], K [Bt,Hkv,L,D] (bf16 bit patterns);
 * votes, pooled [Bt,Hkv,P] fp64 (votes may be NULL).
 */
void qpo_scores(const uint16_t* Qwin, const uint16_t* K, int Bt, int Hq, int Hkv, int D, int L,
                int w, int pool, double* pooled, double* votes) {
  const int G = Hq / Hkv, P = L - w, r = (pool - 1) / 2;
  const double inv_sqrt_d = 1.0 / sqrt((double)D);
#pragma omp parallel for schedule(dynamic)
  for (int bh = 0; bh < Bt * Hkv; ++bh) {
    const int b = bh / Hkv, hk = bh % Hkv;
    const uint16_t* Kh = K + (size_t)bh * L * D;
    double* S = (double*)malloc(sizeof(double) * (size_t)L);
    double* vote = (double*)calloc((size_t)P, sizeof(double));
    for (int g = 0; g < G; ++g) {
      const int h = hk * G + g;
      for (int i = 0; i < w; ++i) {
        const uint16_t* q = Qwin + (((size_t)b * Hq + h) * w + i) * D;
        const int p = P + i;
        double mx = -INFINITY;
        for (int j = 0; j <= p; ++j) {
          double acc = 0.0;
          for (int d = 0; d < D; ++d)
            acc += (double)bf16_to_f32(q[d]) * (double)bf16_to_f32(Kh[(size_t)j * D + d]);
          S[j] = acc * inv_sqrt_d;
          if (S[j] > mx) mx = S[j];
        }
        double Z = 0.0;
        for (int j = 0; j <= p; ++j) Z += exp(S[j] - mx);
        for (int j = 0; j < P; ++j) vote[j] += exp(S[j] - mx) / Z;
      }
    }
    double* out = pooled + (size_t)bh * P;
    for (int j = 0; j < P; ++j) {
      double acc = 0.0;
      for (int t = -r; t <= r; ++t)
        if (j + t >= 0 && j + t < P) acc += vote[j + t];
      out[j] = acc / (double)pool;
    }
    if (votes) memcpy(votes + (size_t)bh * P, vote, sizeof(double) * (size_t)P);
    free(S);
    free(vote);
  }
}

/* ---------- S2: per-head top-k -------------------------------------------- */

typedef struct { double s; int32_t j; } qpo_item;

static int cmp_item(const void* a, const void* b) {
  const qpo_item* x = (const qpo_item*)a;
  const qpo_item* y = (const qpo_item*)b;
  if (x->s > y->s) return -1;        /* larger score first */
  if (x->s < y->s) return 1;
  return (x->j > y->j) - (x->j < y->j); /* equal scores: lower index first */
}

static int cmp_i32(const void* a, const void* b) {
  int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
  return (x > y) - (x < y);
}

/* "KV Pruning": choose n_keep < L tokens per head.  The k = n_keep - w prefix
 * positions with the largest pooled score are kept (ties: lowest index), the w
 * window positions P..L-1 are always kept; output sorted ascending.
 * pooled [Bt,Hkv,P] -> kept [Bt,Hkv,n_keep]. */
void qpo_select(const double* pooled, int Bt, int Hkv, int L, int w, int n_keep, int32_t* kept) {
  const int P = L - w, k = n_keep - w;
#pragma omp parallel for schedule(dynamic)
  for (int bh = 0; bh < Bt * Hkv; ++bh) {
    qpo_item* it = (qpo_item*)malloc(sizeof(qpo_item) * (size_t)(P > 0 ? P : 1));
    for (int j = 0; j < P; ++j) { it[j].s = pooled[(size_t)bh * P + j]; it[j].j = j; }
    qsort(it, (size_t)P, sizeof(qpo_item), cmp_item);
    int32_t* o = kept + (size_t)bh * n_keep;
    for (int t = 0; t < k; ++t) o[t] = it[t].j;
    qsort(o, (size_t)k, sizeof(int32_t), cmp_i32);
    for (int i = 0; i < w; ++i) o[k + i] = P + i;
    free(it);
  }
}

/* ---------- S3: gather + quantize + pack ---------------------------------- */

/* One quantization group (Eq. 4), fp32 in this exact order:
 *   mn, mx exact; z16 = fp16 round-down(mn); zf = float(z16);
 *   range = mx - zf; s32 = range / (2^b - 1); s16 = fp16 round-up(s32);
 *   sf = float(s16); code = clamp(rint((x - zf)/sf), 0, 2^b - 1), 0 if sf == 0.
 * x points at the first element, consecutive elements are `stride` apart. */
static void quant_group_thr(const float* x, int stride, int g, int bits, float thr, uint32_t* codes,
                            uint16_t* s16_out, uint16_t* z16_out) {
  /* thr: elements with |x| > thr are outliers (Sec. 5.3 "Quantization methods", Appendix B: numbers whose
   * absolute value exceeds 6 are excluded from quantization).  They take no part in min/max, get code 0 and
   * are kept exactly elsewhere.  thr = +inf: no filtering.  A group made of outliers only has z = s = 0. */
  float mn = 0.0f, mx = 0.0f;
  int seen = 0;
  for (int e = 0; e < g; ++e) {
    float v = x[(size_t)e * stride];
    if (fabsf(v) > thr) continue;
    if (!seen || v < mn) mn = v;
    if (!seen || v > mx) mx = v;
    seen = 1;
  }
  const int qmax = (1 << bits) - 1;
  uint16_t z16 = f32_to_f16_dir(mn, -1);
  volatile float zf = f16_to_f32(z16);
  volatile float range = mx - zf;
  volatile float s32 = range / (float)qmax;
  uint16_t s16 = f32_to_f16_dir(s32, +1);
  volatile float sf = f16_to_f32(s16);
  for (int e = 0; e < g; ++e) {
    uint32_t c = 0;
    if (sf != 0.0f && !(fabsf(x[(size_t)e * stride]) > thr)) {
      volatile float diff = x[(size_t)e * stride] - zf;
      volatile float qf = diff / sf;
      float rf = rintf(qf);                 /* round half to even */
      if (rf < 0.0f) rf = 0.0f;
      if (rf > (float)qmax) rf = (float)qmax;
      c = (uint32_t)rf;
    }
    codes[e] = c;
  }
  *s16_out = s16;
  *z16_out = z16;
}

static void quant_group(const float* x, int stride, int g, int bits, uint32_t* codes,
                        uint16_t* s16_out, uint16_t* z16_out) {
  quant_group_thr(x, stride, g, bits, INFINITY, codes, s16_out, z16_out);
}

/* element e of a group -> word e / (32/b), bit offset (e mod (32/b)) * b */
static void pack_group(const uint32_t* codes, int g, int bits, uint32_t* words) {
  const int per = 32 / bits;
  for (int wd = 0; wd < g * bits / 32; ++wd) words[wd] = 0;
  for (int e = 0; e < g; ++e) words[e / per] |= codes[e] << ((e % per) * bits);
}

/*
 * "Quantized Pruning": gather the kept rows, then quantize them.
 * K groups: fixed channel d, g consecutive *kept* tokens (per-channel);
 * V groups: fixed kept token, g consecutive channels (per-token).
 * Layouts (n = n_keep, wpg = g*bits/32 words per group):
 *   Kc [Bt,Hkv,n/g,D,wpg] u32, Ks,Kz [Bt,Hkv,n/g,D] fp16
 *   Vc [Bt,Hkv,n,D/g,wpg] u32, Vs,Vz [Bt,Hkv,n,D/g] fp16
 * bits == 16: Kc, Vc receive the gathered bf16 rows [Bt,Hkv,n,D] unchanged
 * (as uint16) and the scale/zero arrays are not touched.
 */
void qpo_quantize(const uint16_t* K, const uint16_t* V, const int32_t* kept, int Bt, int Hkv,
                  int D, int L, int n, int bits, int g, void* Kc_, uint16_t* Ks, uint16_t* Kz,
                  void* Vc_, uint16_t* Vs, uint16_t* Vz) {
#pragma omp parallel for schedule(dynamic)
  for (int bh = 0; bh < Bt * Hkv; ++bh) {
    const uint16_t* Kh = K + (size_t)bh * L * D;
    const uint16_t* Vh = V + (size_t)bh * L * D;
    const int32_t* idx = kept + (size_t)bh * n;
    if (bits == 16) {
      uint16_t* Ko = (uint16_t*)Kc_ + (size_t)bh * n * D;
      uint16_t* Vo = (uint16_t*)Vc_ + (size_t)bh * n * D;
      for (int t = 0; t < n; ++t) {
        memcpy(Ko + (size_t)t * D, Kh + (size_t)idx[t] * D, sizeof(uint16_t) * (size_t)D);
        memcpy(Vo + (size_t)t * D, Vh + (size_t)idx[t] * D, sizeof(uint16_t) * (size_t)D);
      }
      continue;
    }
    const int wpg = g * bits / 32;
    float* Ke = (float*)malloc(sizeof(float) * (size_t)n * D);
    float* Ve = (float*)malloc(sizeof(float) * (size_t)n * D);
    uint32_t* codes = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)g);
    for (int t = 0; t < n; ++t)
      for (int d = 0; d < D; ++d) {
        Ke[(size_t)t * D + d] = bf16_to_f32(Kh[(size_t)idx[t] * D + d]);
        Ve[(size_t)t * D + d] = bf16_to_f32(Vh[(size_t)idx[t] * D + d]);
      }
    uint32_t* Kc = (uint32_t*)Kc_ + (size_t)bh * (n / g) * D * wpg;
    uint32_t* Vc = (uint32_t*)Vc_ + (size_t)bh * n * (D / g) * wpg;
    for (int u = 0; u < n / g; ++u)
      for (int d = 0; d < D; ++d) {
        size_t gi = (size_t)u * D + d;
        quant_group(Ke + (size_t)u * g * D + d, D, g, bits, codes,
                    Ks + (size_t)bh * (n / g) * D + gi, Kz + (size_t)bh * (n / g) * D + gi);
        pack_group(codes, g, bits, Kc + gi * wpg);
      }
    for (int t = 0; t < n; ++t)
      for (int v = 0; v < D / g; ++v) {
        size_t gi = (size_t)t * (D / g) + v;
        quant_group(Ve + (size_t)t * D + (size_t)v * g, 1, g, bits, codes,
                    Vs + (size_t)bh * n * (D / g) + gi, Vz + (size_t)bh * n * (D / g) + gi);
        pack_group(codes, g, bits, Vc + gi * wpg);
      }
    free(Ke);
    free(Ve);
    free(codes);
  }
}

/* ---------- dequantize (Eq. 5) -------------------------------------------- */

/* X' = code * s + z in fp64 from the stored fp16 scale/zero.
 * Outputs Kd, Vd [Bt,Hkv,n,D] fp64.  bits == 16: the stored bf16 values. */
void qpo_dequantize(const void* Kc_, const uint16_t* Ks, const uint16_t* Kz, const void* Vc_,
                    const uint16_t* Vs, const uint16_t* Vz, int Bt, int Hkv, int D, int n,
                    int bits, int g, double* Kd, double* Vd) {
  const size_t tot = (size_t)Bt * Hkv * n * D;
  if (bits == 16) {
    for (size_t i = 0; i < tot; ++i) {
      Kd[i] = (double)bf16_to_f32(((const uint16_t*)Kc_)[i]);
      Vd[i] = (double)bf16_to_f32(((const uint16_t*)Vc_)[i]);
    }
    return;
  }
  const int per = 32 / bits, wpg = g * bits / 32;
  const uint32_t mask = (1u << bits) - 1u;
  const uint32_t* Kc = (const uint32_t*)Kc_;
  const uint32_t* Vc = (const uint32_t*)Vc_;
  for (int bh = 0; bh < Bt * Hkv; ++bh)
    for (int t = 0; t < n; ++t)
      for (int d = 0; d < D; ++d) {
        size_t o = ((size_t)bh * n + t) * D + d;
        { /* key: group (u = t / g, channel d), element e = t mod g */
          size_t gi = ((size_t)bh * (n / g) + t / g) * D + d;
          int e = t % g;
          uint32_t c = (Kc[gi * wpg + e / per] >> ((e % per) * bits)) & mask;
          Kd[o] = (double)c * (double)f16_to_f32(Ks[gi]) + (double)f16_to_f32(Kz[gi]);
        }
        { /* value: group (token t, v = d / g), element e = d mod g */
          size_t gi = ((size_t)bh * n + t) * (D / g) + d / g;
          int e = d % g;
          uint32_t c = (Vc[gi * wpg + e / per] >> ((e % per) * bits)) & mask;
          Vd[o] = (double)c * (double)f16_to_f32(Vs[gi]) + (double)f16_to_f32(Vz[gi]);
        }
      }
}

/* ---------- S4/S5: decode attention (Eq. 3 on the dequantized cache) ------- */

/* q [Bt,Hq,D] bf16; Kd,Vd [Bt,Hkv,n,D] fp64 (from qpo_dequantize);
 * out [Bt,Hq,D] fp64.  Logits are scaled by 1/sqrt(D); softmax over all n
 * kept tokens, no mask. */
void qpo_decode(const uint16_t* q, const double* Kd, const double* Vd, int Bt, int Hq, int Hkv,
                int D, int n, double* out) {
  const int G = Hq / Hkv;
  const double inv_sqrt_d = 1.0 / sqrt((double)D);
#pragma omp parallel for schedule(dynamic)
  for (int bh = 0; bh < Bt * Hkv; ++bh) {
    const int b = bh / Hkv, hk = bh % Hkv;
    const double* Kh = Kd + (size_t)bh * n * D;
    const double* Vh = Vd + (size_t)bh * n * D;
    double* a = (double*)malloc(sizeof(double) * (size_t)n);
    for (int g = 0; g < G; ++g) {
      const int h = hk * G + g;
      const uint16_t* qh = q + ((size_t)b * Hq + h) * D;
      double mx = -INFINITY;
      for (int t = 0; t < n; ++t) {
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += (double)bf16_to_f32(qh[d]) * Kh[(size_t)t * D + d];
        a[t] = acc * inv_sqrt_d;
        if (a[t] > mx) mx = a[t];
      }
      double Z = 0.0;
      for (int t = 0; t < n; ++t) { a[t] = exp(a[t] - mx); Z += a[t]; }
      double* o = out + ((size_t)b * Hq + h) * D;
      for (int d = 0; d < D; ++d) {
        double acc = 0.0;
        for (int t = 0; t < n; ++t) acc += (a[t] / Z) * Vh[(size_t)t * D + d];
        o[d] = acc;
      }
    }
    free(a);
  }
}

/* ---------- other quantization strategies of the ablation (Sec. 5.3 "Quantization methods") ----------- */
/*
 * k_axis = 0: keys per channel over g kept tokens (KIVI, as qpo_quantize).
 * k_axis = 1: keys grouped like the values, g consecutive channels of one token ("FlexGen": both caches
 *             quantized along the token dimension, i.e. token by token; Sec. 5.3).  Layout then
 *             Kc [Bt,Hkv,n,D/g,wpg], Ks,Kz [Bt,Hkv,n,D/g].
 * thr: outlier threshold (Appendix B: |x| > 6 is excluded from quantization); +inf = no filtering.
 * Outliers of a (batch, KV head) are listed in ascending order of t*D + d (t = index among the kept
 * tokens): side_idx [Bt*Hkv, cap] int32, side_val [Bt*Hkv, cap] bf16 bits, side_cnt [Bt*Hkv]
 * (-1 if more than cap).  One list for keys, one for values.  bits < 16 only.
 */
void qpo_quantize_ex(const uint16_t* K, const uint16_t* V, const int32_t* kept, int Bt, int Hkv,
                     int D, int L, int n, int bits, int g, int k_axis, float thr, uint32_t* Kc,
                     uint16_t* Ks, uint16_t* Kz, uint32_t* Vc, uint16_t* Vs, uint16_t* Vz,
                     int32_t* k_side_idx, uint16_t* k_side_val, int32_t* k_side_cnt,
                     int32_t* v_side_idx, uint16_t* v_side_val, int32_t* v_side_cnt, int cap) {
#pragma omp parallel for schedule(dynamic)
  for (int bh = 0; bh < Bt * Hkv; ++bh) {
    const uint16_t* Kh = K + (size_t)bh * L * D;
    const uint16_t* Vh = V + (size_t)bh * L * D;
    const int32_t* idx = kept + (size_t)bh * n;
    const int wpg = g * bits / 32;
    float* Ke = (float*)malloc(sizeof(float) * (size_t)n * D);
    float* Ve = (float*)malloc(sizeof(float) * (size_t)n * D);
    uint32_t* codes = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)g);
    int kc = 0, vc = 0;
    for (int t = 0; t < n; ++t)
      for (int d = 0; d < D; ++d) {
        const uint16_t kb = Kh[(size_t)idx[t] * D + d], vb = Vh[(size_t)idx[t] * D + d];
        Ke[(size_t)t * D + d] = bf16_to_f32(kb);
        Ve[(size_t)t * D + d] = bf16_to_f32(vb);
        if (fabsf(bf16_to_f32(kb)) > thr) {              /* ascending t*D + d by construction */
          if (kc < cap) { k_side_idx[(size_t)bh * cap + kc] = t * D + d; k_side_val[(size_t)bh * cap + kc] = kb; }
          ++kc;
        }
        if (fabsf(bf16_to_f32(vb)) > thr) {
          if (vc < cap) { v_side_idx[(size_t)bh * cap + vc] = t * D + d; v_side_val[(size_t)bh * cap + vc] = vb; }
          ++vc;
        }
      }
    if (k_side_cnt) k_side_cnt[bh] = kc <= cap ? kc : -1;
    if (v_side_cnt) v_side_cnt[bh] = vc <= cap ? vc : -1;
    if (k_axis == 0) {
      uint32_t* Kcb = Kc + (size_t)bh * (n / g) * D * wpg;
      for (int u = 0; u < n / g; ++u)
        for (int d = 0; d < D; ++d) {
          size_t gi = (size_t)u * D + d;
          quant_group_thr(Ke + (size_t)u * g * D + d, D, g, bits, thr, codes,
                          Ks + (size_t)bh * (n / g) * D + gi, Kz + (size_t)bh * (n / g) * D + gi);
          pack_group(codes, g, bits, Kcb + gi * wpg);
        }
    } else {
      uint32_t* Kcb = Kc + (size_t)bh * n * (D / g) * wpg;
      for (int t = 0; t < n; ++t)
        for (int v = 0; v < D / g; ++v) {
          size_t gi = (size_t)t * (D / g) + v;
          quant_group_thr(Ke + (size_t)t * D + (size_t)v * g, 1, g, bits, thr, codes,
                          Ks + (size_t)bh * n * (D / g) + gi, Kz + (size_t)bh * n * (D / g) + gi);
          pack_group(codes, g, bits, Kcb + gi * wpg);
        }
    }
    uint32_t* Vcb = Vc + (size_t)bh * n * (D / g) * wpg;
    for (int t = 0; t < n; ++t)
      for (int v = 0; v < D / g; ++v) {
        size_t gi = (size_t)t * (D / g) + v;
        quant_group_thr(Ve + (size_t)t * D + (size_t)v * g, 1, g, bits, thr, codes,
                        Vs + (size_t)bh * n * (D / g) + gi, Vz + (size_t)bh * n * (D / g) + gi);
        pack_group(codes, g, bits, Vcb + gi * wpg);
      }
    free(Ke);
    free(Ve);
    free(codes);
  }
}

/* Eq. 5 for the layouts of qpo_quantize_ex; a listed outlier is reconstructed as its stored 16-bit value. */
void qpo_dequantize_ex(const uint32_t* Kc, const uint16_t* Ks, const uint16_t* Kz, const uint32_t* Vc,
                       const uint16_t* Vs, const uint16_t* Vz, int Bt, int Hkv, int D, int n, int bits,
                       int g, int k_axis, const int32_t* k_side_idx, const uint16_t* k_side_val,
                       const int32_t* k_side_cnt, const int32_t* v_side_idx, const uint16_t* v_side_val,
                       const int32_t* v_side_cnt, int cap, double* Kd, double* Vd) {
  const int per = 32 / bits, wpg = g * bits / 32;
  const uint32_t mask = (1u << bits) - 1u;
  for (int bh = 0; bh < Bt * Hkv; ++bh) {
    for (int t = 0; t < n; ++t)
      for (int d = 0; d < D; ++d) {
        size_t o = ((size_t)bh * n + t) * D + d;
        {
          size_t gi;
          int e;
          if (k_axis == 0) { gi = ((size_t)bh * (n / g) + t / g) * D + d; e = t % g; }
          else { gi = ((size_t)bh * n + t) * (D / g) + d / g; e = d % g; }
          uint32_t c = (Kc[gi * wpg + e / per] >> ((e % per) * bits)) & mask;
          Kd[o] = (double)c * (double)f16_to_f32(Ks[gi]) + (double)f16_to_f32(Kz[gi]);
        }
        {
          size_t gi = ((size_t)bh * n + t) * (D / g) + d / g;
          int e = d % g;
          uint32_t c = (Vc[gi * wpg + e / per] >> ((e % per) * bits)) & mask;
          Vd[o] = (double)c * (double)f16_to_f32(Vs[gi]) + (double)f16_to_f32(Vz[gi]);
        }
      }
    if (k_side_cnt)
      for (int i = 0; i < k_side_cnt[bh]; ++i)
        Kd[(size_t)bh * n * D + k_side_idx[(size_t)bh * cap + i]] = (double)bf16_to_f32(k_side_val[(size_t)bh * cap + i]);
    if (v_side_cnt)
      for (int i = 0; i < v_side_cnt[bh]; ++i)
        Vd[(size_t)bh * n * D + v_side_idx[(size_t)bh * cap + i]] = (double)bf16_to_f32(v_side_val[(size_t)bh * cap + i]);
  }
}
