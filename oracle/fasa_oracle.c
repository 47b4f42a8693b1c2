/*
 * FASA decode-path oracle: a plain, slow, fp64 CPU statement of what the method
 * computes.  TEST INFRASTRUCTURE ONLY: tests, the smoke check and the CPU-baseline
 * leg of the benchmark may call it; the product path never does.  It shares no
 * code, header, table or helper with the CUDA library.
 *
 * Every function follows one passage of the paper (arxiv 2602.03152):
 *   - RoPE as d/2 two-dimensional frequency chunks (FCs), FC i turning by
 *     m*theta_i at position m, theta_i = B^(-2i/d) with 0-based i  (Sec. 3.1, Eq. 1)
 *   - single-FC raw scores alpha^(i) and full-head raw scores alpha (Sec. 3.3, Eq. 2-3)
 *   - importance score S_t = sum over the dominant FCs of alpha^(i)   (Sec. 4.1, TIP)
 *   - T_t = TopK-I(S_t, N_fac)                                       (Sec. 4.1)
 *   - Gather + Softmax(q K_T^T / sqrt(d)) V_T                         (Sec. 4.2, Eq. 6-7)
 *   - full-KV attention (the FKV baseline)                            (Sec. 5.1)
 *   - contextual agreement CA of a single FC with the full head, and the
 *     offline choice of the dominant FCs from its mean          (Sec. 3.3, Eq. 4; Algorithm 1)
 *
 * Readings taken where the paper is silent (each is listed in the design notes):
 *   FC channel pairing is selectable: 0 = rotate-half (i, i+d/2), 1 = interleaved
 *   (2i, 2i+1, the paper's literal Eq. 1).  With grouped-query attention the
 *   score of a KV head is the sum (or max) over its query heads of the raw
 *   partial logits.  Ties rank the lower index first.  Sink / recent positions
 *   are kept in addition to the budget.  The paper keeps one index set per
 *   (layer, head) (Sec. 4.1); how many query heads share a set is a parameter
 *   here: all heads of a KV head (the default, one gathered set per K/V head),
 *   one (the per-head reading), or any divisor of the group in between.
 *
 * Pins (tests/test_oracle_*.py): sum over all FCs of alpha^(i) equals q.k;
 * the relative-position identity; F = d/2 reproduces the dense top-k; budget >=
 * context reproduces dense attention; library matmul / top-k / SDPA in fp64;
 * hand-worked small cases under tests/golden/.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ bf16 */

/* bf16 is the upper half of an IEEE binary32: widening is exact. */
double fasa_oracle_bf16_to_f64(uint16_t bits) {
  uint32_t u = ((uint32_t)bits) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* Round-to-nearest-even from binary32 bits to bf16 bits (NaN kept quiet). */
uint16_t fasa_oracle_f32_to_bf16(float f) {
  uint32_t u;
  memcpy(&u, &f, sizeof u);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return (uint16_t)(u >> 16);
}

void fasa_oracle_widen_bf16(const uint16_t* bits, int64_t n, double* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = fasa_oracle_bf16_to_f64(bits[i]);
}

/* ------------------------------------------------------------------ FCs */

/* The two channels that make up FC i of a d-dimensional head. */
static void fc_channels(int i, int d, int pairing, int* c0, int* c1) {
  if (pairing == 0) { *c0 = i;     *c1 = i + d / 2; }
  else              { *c0 = 2 * i; *c1 = 2 * i + 1; }
}

/* theta_i = B^(-2i/d), i = 0 .. d/2-1: low i turns fast (Sec. 3.1). */
double fasa_oracle_theta(int i, int d, double base) {
  return pow(base, -2.0 * (double)i / (double)d);
}

/* Eq. 1: FC i of x at position m is turned by the 2x2 rotation R_{m,theta_i}
 *   (x0, x1) -> (x0 cos - x1 sin, x0 sin + x1 cos),  angle = m * theta_i. */
void fasa_oracle_rope(const double* x, int d, double pos, double base, int pairing,
                      double* out) {
  for (int i = 0; i < d / 2; ++i) {
    int c0, c1;
    fc_channels(i, d, pairing, &c0, &c1);
    double ang = pos * fasa_oracle_theta(i, d, base);
    double c = cos(ang), s = sin(ang);
    double x0 = x[c0], x1 = x[c1];
    out[c0] = x0 * c - x1 * s;
    out[c1] = x0 * s + x1 * c;
  }
}

/* Eq. 3 on post-RoPE vectors: alpha^(i)[j] = q^[i] . k_j^[i]  (two products).
 * a is [d/2][L]. */
void fasa_oracle_fc_partial_logits(const double* q, const double* K, int L, int d,
                                   int pairing, double* a) {
  for (int i = 0; i < d / 2; ++i) {
    int c0, c1;
    fc_channels(i, d, pairing, &c0, &c1);
    for (int j = 0; j < L; ++j)
      a[(int64_t)i * L + j] = q[c0] * K[(int64_t)j * d + c0] + q[c1] * K[(int64_t)j * d + c1];
  }
}

/* TIP (Sec. 4.1): S[j] = reduce over the group's query heads g of
 *   sum_{i in I_dom} alpha^(i)_g[j];  reduce = sum (0) or max (1).
 * q is [G][d]; dom holds F distinct FC indices.  No scaling, no softmax. */
void fasa_oracle_fc_score(const double* q, int G, const double* K, int L, int d,
                          int pairing, const int* dom, int F, int group_reduce,
                          double* S) {
  for (int j = 0; j < L; ++j) {
    double red = 0.0;
    for (int g = 0; g < G; ++g) {
      double s = 0.0;
      for (int r = 0; r < F; ++r) {
        int c0, c1;
        fc_channels(dom[r], d, pairing, &c0, &c1);
        s += q[g * d + c0] * K[(int64_t)j * d + c0] + q[g * d + c1] * K[(int64_t)j * d + c1];
      }
      if (g == 0) red = s;
      else if (group_reduce == 0) red += s;
      else if (s > red) red = s;
    }
    S[j] = red;
  }
}

/* ------------------------------------------------------------ selection */

typedef struct { double s; int j; } ranked_t;

static int rank_cmp(const void* pa, const void* pb) {
  const ranked_t* a = (const ranked_t*)pa;
  const ranked_t* b = (const ranked_t*)pb;
  if (a->s > b->s) return -1;
  if (a->s < b->s) return 1;
  return (a->j > b->j) - (a->j < b->j);
}

static int int_cmp(const void* pa, const void* pb) {
  int a = *(const int*)pa, b = *(const int*)pb;
  return (a > b) - (a < b);
}

/* T = forced  U  TopK-I(S restricted to the other positions, k)   (Sec. 4.1).
 * forced = the first n_sink and the last n_recent positions.  Ranking: higher
 * score first, then lower index.  idx_out (capacity >= L) receives the set in
 * ascending order; the return value is its size min(L, |forced| + k).
 *
 * band[0..3] describes the boundary for the parity rule: with s_k and s_k1 the
 * last kept and first dropped ranked scores,
 *   band[0] = 1 if both exist, band[1] = s_k, band[2] = s_k1,
 *   band[3] = 1 if (s_k - s_k1) <= tie_rel * max(|s_k|, |s_k1|)  (a tie band). */
int fasa_oracle_select(const double* S, int L, int k, int n_sink, int n_recent,
                       double tie_rel, int* idx_out, double* band) {
  band[0] = band[1] = band[2] = band[3] = 0.0;
  if (L <= 0) return 0;
  if (k < 0) k = 0;
  ranked_t* r = (ranked_t*)malloc(sizeof(ranked_t) * (size_t)L);
  int n = 0, m = 0;
  for (int j = 0; j < L; ++j) {
    int forced = (j < n_sink) || (j >= L - n_recent);
    if (forced) idx_out[n++] = j;
    else { r[m].s = S[j]; r[m].j = j; ++m; }
  }
  qsort(r, (size_t)m, sizeof(ranked_t), rank_cmp);
  int take = k < m ? k : m;
  for (int t = 0; t < take; ++t) idx_out[n++] = r[t].j;
  if (take > 0 && take < m) {
    double sk = r[take - 1].s, sk1 = r[take].s;
    double mag = fmax(fabs(sk), fabs(sk1));
    band[0] = 1.0; band[1] = sk; band[2] = sk1;
    band[3] = ((sk - sk1) <= tie_rel * mag) ? 1.0 : 0.0;
  }
  free(r);
  qsort(idx_out, (size_t)n, sizeof(int), int_cmp);
  return n;
}

/* ------------------------------------------------------------ attention */

/* Eq. 6-7 for one KV head and its G query heads:
 *   l_j = (q_g . K[idx_j]) * scale over all d channels,  p = softmax(l),
 *   O_g = sum_j p_j V[idx_j].  Rows are used as stored (positions preserved).
 * lse (nullable) receives log(sum_j exp(l_j)).  n == 0 gives O = 0, lse = -inf. */
void fasa_oracle_attn_subset(const double* q, int G, const double* K, const double* V,
                             int d, const int* idx, int n, double scale, double* O,
                             double* lse) {
  double* l = (double*)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
  for (int g = 0; g < G; ++g) {
    for (int c = 0; c < d; ++c) O[g * d + c] = 0.0;
    if (n <= 0) { if (lse) lse[g] = -INFINITY; continue; }
    double mx = -INFINITY;
    for (int t = 0; t < n; ++t) {
      const double* kr = K + (int64_t)idx[t] * d;
      double s = 0.0;
      for (int c = 0; c < d; ++c) s += q[g * d + c] * kr[c];
      l[t] = s * scale;
      if (l[t] > mx) mx = l[t];
    }
    double den = 0.0;
    for (int t = 0; t < n; ++t) { l[t] = exp(l[t] - mx); den += l[t]; }
    for (int t = 0; t < n; ++t) {
      const double* vr = V + (int64_t)idx[t] * d;
      double p = l[t] / den;
      for (int c = 0; c < d; ++c) O[g * d + c] += p * vr[c];
    }
    if (lse) lse[g] = mx + log(den);
  }
  free(l);
}

/* FKV (Sec. 5.1): the same over every cached row 0..L-1. */
void fasa_oracle_attn_dense(const double* q, int G, const double* K, const double* V,
                            int d, int L, double scale, double* O, double* lse) {
  int* idx = (int*)malloc(sizeof(int) * (size_t)(L > 0 ? L : 1));
  for (int j = 0; j < L; ++j) idx[j] = j;
  fasa_oracle_attn_subset(q, G, K, V, d, idx, L, scale, O, lse);
  free(idx);
}

/* ------------------------------------------------------------ calibration */

/* CA (Sec. 3.3, Eq. 4) of every FC for one query head: counts[i] =
 * | TopK-I(alpha, top_k)  intersected with  TopK-I(alpha^(i), top_k) |, i.e. CA times top_k.
 * alpha^(i) are the single-FC raw scores (Eq. 3) and alpha their sum over all FCs, the
 * full-head raw scores (Eq. 2).  TopK-I ranks as everywhere here: higher score first,
 * then lower index.
 * Which index enters a top-k set is an integer decided by floating point, so it is
 * taken in the precision of the path being checked when f32 != 0: each product in
 * binary32 (exact for bf16 inputs), alpha^(i) = their binary32 sum, alpha = the
 * binary32 sum of alpha^(0), alpha^(1), ... in this order.  f32 == 0 is the plain
 * fp64 statement. */
void fasa_oracle_ca_counts(const double* q, const double* K, int L, int d, int pairing,
                           int top_k, int f32, int* counts) {
  int n_fc = d / 2;
  size_t rows = (size_t)(L > 0 ? L : 1);
  double* a = (double*)malloc(sizeof(double) * (size_t)n_fc * rows);
  double* full = (double*)malloc(sizeof(double) * rows);
  int* t_full = (int*)malloc(sizeof(int) * rows);
  int* t_fc = (int*)malloc(sizeof(int) * rows);
  double band[4];
  for (int j = 0; j < L; ++j) {
    double acc = 0.0;
    float acc32 = 0.0f;
    for (int i = 0; i < n_fc; ++i) {
      int c0, c1;
      fc_channels(i, d, pairing, &c0, &c1);
      double p0 = q[c0] * K[(int64_t)j * d + c0], p1 = q[c1] * K[(int64_t)j * d + c1];
      if (f32) {
        volatile float s32 = (float)p0 + (float)p1;   /* one binary32 rounding */
        volatile float t32 = acc32 + s32;
        acc32 = t32;
        a[(int64_t)i * L + j] = (double)s32;
      } else {
        a[(int64_t)i * L + j] = p0 + p1;
        acc += p0 + p1;
      }
    }
    full[j] = f32 ? (double)acc32 : acc;
  }
  int n_full = fasa_oracle_select(full, L, top_k, 0, 0, 0.0, t_full, band);
  for (int i = 0; i < n_fc; ++i) {
    int n_i = fasa_oracle_select(a + (int64_t)i * L, L, top_k, 0, 0, 0.0, t_fc, band);
    int x = 0, y = 0, common = 0;          /* both lists ascending */
    while (x < n_full && y < n_i) {
      if (t_full[x] == t_fc[y]) { ++common; ++x; ++y; }
      else if (t_full[x] < t_fc[y]) ++x;
      else ++y;
    }
    counts[i] = common;
  }
  free(a); free(full); free(t_full); free(t_fc);
}

/* Stage 1 of Algorithm 1 over a batch of bf16 tensors laid out as in the decode
 * step: a sample is a (sequence b, query head g) pair whose sequence is longer
 * than top_k (a shorter one selects every position and says nothing).  Adds each
 * sample's counts to counts[g][i] ([Hq][d/2]) and 1 to n_used[g] ([Hq]).
 * Returns the number of threads used. */
int fasa_oracle_calibrate_bf16(const uint16_t* q_bits, const uint16_t* K_bits,
                               const int32_t* seq_lens, int B, int Hq, int Hkv, int d,
                               int Lmax, int pairing, int top_k, int f32, int n_threads,
                               int64_t* counts, int64_t* n_used) {
  int group = Hq / Hkv, n_fc = d / 2;
  int used = 1;
#ifdef _OPENMP
  if (n_threads > 0) omp_set_num_threads(n_threads);
  used = n_threads > 0 ? n_threads : omp_get_max_threads();
  if (used > B * Hq) used = B * Hq;
#pragma omp parallel for schedule(dynamic, 1)
#endif
  for (int u = 0; u < B * Hq; ++u) {
    int b = u / Hq, g = u % Hq, h = g / group;
    int L = seq_lens[b];
    if (L > Lmax) L = Lmax;
    if (L <= top_k) continue;
    double* Kd = (double*)malloc(sizeof(double) * (size_t)L * (size_t)d);
    double* qd = (double*)malloc(sizeof(double) * (size_t)d);
    int* c = (int*)malloc(sizeof(int) * (size_t)n_fc);
    fasa_oracle_widen_bf16(K_bits + ((int64_t)b * Hkv + h) * (int64_t)Lmax * d, (int64_t)L * d, Kd);
    fasa_oracle_widen_bf16(q_bits + ((int64_t)b * Hq + g) * d, d, qd);
    fasa_oracle_ca_counts(qd, Kd, L, d, pairing, top_k, f32, c);
    for (int i = 0; i < n_fc; ++i) {
#ifdef _OPENMP
#pragma omp atomic
#endif
      counts[(int64_t)g * n_fc + i] += c[i];
    }
#ifdef _OPENMP
#pragma omp atomic
#endif
    n_used[g] += 1;
    free(Kd); free(qd); free(c);
  }
  return used;
}

/* Stage 2 of Algorithm 1: the mean CA of FC i for KV head h is taken over every
 * sample of the query heads that share h (they read the same keys, and the
 * dominant part of the key cache is kept per KV head); I_dom(h) = the F FCs with
 * the highest mean, a lower index first among equal means, returned ascending.
 * mean_ca ([Hkv][n_fc], may be NULL) receives the means (0 where no sample). */
void fasa_oracle_select_dominant(const int64_t* counts, const int64_t* n_used, int Hq,
                                 int Hkv, int n_fc, int top_k, int F, int32_t* dom,
                                 double* mean_ca) {
  int group = Hq / Hkv;
  for (int h = 0; h < Hkv; ++h) {
    ranked_t* r = (ranked_t*)malloc(sizeof(ranked_t) * (size_t)n_fc);
    int64_t samples = 0;
    for (int g = h * group; g < (h + 1) * group; ++g) samples += n_used[g];
    for (int i = 0; i < n_fc; ++i) {
      int64_t sum = 0;
      for (int g = h * group; g < (h + 1) * group; ++g) sum += counts[(int64_t)g * n_fc + i];
      r[i].s = samples > 0 ? (double)sum / ((double)samples * (double)top_k) : 0.0;
      r[i].j = i;
      if (mean_ca) mean_ca[(int64_t)h * n_fc + i] = r[i].s;
    }
    qsort(r, (size_t)n_fc, sizeof(ranked_t), rank_cmp);
    int* pick = (int*)malloc(sizeof(int) * (size_t)F);
    for (int t = 0; t < F; ++t) pick[t] = r[t].j;
    qsort(pick, (size_t)F, sizeof(int), int_cmp);
    for (int t = 0; t < F; ++t) dom[(int64_t)h * F + t] = pick[t];
    free(pick); free(r);
  }
}

/* ------------------------------------------------- whole step on bf16 bits */

/* One decode step over a batch, the steps in the paper's order per selection
 * unit: widen the bf16 bits -> TIP score -> TopK-I (+ forced) -> FAC, and
 * optionally the dense FKV output.  A selection unit is sel_heads consecutive
 * query heads that share one index set (sel_heads = 0 means the whole group
 * Hq / Hkv; it must divide the group); unit hs of a sequence covers query heads
 * hs * sel_heads .. and reads the cache of KV head (hs * sel_heads) / (Hq / Hkv).
 * With Hs = Hq / sel_heads units per sequence, layouts (row-major, the same bits
 * the GPU path reads):
 *   q_bits  [B][Hq][d]           K_bits, V_bits  [B][Hkv][Lmax][d]
 *   seq_lens[B]                  dom [Hkv][F]
 * Outputs (any may be NULL): scores [B][Hs][Lmax] (rows >= L untouched),
 *   idx [B][Hs][n_sel_max] ascending, n_sel [B][Hs], band [B][Hs][4],
 *   out [B][Hq][d], lse [B][Hq], dense_out [B][Hq][d], dense_lse [B][Hq].
 * budget > 0 is absolute; budget < 0 means ceil(-budget/1000 * L) in integers.
 * Units are independent; with OpenMP they are spread over n_threads threads.
 * Returns the number of threads used, or -1 for a sel_heads that does not divide
 * the group. */
int fasa_oracle_decode_bf16(const uint16_t* q_bits, const uint16_t* K_bits,
                            const uint16_t* V_bits, const int32_t* seq_lens,
                            const int32_t* dom, int B, int Hq, int Hkv, int d, int Lmax,
                            int F, int pairing, int group_reduce, int n_sink, int n_recent,
                            int budget, int n_sel_max, double scale, double tie_rel,
                            int n_threads, int sel_heads, double* scores, int32_t* idx,
                            int32_t* n_sel, double* band, double* out, double* lse,
                            double* dense_out, double* dense_lse) {
  int group = Hq / Hkv;
  int G = sel_heads > 0 ? sel_heads : group;   /* query heads per selection unit */
  if (group % G != 0) return -1;
  int Hs = Hq / G;
  int used = 1;
#ifdef _OPENMP
  if (n_threads > 0) omp_set_num_threads(n_threads);
  used = n_threads > 0 ? n_threads : omp_get_max_threads();
  if (used > B * Hs) used = B * Hs;
#pragma omp parallel for schedule(dynamic, 1)
#endif
  for (int u = 0; u < B * Hs; ++u) {
    int b = u / Hs, hs = u % Hs;
    int q0 = hs * G;          /* first query head of the unit */
    int h = q0 / group;       /* the KV head it attends */
    int L = seq_lens[b];
    if (L > Lmax) L = Lmax;
    if (L < 0) L = 0;
    size_t rows = (size_t)(L > 0 ? L : 1);
    double* Kd = (double*)malloc(sizeof(double) * rows * (size_t)d);
    double* Vd = (double*)malloc(sizeof(double) * rows * (size_t)d);
    double* qd = (double*)malloc(sizeof(double) * (size_t)G * (size_t)d);
    double* S = (double*)malloc(sizeof(double) * rows);
    int* sel = (int*)malloc(sizeof(int) * rows);
    const uint16_t* Kb = K_bits + ((int64_t)b * Hkv + h) * (int64_t)Lmax * d;
    const uint16_t* Vb = V_bits + ((int64_t)b * Hkv + h) * (int64_t)Lmax * d;
    fasa_oracle_widen_bf16(Kb, (int64_t)L * d, Kd);
    fasa_oracle_widen_bf16(Vb, (int64_t)L * d, Vd);
    fasa_oracle_widen_bf16(q_bits + ((int64_t)b * Hq + q0) * d, (int64_t)G * d, qd);

    fasa_oracle_fc_score(qd, G, Kd, L, d, pairing, dom + (int64_t)h * F, F, group_reduce, S);
    if (scores) memcpy(scores + (int64_t)u * Lmax, S, sizeof(double) * (size_t)L);

    int k = budget;
    if (budget < 0) k = (int)(((int64_t)(-budget) * L + 999) / 1000);
    double bd[4];
    int n = fasa_oracle_select(S, L, k, n_sink, n_recent, tie_rel, sel, bd);
    if (band) memcpy(band + (int64_t)u * 4, bd, sizeof bd);
    if (n_sel) n_sel[u] = n;
    if (idx) {
      int w = n < n_sel_max ? n : n_sel_max;
      for (int t = 0; t < w; ++t) idx[(int64_t)u * n_sel_max + t] = sel[t];
    }
    if (out)
      fasa_oracle_attn_subset(qd, G, Kd, Vd, d, sel, n, scale,
                              out + ((int64_t)b * Hq + q0) * d,
                              lse ? lse + (int64_t)b * Hq + q0 : NULL);
    if (dense_out)
      fasa_oracle_attn_dense(qd, G, Kd, Vd, d, L, scale,
                             dense_out + ((int64_t)b * Hq + q0) * d,
                             dense_lse ? dense_lse + (int64_t)b * Hq + q0 : NULL);
    free(Kd); free(Vd); free(qd); free(S); free(sel);
  }
  return used;
}
