/*
 * e3 oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of what the vocabulary-side path computes.
 * Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
 * build, load or call this file.  It shares no source, header, table or helper
 * with the CUDA library; the two are written separately from the same passages
 * of the paper.
 *
 * Every function is the definition written out in the paper's notation, one
 * straightforward loop per sum, no blocking, no fusion, no reordering.  The
 * only parallelism is an OpenMP "parallel for" over independent rows.
 *
 * Parity status of the readings the paper leaves open:
 *   - Algorithm 1, last step ("distribute greedily"): two readings are
 *     implemented (fill-to-cap, round-robin).  Which of the two the authors
 *     meant is PARITY UNPINNED; everything else in Algorithm 1 is pinned by
 *     invariants and brute force.
 *   - Everything else below is pinned by closed forms, invariants, library
 *     routines or statistical tests in tests/ (see each function's comment).
 *
 * Passages followed:
 *   App. A (softmax with temperature, shifted form, Z(beta))   -> row_softmax_stats
 *   Eq. "entropy" and its decomposition (App. A)               -> row_softmax_stats
 *   Sec. 3.1 importance ratio (needs ln pi(o_t))               -> log-prob output
 *   Sec. 2 / Sec. 5.1 (tokens are drawn from softmax(z/tau))   -> e3o_sample
 *   Sec. 4.2 ("logits are also divided by the temperature
 *             during forward propagation after sampling")     -> e3o_token_logp_entropy
 *   Sec. 3.1 objective, Sec. 4.2 entropy regulariser (chain rule
 *             through the softmax of App. A)                   -> e3o_token_logp_entropy_backward
 *   Sec. 4.2 (H_init, H_t: average entropy of a batch)         -> e3o_masked_mean_entropy
 *   Eq. "adv" (Sec. 3.1)                                       -> e3o_group_advantage
 *   GRPO objective (Sec. 3.1, no KL term)                      -> e3o_grpo_objective
 *   Algorithm 1 (Sec. 4.1)                                     -> e3o_allocate_budget
 *   Sec. 4.1 difficulty model, G_min/G_max curriculum          -> e3o_difficulty_*, e3o_budget_curriculum
 *   Eq. "tp_adj" and the annealing equation (Sec. 4.2)         -> e3o_update_temperature
 *   Eq. "tp_relation_1" with Delta from the entropy (App. A)   -> e3o_entropy_gap, e3o_update_temperature_gap
 */
#define _GNU_SOURCE
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { E3O_F32 = 0, E3O_BF16 = 1 };
enum { E3O_SAMPLER_TOKEN = 0, E3O_SAMPLER_BLOCK = 1 };
#define E3O_SAMPLE_BLOCK 256

/* Number of threads the row loops use (reported by the benchmark). */
int e3o_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Exact widening of one stored logit to double (bf16 = upper half of an fp32). */
static double widen(const void *base, int dt, int64_t idx) {
  if (dt == E3O_F32) return (double)((const float *)base)[idx];
  uint32_t bits = (uint32_t)((const uint16_t *)base)[idx] << 16;
  float f;
  memcpy(&f, &bits, 4);
  return (double)f;
}

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as    */
/* easy as 1, 2, 3", SC'11).  One call maps a 128-bit counter and a 64-bit    */
/* key to four 32-bit words.  Pinned in tests against an independent library  */
/* implementation and by equidistribution tests.                              */
/* ------------------------------------------------------------------------- */
void e3o_philox4x32_10(uint32_t key_lo, uint32_t key_hi, const uint32_t ctr[4], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key_lo, k1 = key_hi;
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The sampler's random streams.  A call is addressed by
 *   counter words = (j, global row, step counter low word,
 *                    (step counter high bits << 8) | stream tag),
 *   key           = 64-bit seed.
 * j is the call index inside the stream; tag separates the streams:
 *   0 coarse bytes, 1 fine words, 2 one word per vocabulary block, 3 in-block draw. */
static void stream_call(uint64_t seed, uint64_t counter, uint32_t grow, uint32_t j, uint32_t tag,
                        uint32_t w[4]) {
  uint32_t ctr[4];
  ctr[0] = j;
  ctr[1] = grow;
  ctr[2] = (uint32_t)(counter & 0xffffffffu);
  ctr[3] = ((uint32_t)(counter >> 32) << 8) | tag;
  e3o_philox4x32_10((uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32), ctr, w);
}

/* Per-token uniform of sampler 0: 8 coarse bits + 32 fine bits,
 *   u_i = (c_i + (x_i + 1/2) 2^-32) / 256,   strictly inside (0,1), exact in fp64.
 * c_i is byte (i mod 4) (little endian) of word (i mod 16)/4 of coarse call i/16;
 * x_i is word (i mod 4) of fine call i/4. */
double e3o_token_uniform(uint64_t seed, uint64_t counter, uint32_t grow, int64_t i) {
  uint32_t w[4];
  stream_call(seed, counter, grow, (uint32_t)(i >> 4), 0u, w);
  uint32_t c = (w[(i & 15) >> 2] >> (8 * (i & 3))) & 0xffu;
  stream_call(seed, counter, grow, (uint32_t)(i >> 2), 1u, w);
  uint32_t x = w[i & 3];
  return ((double)c + ((double)x + 0.5) * 0x1p-32) / 256.0;
}

/* One 32-bit-resolution uniform (x + 1/2) 2^-32 from a tagged stream. */
static double word_uniform(uint64_t seed, uint64_t counter, uint32_t grow, int64_t idx, uint32_t tag) {
  uint32_t w[4];
  stream_call(seed, counter, grow, (uint32_t)(idx >> 2), tag, w);
  return ((double)w[idx & 3] + 0.5) * 0x1p-32;
}
double e3o_block_uniform(uint64_t seed, uint64_t counter, uint32_t grow, int64_t b) {
  return word_uniform(seed, counter, grow, b, 2u);
}
double e3o_inblock_uniform(uint64_t seed, uint64_t counter, uint32_t grow) {
  return word_uniform(seed, counter, grow, 0, 3u);
}

/* Standard Gumbel variate from a uniform: g = -ln(-ln u). */
static double gumbel(double u) { return -log(-log(u)); }

/* ------------------------------------------------------------------------- */
/* App. A: p_i = exp(z_i/tau) / sum_j exp(z_j/tau), written in the shifted    */
/* form with Delta_i = z_max - z_i, beta = 1/tau, Z(beta) = sum exp(-beta     */
/* Delta_j); Eq. "entropy": H = -sum p_i ln p_i; its decomposition            */
/* H = beta sum p_i Delta_i + ln Z(beta).                                     */
/* Returns 0 when the row is valid, non-zero otherwise (NaN or +inf logit,    */
/* every logit -inf, tau not > 0).  s[] receives s_i = z_i / tau.             */
/* Pins: uniform row -> ln V; two-level row closed form; the two entropy      */
/* formulas agree; shift / permutation invariance; sum p = 1.                 */
/* ------------------------------------------------------------------------- */
typedef struct {
  double m;      /* max_i s_i                                  */
  double Z;      /* sum_i exp(s_i - m)                         */
  double H_def;  /* -sum p ln p   (Eq. "entropy")              */
  double H_dec;  /* beta sum p Delta + ln Z (the decomposition) */
} row_stats;

static int row_softmax_stats(const void *row, int dt, int64_t V, double tau, double *s, row_stats *st) {
  if (!(tau > 0.0) || isinf(tau)) return 1;
  double m = -INFINITY;
  for (int64_t i = 0; i < V; ++i) {
    double z = widen(row, dt, i);
    if (isnan(z) || z == INFINITY) return 2;
    s[i] = z / tau;
    if (s[i] > m) m = s[i];
  }
  if (m == -INFINITY) return 3;
  double Z = 0.0;
  for (int64_t i = 0; i < V; ++i) Z += exp(s[i] - m);
  double H_def = 0.0, pd = 0.0;
  for (int64_t i = 0; i < V; ++i) {
    double p = exp(s[i] - m) / Z;
    if (p > 0.0) {
      H_def -= p * log(p);
      pd += p * (m - s[i]); /* beta * p_i * Delta_i, since m - s_i = beta (z_max - z_i) */
    }
  }
  st->m = m;
  st->Z = Z;
  st->H_def = H_def;
  st->H_dec = pd + log(Z);
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Rollout side: one token per row drawn from softmax(z / tau_row) with the   */
/* Gumbel-max construction, plus that token's log-probability and the row's   */
/* entropy.                                                                   */
/*   sampler 0: tok = lowest index attaining max_i (s_i + g_i), g_i from the  */
/*              per-token uniform above.                                      */
/*   sampler 1: vocabulary cut into blocks of 256 consecutive indices.        */
/*              L_b = m_b + ln sum_{i in b} exp(s_i - m_b); one Gumbel per    */
/*              block, Y_b = L_b + g_b; b* = lowest-index argmax; then one    */
/*              uniform v picks inside b* by inverse CDF over the weights     */
/*              exp(s_i - m_b*) in index order.                               */
/*   tau == 0 : greedy, tok = lowest-index argmax z, logp = 0, ent = 0.       */
/* Invalid rows: tok = -1, logp = ent = NaN.                                  */
/* y1/y2: best and second-best perturbed score (Y_b for sampler 1);           */
/* cdf_margin (sampler 1): distance of the in-block threshold to the nearest  */
/* prefix-sum boundary, relative to the block sum.  All optional.             */
/* Pins: chi-square of 10^6 draws vs softmax; dominance rule (gap/tau >       */
/* 31.77 -> argmax); V <= 256 with sampler 1 = textbook inverse CDF.          */
/* ------------------------------------------------------------------------- */
static void sample_row(const void *row, int dt, int64_t V, double tau, uint64_t seed, uint64_t counter,
                       uint32_t grow, int sampler, double *s, int32_t *tok, double *logp, double *ent,
                       double *ent_dec, double *y1o, double *y2o, double *cdfm) {
  *tok = -1; *logp = NAN; *ent = NAN;
  if (ent_dec) *ent_dec = NAN;
  if (y1o) *y1o = NAN;
  if (y2o) *y2o = NAN;
  if (cdfm) *cdfm = NAN;

  if (tau == 0.0) { /* greedy */
    double zmax = -INFINITY;
    int64_t arg = -1;
    for (int64_t i = 0; i < V; ++i) {
      double z = widen(row, dt, i);
      if (isnan(z) || z == INFINITY) return;
      if (z > zmax) { zmax = z; arg = i; }
    }
    if (arg < 0) return;
    *tok = (int32_t)arg; *logp = 0.0; *ent = 0.0;
    if (ent_dec) *ent_dec = 0.0;
    return;
  }

  row_stats st;
  if (row_softmax_stats(row, dt, V, tau, s, &st) != 0) return;

  int64_t best = -1;
  double y1 = -INFINITY, y2 = -INFINITY;
  if (sampler == E3O_SAMPLER_TOKEN) {
    for (int64_t i = 0; i < V; ++i) {
      if (s[i] == -INFINITY) continue;
      double y = s[i] + gumbel(e3o_token_uniform(seed, counter, grow, i));
      if (y > y1) { y2 = y1; y1 = y; best = i; }
      else if (y > y2) { y2 = y; }
    }
  } else {
    int64_t nb = (V + E3O_SAMPLE_BLOCK - 1) / E3O_SAMPLE_BLOCK, bstar = -1;
    for (int64_t b = 0; b < nb; ++b) {
      int64_t lo = b * E3O_SAMPLE_BLOCK, hi = lo + E3O_SAMPLE_BLOCK < V ? lo + E3O_SAMPLE_BLOCK : V;
      double mb = -INFINITY;
      for (int64_t i = lo; i < hi; ++i) if (s[i] > mb) mb = s[i];
      if (mb == -INFINITY) continue;
      double Sb = 0.0;
      for (int64_t i = lo; i < hi; ++i) Sb += exp(s[i] - mb);
      double Y = mb + log(Sb) + gumbel(e3o_block_uniform(seed, counter, grow, b));
      if (Y > y1) { y2 = y1; y1 = Y; bstar = b; }
      else if (Y > y2) { y2 = Y; }
    }
    int64_t lo = bstar * E3O_SAMPLE_BLOCK, hi = lo + E3O_SAMPLE_BLOCK < V ? lo + E3O_SAMPLE_BLOCK : V;
    double mb = -INFINITY, Sb = 0.0;
    for (int64_t i = lo; i < hi; ++i) if (s[i] > mb) mb = s[i];
    for (int64_t i = lo; i < hi; ++i) Sb += exp(s[i] - mb);
    double t = e3o_inblock_uniform(seed, counter, grow) * Sb;
    double prefix = 0.0, margin = INFINITY;
    int64_t last_nonzero = -1;
    for (int64_t i = lo; i < hi; ++i) {
      double w = exp(s[i] - mb);
      if (w > 0.0) last_nonzero = i;
      prefix += w;
      if (best < 0 && prefix > t) best = i;
      if (i + 1 < hi && fabs(prefix - t) < margin) margin = fabs(prefix - t);
    }
    if (best < 0) best = last_nonzero;
    if (cdfm) *cdfm = margin / Sb;
  }
  *tok = (int32_t)best;
  *logp = s[best] - st.m - log(st.Z);
  *ent = st.H_def;
  if (ent_dec) *ent_dec = st.H_dec;
  if (y1o) *y1o = y1;
  if (y2o) *y2o = y2;
}

int e3o_sample(const void *logits, int dt, int64_t rows, int64_t V, int64_t row_stride,
               const float *temps, uint64_t seed, uint64_t counter, int64_t row_base, int sampler,
               int32_t *out_tok, double *out_logp, double *out_ent, double *out_ent_dec,
               double *out_y1, double *out_y2, double *out_cdf_margin) {
  if (rows < 0 || V < 1 || row_stride < V || (dt != E3O_F32 && dt != E3O_BF16)) return 1;
  if (sampler != E3O_SAMPLER_TOKEN && sampler != E3O_SAMPLER_BLOCK) return 1;
  size_t esz = dt == E3O_F32 ? 4 : 2;
#pragma omp parallel
  {
    double *s = (double *)malloc(sizeof(double) * (size_t)V);
#pragma omp for schedule(dynamic, 1)
    for (int64_t r = 0; r < rows; ++r) {
      const char *row = (const char *)logits + (size_t)r * (size_t)row_stride * esz;
      int32_t tok; double lp, en, ed, y1, y2, cm;
      sample_row(row, dt, V, (double)temps[r], seed, counter, (uint32_t)(row_base + r), sampler, s,
                 &tok, &lp, &en, &ed, &y1, &y2, &cm);
      out_tok[r] = tok;
      if (out_logp) out_logp[r] = lp;
      if (out_ent) out_ent[r] = en;
      if (out_ent_dec) out_ent_dec[r] = ed;
      if (out_y1) out_y1[r] = y1;
      if (out_y2) out_y2[r] = y2;
      if (out_cdf_margin) out_cdf_margin[r] = cm;
    }
    free(s);
  }
  return 0;
}

/* n independent draws from ONE row (the step counter runs counter0, counter0+1, ...):
 * what a rollout does at one position over many decode steps.  Used by the
 * chi-square pin. */
int e3o_sample_repeat(const void *row, int dt, int64_t V, float tau, uint64_t seed, uint64_t counter0,
                      int64_t grow, int sampler, int64_t n, int32_t *out_tok) {
  if (V < 1 || n < 0) return 1;
#pragma omp parallel
  {
    double *s = (double *)malloc(sizeof(double) * (size_t)V);
#pragma omp for schedule(static)
    for (int64_t d = 0; d < n; ++d) {
      double lp, en;
      sample_row(row, dt, V, (double)tau, seed, counter0 + (uint64_t)d, (uint32_t)grow, sampler, s,
                 &out_tok[d], &lp, &en, NULL, NULL, NULL, NULL);
    }
    free(s);
  }
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Training side: log-probability of a given token and entropy of             */
/* softmax(z / tau) per row (Sec. 3.1 ratio; Sec. 4.2: the training forward   */
/* divides the logits by the same temperature).  Rows with mask == 0 give 0   */
/* and are not looked at.  temps == NULL -> temp_scalar for every row.        */
/* tau must be > 0 here; an invalid row gives NaN; a target outside [0,V)     */
/* gives logp = NaN with a valid entropy.                                     */
/* ------------------------------------------------------------------------- */
int e3o_token_logp_entropy(const void *logits, int dt, int64_t rows, int64_t V, int64_t row_stride,
                           const int32_t *targets, const uint8_t *mask, const float *temps,
                           float temp_scalar, double *out_logp, double *out_ent, double *out_ent_dec) {
  if (rows < 0 || V < 1 || row_stride < V || (dt != E3O_F32 && dt != E3O_BF16)) return 1;
  size_t esz = dt == E3O_F32 ? 4 : 2;
#pragma omp parallel
  {
    double *s = (double *)malloc(sizeof(double) * (size_t)V);
#pragma omp for schedule(dynamic, 1)
    for (int64_t r = 0; r < rows; ++r) {
      double lp = 0.0, en = 0.0, ed = 0.0;
      if (!mask || mask[r]) {
        const char *row = (const char *)logits + (size_t)r * (size_t)row_stride * esz;
        double tau = temps ? (double)temps[r] : (double)temp_scalar;
        row_stats st;
        if (row_softmax_stats(row, dt, V, tau, s, &st) != 0) {
          lp = en = ed = NAN;
        } else {
          en = st.H_def;
          ed = st.H_dec;
          int32_t t = targets[r];
          lp = (t < 0 || t >= V) ? NAN : s[t] - st.m - log(st.Z);
        }
      }
      if (out_logp) out_logp[r] = lp;
      if (out_ent) out_ent[r] = en;
      if (out_ent_dec) out_ent_dec[r] = ed;
    }
    free(s);
  }
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Mean logit gap of a row in units of tau (App. A): with Delta_i = z_max -   */
/* z_i and beta = 1/tau,  gap = beta sum_i p_i Delta_i = sum_i p_i (s_max -   */
/* s_i), the first term of the decomposition H = beta sum p Delta + ln Z.     */
/* It is the quantity Eq. "tp_relation_1" needs an estimate of (beta Delta of */
/* the two-level model).  Rows with mask == 0 give 0; tau == 0 with greedy    */
/* != 0 gives 0 (point mass on the arg-max); an invalid row gives NaN.        */
/* Written out from the definition with its own loops (no shared state with   */
/* the entropy routine above).                                                */
/* Pins: two-level row -> beta Delta q / (1 + q), q = (N-1) exp(-beta Delta); */
/* uniform row -> 0; H = ln Z + gap with H from -sum p ln p; invariance under */
/* a shift of the row.                                                        */
/* ------------------------------------------------------------------------- */
int e3o_row_gap(const void *logits, int dt, int64_t rows, int64_t V, int64_t row_stride, const uint8_t *mask,
                const float *temps, float temp_scalar, int greedy, double *out_gap) {
  if (rows < 0 || V < 1 || row_stride < V || (dt != E3O_F32 && dt != E3O_BF16) || !out_gap) return 1;
  size_t esz = dt == E3O_F32 ? 4 : 2;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t r = 0; r < rows; ++r) {
    if (mask && !mask[r]) { out_gap[r] = 0.0; continue; }
    const char *row = (const char *)logits + (size_t)r * (size_t)row_stride * esz;
    double tau = temps ? (double)temps[r] : (double)temp_scalar;
    int bad = 0;
    double zmax = -INFINITY;
    for (int64_t i = 0; i < V; ++i) {
      double z = widen(row, dt, i);
      if (isnan(z) || z == INFINITY) bad = 1;
      if (z > zmax) zmax = z;
    }
    if (bad || zmax == -INFINITY) { out_gap[r] = NAN; continue; }
    if (greedy && tau == 0.0) { out_gap[r] = 0.0; continue; }
    if (!(tau > 0.0) || isinf(tau)) { out_gap[r] = NAN; continue; }
    double beta = 1.0 / tau, Z = 0.0, num = 0.0;
    for (int64_t i = 0; i < V; ++i) {
      double delta = zmax - widen(row, dt, i); /* Delta_i >= 0, +inf for a -inf logit */
      if (delta == INFINITY) continue;          /* p_i = 0 */
      double w = exp(-beta * delta);
      Z += w;
      num += w * (beta * delta);
    }
    out_gap[r] = num / Z;
  }
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Gradient of the training-side outputs with respect to the logits.  The     */
/* objective of Sec. 3.1 depends on the logits through ln pi(o_t), the        */
/* entropy-regularised objective discussed in Sec. 4.2 also through H; with   */
/* p = softmax(z / tau), beta = 1/tau (App. A) the chain rule through the     */
/* softmax gives                                                              */
/*   d ln p_tok / d z_i = beta (1[i == tok] - p_i)                            */
/*   d H        / d z_i = -beta p_i (ln p_i + H)                              */
/* so that, for upstream gradients g_logp and g_ent of a row,                 */
/*   dlogits_i = beta [ g_logp (1[i == tok] - p_i) - g_ent p_i (ln p_i + H) ].*/
/* Rows with mask == 0 get zeros; an invalid row or a target outside [0, V)   */
/* gives NaN.  Entries with p_i = 0 (logit -inf) get 0 from the entropy term. */
/* Pins: central differences of e3o_token_logp_entropy itself; the gradient   */
/* sums to zero over a row; an autograd library on tiny rows.                 */
/* ------------------------------------------------------------------------- */
int e3o_token_logp_entropy_backward(const void *logits, int dt, int64_t rows, int64_t V, int64_t row_stride,
                                    const int32_t *targets, const uint8_t *mask, const float *temps,
                                    float temp_scalar, const float *g_logp, const float *g_ent,
                                    double *out_dlogits /* [rows, V] dense */) {
  if (rows < 0 || V < 1 || row_stride < V || (dt != E3O_F32 && dt != E3O_BF16)) return 1;
  size_t esz = dt == E3O_F32 ? 4 : 2;
#pragma omp parallel
  {
    double *s = (double *)malloc(sizeof(double) * (size_t)V);
#pragma omp for schedule(dynamic, 1)
    for (int64_t r = 0; r < rows; ++r) {
      double *d = out_dlogits + (size_t)r * (size_t)V;
      if (mask && !mask[r]) {
        for (int64_t i = 0; i < V; ++i) d[i] = 0.0;
        continue;
      }
      const char *row = (const char *)logits + (size_t)r * (size_t)row_stride * esz;
      double tau = temps ? (double)temps[r] : (double)temp_scalar;
      row_stats st;
      int32_t t = targets[r];
      if (row_softmax_stats(row, dt, V, tau, s, &st) != 0 || t < 0 || t >= V) {
        for (int64_t i = 0; i < V; ++i) d[i] = NAN;
        continue;
      }
      double beta = 1.0 / tau, H = st.H_def, lnZ = log(st.Z);
      double gl = g_logp ? (double)g_logp[r] : 0.0, ge = g_ent ? (double)g_ent[r] : 0.0;
      for (int64_t i = 0; i < V; ++i) {
        double lnp = s[i] - st.m - lnZ;
        double p = exp(lnp);
        double ent_term = p > 0.0 ? p * (lnp + H) : 0.0;
        d[i] = beta * (gl * ((i == t ? 1.0 : 0.0) - p) - ge * ent_term);
      }
    }
    free(s);
  }
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Sec. 4.2: "average entropy" of a batch, read as the mean over all          */
/* response tokens of the batch: H_t = sum_j mask_j H_j / sum_j mask_j.       */
/* mask == NULL -> every token counts.  count == 0 -> mean NaN.               */
/* Pins: all-ones mask = plain mean; count = sum of mask; brute force.        */
/* ------------------------------------------------------------------------- */
int e3o_masked_mean_entropy(const float *ent, const uint8_t *mask, int64_t n, double *out_mean,
                            double *out_count) {
  if (n < 0) return 1;
  double sum = 0.0, cnt = 0.0;
  for (int64_t j = 0; j < n; ++j) {
    if (!mask || mask[j]) { sum += (double)ent[j]; cnt += 1.0; }
  }
  *out_mean = cnt > 0.0 ? sum / cnt : NAN;
  *out_count = cnt;
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Eq. "adv": A_i = (r_i - mean(r)) / std(r) inside each rollout group.       */
/* Groups are rows [off_g, off_{g+1}).  std is the sample (n-1) or population */
/* (n) standard deviation; eps is added to it so that a group whose rewards   */
/* are all equal gets advantage exactly 0 (Sec. 4.2 relies on that).  A group */
/* of one gets 0.  flags: bit 0 = all rewards equal, bit 1 = all rewards 0.   */
/* Pins: worked example r=(1,0,...,0); zero group mean; textbook z-score.     */
/* ------------------------------------------------------------------------- */
/* The other reading of "average entropy" (Sec. 4.2): the mean over sequences of every sequence's own mean   */
/* token entropy; tokens laid out [n_seq, seq_len]; sequences without a token take no part; none at all: NaN. */
/* Pins: brute force; equal-length sequences give the token mean; hand case where the two readings differ.    */
int e3o_sequence_mean_entropy(const float *ent, const uint8_t *mask, int64_t n_seq, int64_t seq_len,
                              double *out_mean, double *out_count) {
  if (n_seq < 0 || seq_len < 0 || !out_mean || !out_count) return 1;
  double total = 0.0, used = 0.0;
  for (int64_t s = 0; s < n_seq; ++s) {
    double sum = 0.0, cnt = 0.0;
    for (int64_t t = 0; t < seq_len; ++t) {
      int64_t j = s * seq_len + t;
      if (!mask || mask[j]) { sum += (double)ent[j]; cnt += 1.0; }
    }
    if (cnt > 0.0) { total += sum / cnt; used += 1.0; }
  }
  *out_mean = used > 0.0 ? total / used : NAN;
  *out_count = used;
  return 0;
}

int e3o_group_advantage(const float *rewards, const int64_t *group_offsets, int64_t n_groups, float eps,
                        int unbiased, double *out_adv, uint8_t *out_flags) {
  if (n_groups < 0) return 1;
  for (int64_t g = 0; g < n_groups; ++g) {
    int64_t lo = group_offsets[g], hi = group_offsets[g + 1], n = hi - lo;
    if (n < 0) return 2;
    if (n == 0) { if (out_flags) out_flags[g] = 0; continue; }
    double mean = 0.0;
    for (int64_t i = lo; i < hi; ++i) mean += (double)rewards[i];
    mean /= (double)n;
    double ss = 0.0;
    int all_equal = 1, all_zero = 1;
    for (int64_t i = lo; i < hi; ++i) {
      double d = (double)rewards[i] - mean;
      ss += d * d;
      if (rewards[i] != rewards[lo]) all_equal = 0;
      if (rewards[i] != 0.0f) all_zero = 0;
    }
    double denom = unbiased ? (double)(n - 1) : (double)n;
    double sd = (n == 1) ? 0.0 : sqrt(ss / denom);
    for (int64_t i = lo; i < hi; ++i)
      /* Sec. 4.2: a group whose rewards are all equal has advantage 0; with eps == 0 the quotient would be 0/0 */
      out_adv[i] = (n == 1 || sd + (double)eps == 0.0) ? 0.0 : ((double)rewards[i] - mean) / (sd + (double)eps);
    if (out_flags) out_flags[g] = (uint8_t)((all_equal ? 1 : 0) | (all_zero ? 2 : 0));
  }
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 1 (Dynamic Rollout Budget), in the paper's step order.           */
/*   N_total = B G; G_i = G_min; N_rem = N_total - B G_min;                   */
/*   G_i += floor(N_rem k_i / sum_j k_j)  (capped at G_max);                  */
/*   N_rem = N_total - sum G_i; hand N_rem out in descending order of k,      */
/*   never beyond G_max.                                                      */
/* Readings: the cap is applied already in the proportional step (the paper   */
/* names it only in the last step); sum k = 0 -> every G_i = G; ties in k go  */
/* to the lower index first.  greedy_mode 0 = fill each item to the cap in    */
/* turn; 1 = one rollout per item per sweep.  Which of the two the paper      */
/* means is PARITY UNPINNED.                                                  */
/* Returns 0 ok, 1 invalid argument, 2 infeasible (needs G_min<=G<=G_max).    */
/* ------------------------------------------------------------------------- */
typedef struct { double k; int64_t idx; } kv;
static int by_k_desc(const void *a, const void *b) {
  const kv *x = (const kv *)a, *y = (const kv *)b;
  if (x->k > y->k) return -1;
  if (x->k < y->k) return 1;
  return x->idx < y->idx ? -1 : (x->idx > y->idx ? 1 : 0);
}
int e3o_allocate_budget(const double *k, int64_t B, int32_t G, int32_t G_min, int32_t G_max,
                        int greedy_mode, int32_t *out_G) {
  if (B < 0 || G_min < 0) return 1;
  if (G_min > G || G > G_max) return 2;
  double ksum = 0.0;
  for (int64_t i = 0; i < B; ++i) {
    if (!(k[i] >= 0.0 && k[i] <= 1.0)) return 1;
    ksum += k[i];
  }
  if (B == 0) return 0;
  if (ksum == 0.0) { for (int64_t i = 0; i < B; ++i) out_G[i] = G; return 0; }
  int64_t N_total = B * (int64_t)G;
  for (int64_t i = 0; i < B; ++i) out_G[i] = G_min;
  int64_t N_rem = N_total - B * (int64_t)G_min;
  for (int64_t i = 0; i < B; ++i) {
    int64_t add = (int64_t)floor((double)N_rem * (k[i] / ksum));
    int64_t g = (int64_t)out_G[i] + add;
    out_G[i] = (int32_t)(g > G_max ? G_max : g);
  }
  int64_t total = 0;
  for (int64_t i = 0; i < B; ++i) total += out_G[i];
  N_rem = N_total - total;
  kv *order = (kv *)malloc(sizeof(kv) * (size_t)B);
  for (int64_t i = 0; i < B; ++i) { order[i].k = k[i]; order[i].idx = i; }
  qsort(order, (size_t)B, sizeof(kv), by_k_desc);
  if (greedy_mode == 0) {
    for (int64_t q = 0; q < B && N_rem > 0; ++q) {
      int64_t i = order[q].idx, room = (int64_t)G_max - out_G[i];
      int64_t give = room < N_rem ? room : N_rem;
      out_G[i] += (int32_t)give;
      N_rem -= give;
    }
  } else {
    while (N_rem > 0) {
      int moved = 0;
      for (int64_t q = 0; q < B && N_rem > 0; ++q) {
        int64_t i = order[q].idx;
        if (out_G[i] < G_max) { out_G[i] += 1; N_rem -= 1; moved = 1; }
      }
      if (!moved) break;
    }
  }
  free(order);
  return N_rem == 0 ? 0 : 2;
}

/* ------------------------------------------------------------------------- */
/* Eq. "tp_adj": tau' = tau (1 + tau ln(alpha) / (ln|V| + ln ln|V|)),         */
/* alpha = H_target / H_t; H_target = H_init before t_anneal, afterwards      */
/* H_init [eta + (1-eta) (1/2)(1 + cos(pi (t - t_anneal)/(t_max - t_anneal)))]*/
/* (the annealing equation; its brackets are unbalanced in print, this is the */
/* reading that runs from H_init down to eta H_init as the text says).        */
/* The first call with H_init unset (NaN or <= 0) records H_init = H_t        */
/* ("average entropy of the first batch") and leaves tau as it is.            */
/* t advances by one per call.  tau is clamped to [tau_min, tau_max] when     */
/* tau_max > 0.  Returns 0 ok, 1 invalid argument.                            */
/* Pins: alpha = 1 fixed point; printed end points of the anneal; hand value. */
/* ------------------------------------------------------------------------- */
typedef struct {
  double tau, H_init;
  int64_t t, t_anneal, t_max;
  double eta;
  int64_t V;
  double tau_min, tau_max;
} e3o_sched;

double e3o_anneal_target(const e3o_sched *s) {
  if (s->t < s->t_anneal || s->t_max <= s->t_anneal) return s->H_init;
  double frac = (double)(s->t - s->t_anneal) / (double)(s->t_max - s->t_anneal);
  if (frac > 1.0) frac = 1.0;
  return s->H_init * (s->eta + (1.0 - s->eta) * 0.5 * (1.0 + cos(M_PI * frac)));
}

int e3o_update_temperature(e3o_sched *s, double H_t, double *tau_next) {
  if (!(H_t > 0.0) || isinf(H_t) || s->V < 3 || !(s->tau > 0.0)) return 1;
  if (!(s->H_init > 0.0)) {
    s->H_init = H_t;
    s->t += 1;
    *tau_next = s->tau;
    return 0;
  }
  double alpha = e3o_anneal_target(s) / H_t;
  double lnV = log((double)s->V);
  double tau = s->tau * (1.0 + s->tau * log(alpha) / (lnV + log(lnV)));
  if (!(tau > 0.0)) return 1; /* the formula left the domain tau > 0 of App. A: state unchanged */
  if (s->tau_max > 0.0) {
    if (tau < s->tau_min) tau = s->tau_min;
    if (tau > s->tau_max) tau = s->tau_max;
  }
  s->tau = tau;
  s->t += 1;
  *tau_next = tau;
  return 0;
}

/* ------------------------------------------------------------------------- */
/* The un-simplified scheduler of App. A.  Under the two-level model of the    */
/* logits (one dominant logit, N-1 others at gap Delta) the entropy is          */
/*   H ~ (N-1) beta Delta exp(-beta Delta)                                      */
/* and scaling it by alpha needs  tau_1 ~ tau_0 (1 + tau_0 ln(alpha) / Delta)   */
/* (Eq. "tp_relation_1").  The paper then replaces Delta by ln N + ln ln N so   */
/* that Delta need not be estimated.  Here Delta is estimated instead, from    */
/* the measured entropy itself by inverting the model: x = beta_0 Delta is the  */
/* root x >= 1 of (N-1) x exp(-x) = H_t, and the update becomes                 */
/*   tau_1 = tau_0 (1 + ln(alpha) / x).                                         */
/* (The paper's own reduction, x = ln N + c with c = ln(ln N + c) - ln(eps), is  */
/* this equation with N-1 ~ N; it drops -ln(eps), this function keeps it.)      */
/* Reading: "logits can be utilized to estimate Delta" is silent on how; the    */
/* entropy of the same logits is used.  Needs H_t <= (N-1)/e.                   */
/* Pins: root identity; recovery of beta Delta on exact two-level rows; the     */
/* updated temperature scales the closed-form entropy of such rows by alpha to  */
/* within a few percent, closer than the simplified formula when Delta differs  */
/* from ln N + ln ln N.                                                         */
/* ------------------------------------------------------------------------- */
double e3o_entropy_gap(double H, int64_t N) {
  if (!(H > 0.0) || N < 3 || H > ((double)N - 1.0) / M_E) return NAN;
  double lo = 1.0, hi = 1.0; /* x exp(-x) decreases on [1, inf): bracket the root, then bisect */
  while (((double)N - 1.0) * hi * exp(-hi) > H) hi *= 2.0;
  for (int it = 0; it < 200; ++it) {
    double mid = 0.5 * (lo + hi);
    if (((double)N - 1.0) * mid * exp(-mid) > H) lo = mid; else hi = mid;
  }
  return 0.5 * (lo + hi);
}

int e3o_update_temperature_gap(e3o_sched *s, double H_t, double *tau_next) {
  if (!(H_t > 0.0) || isinf(H_t) || s->V < 3 || !(s->tau > 0.0)) return 1;
  double x = e3o_entropy_gap(H_t, s->V);
  if (isnan(x)) return 1;
  if (!(s->H_init > 0.0)) {
    s->H_init = H_t;
    s->t += 1;
    *tau_next = s->tau;
    return 0;
  }
  double alpha = e3o_anneal_target(s) / H_t;
  double tau = s->tau * (1.0 + log(alpha) / x);
  if (!(tau > 0.0)) return 1;
  if (s->tau_max > 0.0) {
    if (tau < s->tau_min) tau = s->tau_min;
    if (tau > s->tau_max) tau = s->tau_max;
  }
  s->tau = tau;
  s->t += 1;
  *tau_next = tau;
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Sec. 4.1, difficulty model.  For every question q_i of the dataset its      */
/* cumulative rollout count n_i^c and cumulative reward r_i^c are recorded;    */
/* at the end of a dataset iteration the questions are ranked by their         */
/* average reward r_i^c / n_i^c in DESCENDING order (rank 1 = highest average  */
/* reward = easiest) and k_i = rank(q_i) / |D|, so a larger k_i means a harder */
/* question.  Readings where the paper is silent: equal averages keep dataset  */
/* order (the earlier question gets the smaller rank); a question that was     */
/* never rolled out has average reward 0.                                      */
/* Pins: brute-force ranking with a library sort; k is a permutation of        */
/* {1/|D|, ..., 1}; a harder question never has a smaller k.                    */
/* ------------------------------------------------------------------------- */
int e3o_difficulty_accumulate(int64_t D, int64_t *n_c, double *r_c, const int64_t *question_ids,
                              const int32_t *G, const float *rewards, int64_t B) {
  if (D < 0 || B < 0) return 1;
  int64_t pos = 0;
  for (int64_t b = 0; b < B; ++b) {
    if (question_ids[b] < 0 || question_ids[b] >= D || G[b] < 0) return 1;
    for (int32_t j = 0; j < G[b]; ++j) r_c[question_ids[b]] += (double)rewards[pos + j];
    n_c[question_ids[b]] += G[b];
    pos += G[b];
  }
  return 0;
}

int e3o_difficulty_rank(int64_t D, const int64_t *n_c, const double *r_c, double *out_k) {
  if (D < 0) return 1;
  for (int64_t i = 0; i < D; ++i) {
    double ai = n_c[i] > 0 ? r_c[i] / (double)n_c[i] : 0.0;
    int64_t rank = 1; /* 1 + number of questions that come before q_i in the descending order */
    for (int64_t j = 0; j < D; ++j) {
      if (j == i) continue;
      double aj = n_c[j] > 0 ? r_c[j] / (double)n_c[j] : 0.0;
      if (aj > ai || (aj == ai && j < i)) ++rank;
    }
    out_k[i] = (double)rank / (double)D;
  }
  return 0;
}

/* Sec. 4.1 / Sec. 5.2: G_min and G_max start at G; after each iteration of the   */
/* dataset G_max grows and G_min shrinks by `step` (2 in the paper's runs) until  */
/* the predefined limits are reached.  `epochs_done` = completed iterations.      */
/* Pins: the paper's setting G = 8, step 2: (8,8), (6,10), (4,12), ...; limits.   */
int e3o_budget_curriculum(int32_t G, int32_t step, int32_t G_min_limit, int32_t G_max_limit, int64_t epochs_done,
                          int32_t *G_min, int32_t *G_max) {
  if (G < 0 || step < 0 || epochs_done < 0 || G_min_limit < 0 || G_min_limit > G || G_max_limit < G) return 1;
  int64_t lo = (int64_t)G, hi = (int64_t)G;
  for (int64_t e = 0; e < epochs_done; ++e) {
    if (hi + step <= G_max_limit) hi += step; else hi = G_max_limit;
    if (lo - step >= G_min_limit) lo -= step; else lo = G_min_limit;
    if (hi == G_max_limit && lo == G_min_limit) break;
  }
  *G_min = (int32_t)lo;
  *G_max = (int32_t)hi;
  return 0;
}

/* ------------------------------------------------------------------------- */
/* The GRPO objective of Sec. 3.1 without the KL term (the paper drops it):    */
/*   J = mean over questions q of                                              */
/*         (1/G_q) sum_{i in group q} (1/|o_i|) sum_{t=1..|o_i|}               */
/*           min( r_{i,t} A_i , clip(r_{i,t}, 1-eps, 1+eps) A_i ),             */
/*   r_{i,t} = pi_theta(o_{i,t}) / pi_theta_old(o_{i,t}) = exp(logp - logp_old).*/
/* Tokens are laid out [n_seq, seq_len]; mask marks the |o_i| response tokens  */
/* of sequence i; A_i is the group-relative advantage of response i (Eq. adv),  */
/* the same for all its tokens; groups are runs of sequences given by offsets   */
/* (their sizes G_q differ under the dynamic rollout budget).  A response       */
/* without tokens contributes 0 but still counts in G_q.                        */
/* Also returns dJ/dlogp per token (0 where the clipped branch is the smaller    */
/* one, i.e. A > 0 and r > 1+eps, or A < 0 and r < 1-eps; 0 on masked tokens)    */
/* and the fraction of response tokens where that happened.                     */
/* Pins: logp == logp_old gives J = mean_q mean_i A_i; hand cases of the clip;   */
/* central differences of J; an autograd library.                               */
/* ------------------------------------------------------------------------- */
int e3o_grpo_objective(const float *logp, const float *logp_old, const uint8_t *mask, int64_t n_seq,
                       int64_t seq_len, const float *adv, const int64_t *group_offsets, int64_t n_groups,
                       float clip_eps, double *out_grad /* [n_seq*seq_len] or NULL */, double *out_J,
                       double *out_clip_frac) {
  if (n_seq < 0 || seq_len < 0 || n_groups < 0 || !(clip_eps >= 0.0f)) return 1;
  if (n_groups > 0 && (group_offsets[0] != 0 || group_offsets[n_groups] != n_seq)) return 1;
  double J = 0.0, clipped = 0.0, tokens = 0.0;
  double lo = 1.0 - (double)clip_eps, hi = 1.0 + (double)clip_eps;
  for (int64_t q = 0; q < n_groups; ++q) {
    int64_t a = group_offsets[q], b = group_offsets[q + 1];
    if (b < a) return 1;
    double Gq = (double)(b - a), Jq = 0.0;
    for (int64_t i = a; i < b; ++i) {
      double len = 0.0;
      for (int64_t t = 0; t < seq_len; ++t) len += (!mask || mask[i * seq_len + t]) ? 1.0 : 0.0;
      double A = (double)adv[i], Ji = 0.0;
      for (int64_t t = 0; t < seq_len; ++t) {
        int64_t j = i * seq_len + t;
        if (out_grad) out_grad[j] = 0.0;
        if (mask && !mask[j]) continue;
        double r = exp((double)logp[j] - (double)logp_old[j]);
        double rc = r < lo ? lo : (r > hi ? hi : r);
        double s1 = r * A, s2 = rc * A;
        int clip_active = s2 < s1; /* the clipped term is the strictly smaller one: no gradient */
        Ji += clip_active ? s2 : s1;
        tokens += 1.0;
        clipped += clip_active ? 1.0 : 0.0;
        if (out_grad) out_grad[j] = clip_active ? 0.0 : s1 / (len * Gq * (double)n_groups);
      }
      if (len > 0.0) Jq += Ji / len;
    }
    if (Gq > 0.0) J += Jq / Gq;
  }
  *out_J = n_groups > 0 ? J / (double)n_groups : 0.0;
  if (out_clip_frac) *out_clip_frac = tokens > 0.0 ? clipped / tokens : 0.0;
  return 0;
}

