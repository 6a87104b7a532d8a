/*
 * csd_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of one verification round of relaxed
 * speculative decoding with annealed relaxation (Cool-SD): Algorithm 1 of the
 * paper (verification stage), the relaxed acceptance probability (Eq. relax),
 * the annealing schedules (UniformRSD, Eq. sdar, and the linear variant of the
 * schedule ablation), and the bound-minimising resampling distribution
 * (Eq. opt_G, Theorem 2 / Proposition LP); the same walk over a static tree of
 * candidates (the draft structure of the paper's experiments; see orc_verify_tree
 * for the reading of several candidates per node); the drafting stage's token draws
 * x~_i ~ Q(. | prefix) (Algorithm 1, drafting stage); and, per position, the two sums that
 * Theorem 2 is made of: the acceptance mass sum_x Q f (the inner sum of Eq.
 * token_exp) and the bracket of Eq. bd2, sum_x |P - Q f| - sum_x (1 - f) Q.
 *
 * It shares no code with the CUDA library.  Only the tests, the smoke check and
 * the benchmark's CPU-baseline leg may call it.  Everything is written as the
 * paper writes it: one sequence at a time, a sequential for/break over the
 * draft positions, full V-length distributions formed explicitly.  There is no
 * blocking, fusion or reordering.  OpenMP (if compiled in) only runs different
 * sequences on different cores.
 *
 * Readings of points the paper leaves open (each is the build's choice and is
 * mirrored, not shared, by the CUDA side):
 *   - index base of the schedule: i = 1..L (Eq. sdar is stated for i in [L]).
 *   - 0/0 := 1 (Notations appendix): q = 0 gives f = 1; p = 0 < q gives f = 0.
 *   - G* is always Eq. opt_G, Norm([P - Q f]_+), also where omega_i < 1.
 *   - sampling from G* is by inverse CDF in token-id order with ONE supplied
 *     uniform u per sequence: smallest x with C(x) > u*Z; if rounding leaves no
 *     such x, the last x with positive mass.
 *   - Z = 0 (only when P == Q and omega >= 1): fall back to G := P.
 *   - the bonus token (tau = L) uses the same u and needs an (L+1)-th target
 *     row; without it the slot is -1.
 *   - guidance mix (not in the paper's verify step; an input-preparation
 *     reading): z = fmaf(s, c - u, u) evaluated in fp32, then everything in fp64.
 *   - top-k (not in the paper): keep every logit >= the k-th largest of the row.
 *   - rows holding NaN or +inf, or with no finite entry, are "invalid": the
 *     position rejects (f := 0); an invalid drafter row resamples from P (the
 *     value of Eq. opt_G at f = 0); an invalid target row emits -1.
 *   - a draft token outside [0, V) rejects (f := 0) and is flagged.
 *   - a multiplier omega_i that is negative or NaN counts as 0 (Eq. relax is
 *     stated for omega >= 0).
 *
 * Resolution: the weights of Eq. opt_G are formed from fp64 probabilities, as
 * the equation is written, so each carries an absolute rounding of about 1e-16.
 * Where both models put all but that much of their mass on one token, the
 * difference of two probabilities next to 1 at that token is lost; a draw at a
 * position whose normaliser Z is below about 1e-10 is therefore outside what
 * this oracle resolves (a valid draft token is rejected there with probability Z).
 *
 * Pins (tests/test_oracle_*.py): Theorem 1 by exact enumeration and chi-square,
 * Theorem 2's expectation and TV bound by brute force on tiny alphabets,
 * Proposition LP's closed form against random and grid search over G,
 * Proposition 2, the schedule's normalisation, the per-position sums against
 * their closed forms and against the brute-force bound, and textbook routines
 * (log-sum-exp, partition, cumsum/searchsorted) for the building blocks.
 * Parity unpinned: nothing -- the paper prints no worked numeric example, so
 * there is no printed value to pin to; every function has an analytic pin.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_F32 0
#define ORC_BF16 1
#define ORC_F64 2

#define ORC_STATUS_BADROW 1
#define ORC_STATUS_BADTOKEN 2
#define ORC_STATUS_ZFALLBACK 4

typedef struct {
  const void *target_logits; /* [B, target_rows, V] (batch stride below) */
  const void *draft_logits;  /* [B, gamma, V] */
  const void *target_uncond; /* NULL: no guidance mix */
  const void *draft_uncond;
  int32_t dtype; /* ORC_F32 / ORC_BF16 / ORC_F64 */
  float cfg_scale;
  int32_t top_k; /* 0: off */
  int32_t B, gamma, V, target_rows;
  int64_t target_batch_stride, draft_batch_stride; /* in elements */
  const int32_t *draft_tokens; /* [B, gamma] */
  const float *uniforms;       /* [B, gamma+1] */
  const float *relax_schedule; /* [gamma] omega_i */
  int32_t *out_tokens;         /* [B, gamma+1] */
  int32_t *out_accept_len;     /* [B] */
  int32_t *out_status;         /* [B] or NULL */
  double *p, *q, *f;           /* [B, gamma] or NULL: all positions, for comparison */
  double *G;                   /* [B, V] or NULL: distribution drawn from */
  double *margin_accept;       /* [B, gamma] or NULL: |r_i - f_i| where the test ran, else +inf */
  double *margin_cdf;          /* [B] or NULL: distance of u to the nearest CDF boundary of the pick */
  double *accept_mass;         /* [B, gamma] or NULL: sum_x Q_i(x) f_i(x) at every position (NaN: unusable row) */
  double *bound_term;          /* [B, gamma] or NULL: the bracket of Eq. bd2 at every position */
  /* Similarity relaxation of LANTERN++ with the paper's resampling distribution (Ablation, "Principled
   * Resampling Strategy"); NULL / 0: off, and nothing above changes. */
  const int32_t *neighbours;   /* [V, nbr_k]: for every token its nearest tokens, nearest first (-1: none) */
  int32_t nbr_k;
  float nbr_lambda;
} orc_params;

int orc_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void orc_set_num_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

/* ---- stored value -> the fp32 value it encodes ---------------------------- */
static float bf16_to_float(uint16_t h) {
  uint32_t w = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &w, sizeof f);
  return f;
}

static double load_value(const void *base, int dtype, int64_t idx) {
  if (dtype == ORC_F32) return (double)((const float *)base)[idx];
  if (dtype == ORC_BF16) return (double)bf16_to_float(((const uint16_t *)base)[idx]);
  return ((const double *)base)[idx];
}

/* ---- schedules ------------------------------------------------------------ */
/* kind 0: UniformRSD, omega_i = delta.
 * kind 1: Eq. sdar, omega_i = delta * exp(-nu*i - mu), mu fixed by
 *         sum_{i=1..L} exp(-nu*i - mu) = L.
 * kind 2: linear variant, omega_i = delta * L * w_i / sum_j w_j with
 *         w_i = (ell - i) / (ell (ell + 1)), clamped at 0 for i >= ell.
 * Returns 0, or -1 on bad arguments. */
int orc_make_schedule(int kind, double delta, double nu_or_ell, int L, double *omega) {
  if (L < 1 || !omega || !(delta >= 0.0)) return -1;
  if (kind == 0) {
    for (int i = 1; i <= L; ++i) omega[i - 1] = delta;
    return 0;
  }
  if (kind == 1) {
    double nu = nu_or_ell;
    if (!(nu >= 0.0)) return -1;
    double total = 0.0;
    for (int i = 1; i <= L; ++i) total += exp(-nu * (double)i);
    double mu = log(total / (double)L); /* sum_i exp(-nu i - mu) = L */
    for (int i = 1; i <= L; ++i) omega[i - 1] = delta * exp(-nu * (double)i - mu);
    return 0;
  }
  if (kind == 2) {
    double ell = nu_or_ell;
    if (!(ell > 1.0)) return -1;
    double total = 0.0;
    for (int i = 1; i <= L; ++i) {
      double w = (ell - (double)i) / (ell * (ell + 1.0));
      if (w < 0.0) w = 0.0;
      omega[i - 1] = w;
      total += w;
    }
    if (!(total > 0.0)) return -1;
    for (int i = 1; i <= L; ++i) omega[i - 1] = delta * (double)L * omega[i - 1] / total;
    return 0;
  }
  return -1;
}

/* ---- building blocks -------------------------------------------------------*/

/* Relaxed acceptance probability, Eq. relax: min{1, omega p / q}, 0/0 := 1.
 * Eq. relax is stated for omega >= 0; a multiplier that is negative or NaN is
 * read as 0 (no relaxation can make f negative), so f = 0 wherever q > 0. */
double orc_accept_prob(double p, double q, double omega) {
  if (q == 0.0) return 1.0; /* p/q = +inf for p > 0, and 0/0 := 1 */
  if (p == 0.0) return 0.0;
  if (!(omega >= 0.0)) omega = 0.0;
  double ratio = omega * p / q;
  return ratio < 1.0 ? ratio : 1.0;
}

/* Softmax of a V-vector of logits.  Returns 1 if the row is valid. */
int orc_softmax(const double *z, int V, double *P) {
  double m = -INFINITY;
  for (int x = 0; x < V; ++x) {
    if (isnan(z[x]) || z[x] == INFINITY) return 0;
    if (z[x] > m) m = z[x];
  }
  if (m == -INFINITY) return 0;
  double S = 0.0;
  for (int x = 0; x < V; ++x) S += exp(z[x] - m);
  for (int x = 0; x < V; ++x) P[x] = exp(z[x] - m) / S;
  return 1;
}

/* Unnormalised Eq. opt_G: g(x) = [P(x) - Q(x) f(x)]_+ with
 * f(x) = min{1, omega P(x)/Q(x)} (Eq. relax evaluated at candidate x).
 * Returns Z = sum_x g(x). */
double orc_resample_weights(const double *P, const double *Q, double omega, int V, double *g) {
  double Z = 0.0;
  for (int x = 0; x < V; ++x) {
    double fx = orc_accept_prob(P[x], Q[x], omega);
    double v = P[x] - Q[x] * fx;
    if (!(v > 0.0)) v = 0.0;
    g[x] = v;
    Z += v;
  }
  return Z;
}

/* The two per-position sums of Theorem 2 for one pair of distributions, written as the paper writes
 * them, with f(x) = min{1, omega P(x)/Q(x)} (Eq. relax at candidate x):
 *   *accept_mass = sum_x Q(x) f(x)                  (inner sum of Eq. token_exp: the probability that
 *                                                    the position accepts, given its prefix)
 *   *bound_term  = sum_x |P(x) - Q(x) f(x)| - sum_x (1 - f(x)) Q(x)     (the bracket of Eq. bd2,
 *                                                    i.e. the infimum of Proposition LP) */
void orc_position_terms(const double *P, const double *Q, double omega, int V, double *accept_mass,
                        double *bound_term) {
  double a = 0.0, abs_sum = 0.0, rej = 0.0;
  for (int x = 0; x < V; ++x) {
    const double fx = orc_accept_prob(P[x], Q[x], omega);
    a += Q[x] * fx;
    abs_sum += fabs(P[x] - Q[x] * fx);
    rej += (1.0 - fx) * Q[x];
  }
  *accept_mass = a;
  *bound_term = abs_sum - rej;
}

/* LANTERN++'s aggregated mass of candidate x (the first case of its P^{k,lambda}): P(x) plus the mass
 * of the selected subset A of x's k nearest tokens.  The paper only says that A is "a selected subset"
 * with sum_{A \ x} P < lambda P(x); the reading here: neighbours are taken nearest first while the
 * running sum stays strictly below lambda P(x), and the first one that would break it ends the
 * selection.  Entries that are -1, out of range or x itself are skipped. */
double orc_neighbour_mass(const double *P, int V, const int32_t *nbr_row, int k, double lambda, int x) {
  const double own = P[x];
  double extra = 0.0;
  for (int j = 0; j < k; ++j) {
    const int y = nbr_row[j];
    if (y < 0 || y >= V || y == x) continue;
    if (extra + P[y] < lambda * own) extra += P[y];
    else break;
  }
  return own + extra;
}

/* Eq. opt_G with LANTERN++'s acceptance f^{k,lambda} (times the multiplier omega) at every candidate:
 * g(x) = [P(x) - Q(x) min{1, omega A(x)/Q(x)}]_+ with A(x) the aggregated mass above.  Returns Z. */
double orc_resample_weights_nbr(const double *P, const double *Q, double omega, int V, const int32_t *nbr, int k,
                                double lambda, double *g) {
  double Z = 0.0;
  for (int x = 0; x < V; ++x) {
    const double fx = orc_accept_prob(orc_neighbour_mass(P, V, nbr + (int64_t)x * k, k, lambda, x), Q[x], omega);
    double v = P[x] - Q[x] * fx;
    if (!(v > 0.0)) v = 0.0;
    g[x] = v;
    Z += v;
  }
  return Z;
}

/* Eq. opt_G normalised; falls back to P when Z = 0.  Returns Z. */
double orc_resample_dist(const double *P, const double *Q, double omega, int V, double *G) {
  double Z = orc_resample_weights(P, Q, omega, V, G);
  if (Z > 0.0) {
    for (int x = 0; x < V; ++x) G[x] /= Z;
  } else {
    for (int x = 0; x < V; ++x) G[x] = P[x];
  }
  return Z;
}

/* Inverse-CDF draw from unnormalised non-negative weights g with total Z:
 * smallest x with C(x) > u Z; else the last x with g(x) > 0.  *margin gets the
 * distance (in probability units) from u to the nearest boundary of the picked
 * token's CDF interval that separates it from another token of positive mass. */
int orc_inverse_cdf(const double *g, int V, double Z, double u, double *margin) {
  double target = u * Z;
  double c = 0.0, c_lo = 0.0, c_hi = 0.0;
  int tok = -1, last_pos = -1, first_pos = -1;
  for (int x = 0; x < V; ++x) {
    double c_prev = c;
    c += g[x];
    if (g[x] > 0.0) {
      last_pos = x;
      if (first_pos < 0) first_pos = x;
    }
    if (tok < 0 && c > target) {
      tok = x;
      c_lo = c_prev;
      c_hi = c;
    }
  }
  if (tok < 0) {
    tok = last_pos;
    if (margin) *margin = 0.0; /* decided by rounding alone */
    return tok;
  }
  if (margin) {
    double mg = INFINITY;
    if (tok != first_pos) mg = fabs(u - c_lo / Z);
    if (tok != last_pos) {
      double d = fabs(u - c_hi / Z);
      if (d < mg) mg = d;
    }
    *margin = mg;
  }
  return tok;
}

/* Row preparation: stored values -> fp64 logits, optional guidance mix (fp32
 * fmaf, see header) and optional top-k mask. */
static int cmp_desc(const void *a, const void *b) {
  double x = *(const double *)a, y = *(const double *)b;
  return (x < y) - (x > y);
}

void orc_prepare_row(const void *cond, const void *uncond, int dtype, int64_t offset, int V,
                     float cfg_scale, int top_k, double *z, double *scratch) {
  for (int x = 0; x < V; ++x) {
    if (uncond) {
      volatile float c = (float)load_value(cond, dtype, offset + x);
      volatile float un = (float)load_value(uncond, dtype, offset + x);
      volatile float d = c - un; /* rounded to fp32 */
      float mixed = fmaf(cfg_scale, d, un);
      z[x] = (double)mixed;
    } else {
      z[x] = load_value(cond, dtype, offset + x);
    }
  }
  if (top_k > 0 && top_k < V) {
    int has_nan = 0;
    for (int x = 0; x < V; ++x) has_nan |= isnan(z[x]);
    if (!has_nan) {
      memcpy(scratch, z, (size_t)V * sizeof(double));
      qsort(scratch, (size_t)V, sizeof(double), cmp_desc);
      double kth = scratch[top_k - 1];
      for (int x = 0; x < V; ++x)
        if (z[x] < kth) z[x] = -INFINITY;
    }
  }
}

/* ---- Algorithm 1, verification stage, one sequence ------------------------ */
static void verify_one(const orc_params *a, int b, double *zt, double *zd, double *P, double *Q,
                       double *g, double *scratch) {
  const int L = a->gamma, V = a->V;
  const int32_t *tok = a->draft_tokens + (int64_t)b * L;
  const float *unif = a->uniforms + (int64_t)b * (L + 1);
  int32_t *out = a->out_tokens + (int64_t)b * (L + 1);
  for (int i = 0; i <= L; ++i) out[i] = -1;
  if (a->margin_accept)
    for (int i = 0; i < L; ++i) a->margin_accept[(int64_t)b * L + i] = INFINITY;
  if (a->margin_cdf) a->margin_cdf[b] = INFINITY;
  if (a->G)
    for (int x = 0; x < V; ++x) a->G[(int64_t)b * V + x] = 0.0;

  int status = 0;
  int tau = 0;
  int emitted = 0; /* set once the (tau+1)-th token slot has been decided */
  const double u = (double)unif[L];

  for (int i = 1; i <= L; ++i) {
    const int64_t t_off = (int64_t)b * a->target_batch_stride + (int64_t)(i - 1) * V;
    const int64_t d_off = (int64_t)b * a->draft_batch_stride + (int64_t)(i - 1) * V;
    orc_prepare_row(a->target_logits, a->target_uncond, a->dtype, t_off, V, a->cfg_scale, a->top_k,
                    zt, scratch);
    orc_prepare_row(a->draft_logits, a->draft_uncond, a->dtype, d_off, V, a->cfg_scale, a->top_k,
                    zd, scratch);
    const int t_ok = orc_softmax(zt, V, P);
    const int d_ok = orc_softmax(zd, V, Q);
    const double omega = (double)a->relax_schedule[i - 1];
    const int x_i = tok[i - 1];
    const int tok_ok = (x_i >= 0 && x_i < V);
    double f;
    if (!t_ok || !d_ok) {
      f = 0.0;
      status |= ORC_STATUS_BADROW;
    } else if (!tok_ok) {
      f = 0.0;
      status |= ORC_STATUS_BADTOKEN;
    } else if (a->neighbours) {
      f = orc_accept_prob(orc_neighbour_mass(P, V, a->neighbours + (int64_t)x_i * a->nbr_k, a->nbr_k,
                                             (double)a->nbr_lambda, x_i), Q[x_i], omega);
    } else {
      f = orc_accept_prob(P[x_i], Q[x_i], omega);
    }
    const double r = (double)unif[i - 1];
    if (a->margin_accept && t_ok && d_ok && tok_ok)
      a->margin_accept[(int64_t)b * L + (i - 1)] = fabs(r - f);
    if (r <= f) {
      tau = i;
      out[i - 1] = x_i;
    } else {
      /* rejected at position i: draw x_i from G*_i */
      if (!t_ok) {
        out[i - 1] = -1;
      } else {
        double Z;
        if (d_ok && a->neighbours) {
          Z = orc_resample_weights_nbr(P, Q, omega, V, a->neighbours, a->nbr_k, (double)a->nbr_lambda, g);
        } else if (d_ok) {
          Z = orc_resample_weights(P, Q, omega, V, g);
        } else { /* f == 0 for every candidate: Eq. opt_G gives P */
          Z = 0.0;
          for (int x = 0; x < V; ++x) {
            g[x] = P[x];
            Z += P[x];
          }
        }
        if (!(Z > 0.0)) {
          status |= ORC_STATUS_ZFALLBACK;
          Z = 0.0;
          for (int x = 0; x < V; ++x) {
            g[x] = P[x];
            Z += P[x];
          }
        }
        double mg = INFINITY;
        out[i - 1] = orc_inverse_cdf(g, V, Z, u, &mg);
        if (a->margin_cdf) a->margin_cdf[b] = mg;
        if (a->G)
          for (int x = 0; x < V; ++x) a->G[(int64_t)b * V + x] = g[x] / Z;
      }
      emitted = 1;
      break;
    }
  }

  if (!emitted && tau == L && a->target_rows == L + 1) {
    /* bonus token x_{L+1} ~ P(. | x_{1:L}) */
    const int64_t t_off = (int64_t)b * a->target_batch_stride + (int64_t)L * V;
    orc_prepare_row(a->target_logits, a->target_uncond, a->dtype, t_off, V, a->cfg_scale, a->top_k,
                    zt, scratch);
    if (orc_softmax(zt, V, P)) {
      double Z = 0.0;
      for (int x = 0; x < V; ++x) Z += P[x];
      double mg = INFINITY;
      out[L] = orc_inverse_cdf(P, V, Z, u, &mg);
      if (a->margin_cdf) a->margin_cdf[b] = mg;
      if (a->G)
        for (int x = 0; x < V; ++x) a->G[(int64_t)b * V + x] = P[x] / Z;
    } else {
      status |= ORC_STATUS_BADROW;
      out[L] = -1;
    }
  }
  a->out_accept_len[b] = tau;
  if (a->out_status) a->out_status[b] = status;

  /* Diagnostics for comparison only (not part of the procedure): p, q, f at
   * every position, including those after the first rejection. */
  if (a->p || a->q || a->f || a->accept_mass || a->bound_term) {
    for (int i = 1; i <= L; ++i) {
      const int64_t t_off = (int64_t)b * a->target_batch_stride + (int64_t)(i - 1) * V;
      const int64_t d_off = (int64_t)b * a->draft_batch_stride + (int64_t)(i - 1) * V;
      orc_prepare_row(a->target_logits, a->target_uncond, a->dtype, t_off, V, a->cfg_scale,
                      a->top_k, zt, scratch);
      orc_prepare_row(a->draft_logits, a->draft_uncond, a->dtype, d_off, V, a->cfg_scale, a->top_k,
                      zd, scratch);
      const int t_ok = orc_softmax(zt, V, P);
      const int d_ok = orc_softmax(zd, V, Q);
      const int x_i = tok[i - 1];
      const int ok = t_ok && d_ok && x_i >= 0 && x_i < V;
      const int64_t o = (int64_t)b * L + (i - 1);
      double pv = ok ? P[x_i] : NAN;
      const double qv = ok ? Q[x_i] : NAN;
      if (ok && a->neighbours) /* the mass the test used */
        pv = orc_neighbour_mass(P, V, a->neighbours + (int64_t)x_i * a->nbr_k, a->nbr_k, (double)a->nbr_lambda, x_i);
      if (a->p) a->p[o] = pv;
      if (a->q) a->q[o] = qv;
      if (a->f) a->f[o] = ok ? orc_accept_prob(pv, qv, (double)a->relax_schedule[i - 1]) : 0.0;
      if (a->accept_mass || a->bound_term) {
        double am = NAN, bt = NAN;
        if (t_ok && d_ok) orc_position_terms(P, Q, (double)a->relax_schedule[i - 1], V, &am, &bt);
        if (a->accept_mass) a->accept_mass[o] = am;
        if (a->bound_term) a->bound_term[o] = bt;
      }
    }
  }
}

/* ---- Tree-structured drafts ------------------------------------------------------------------
 * The paper's experiments draft a static tree of candidates (Experiments, "Implementation Details");
 * Algorithm 1 states the chain.  The paper gives no rule for several candidate children of one node
 * under the relaxed test, so this is the build's reading, chosen so that it contains Algorithm 1 and
 * stays lossless at omega == 1 (Theorem 1):
 *   - The candidates of a node are drawn independently from the drafter's distribution Q in that
 *     node's context (with replacement), and are tried in their stored order.
 *   - With P' the target's distribution in that context, a candidate x at level i is accepted with
 *     probability f = min{1, omega_i P'(x)/Q(x)} (Eq. relax on the current residual).  On a rejection
 *     the residual becomes P' <- Norm([P' - Q f(.)]_+), i.e. Eq. opt_G applied to P' (for omega_i = 1
 *     this is the recursive rejection sampling of multi-candidate speculative decoding), and the next
 *     sibling is tried against it with the same Q.
 *   - An accepted candidate becomes the context of the next level; a node without children ends
 *     the walk with a bonus token from the target's distribution there (Algorithm 1, last step).
 *   - When every candidate of a node has been rejected, the emitted token is drawn from the final
 *     residual by inverse CDF with the sequence's one extra uniform.
 * A chain (every node the only child of the previous one) is Algorithm 1 itself: the arithmetic below
 * is then, operation for operation, that of verify_one.
 *
 * Layout: contexts are numbered 0 (the root: the prefix alone) and n + 1 (after node n); row c of
 * target_logits / draft_logits is the model's output in context c.  parent[n] is -1 for a child of the
 * root, else the index of an EARLIER node.  Siblings are tried in increasing node index.
 */
typedef struct {
  const void *target_logits; /* [B, N+1, V] */
  const void *draft_logits;  /* [B, N+1, V] (rows of contexts without children are not read) */
  const void *target_uncond; /* NULL: no guidance mix */
  const void *draft_uncond;
  int32_t dtype;
  float cfg_scale;
  int32_t top_k;
  int32_t B, N, V, D;          /* N nodes; D = deepest level (the root's children are level 1) */
  const int32_t *parent;       /* [N] */
  const int32_t *draft_tokens; /* [B, N] */
  const float *uniforms;       /* [B, N+1]: the accept draw of every node, then the resample / bonus draw */
  const float *relax_schedule; /* [D] omega of levels 1..D */
  int32_t *out_tokens;         /* [B, D+1]: accepted path, then the drawn token, then -1 */
  int32_t *out_accept_len;     /* [B] number of accepted levels */
  int32_t *out_nodes;          /* [B, D] or NULL: the node accepted at each level, then -1 */
  int32_t *out_status;         /* [B] or NULL */
  double *G;                   /* [B, V] or NULL: distribution the emitted token was drawn from */
  double *margin_accept;       /* [B, N] or NULL: |r - f| where the test ran on usable data, else +inf */
  double *margin_cdf;          /* [B] or NULL */
} orc_tree_params;

static void verify_tree_one(const orc_tree_params *a, int b, double *zt, double *zd, double *P, double *Q,
                            double *g, double *scratch) {
  const int N = a->N, V = a->V, D = a->D;
  const int64_t stride = (int64_t)(N + 1) * V;
  const int32_t *tok = a->draft_tokens + (int64_t)b * N;
  const float *unif = a->uniforms + (int64_t)b * (N + 1);
  int32_t *out = a->out_tokens + (int64_t)b * (D + 1);
  for (int i = 0; i <= D; ++i) out[i] = -1;
  if (a->out_nodes)
    for (int i = 0; i < D; ++i) a->out_nodes[(int64_t)b * D + i] = -1;
  if (a->margin_accept)
    for (int n = 0; n < N; ++n) a->margin_accept[(int64_t)b * N + n] = INFINITY;
  if (a->margin_cdf) a->margin_cdf[b] = INFINITY;
  if (a->G)
    for (int x = 0; x < V; ++x) a->G[(int64_t)b * V + x] = 0.0;

  const double u = (double)unif[N];
  int status = 0, level = 0, ctx = 0; /* ctx: 0 root, n+1 after node n */
  for (;;) {
    const int64_t off = (int64_t)b * stride + (int64_t)ctx * V;
    orc_prepare_row(a->target_logits, a->target_uncond, a->dtype, off, V, a->cfg_scale, a->top_k, zt, scratch);
    const int t_ok = orc_softmax(zt, V, P);
    int first_child = -1;
    for (int n = 0; n < N; ++n)
      if (a->parent[n] == ctx - 1) { first_child = n; break; }
    if (first_child < 0 || level >= D) {
      /* a leaf: bonus token from the target's distribution in this context */
      if (t_ok) {
        double Z = 0.0;
        for (int x = 0; x < V; ++x) Z += P[x];
        double mg = INFINITY;
        out[level] = orc_inverse_cdf(P, V, Z, u, &mg);
        if (a->margin_cdf) a->margin_cdf[b] = mg;
        if (a->G)
          for (int x = 0; x < V; ++x) a->G[(int64_t)b * V + x] = P[x] / Z;
      } else {
        status |= ORC_STATUS_BADROW;
        out[level] = -1;
      }
      break;
    }
    orc_prepare_row(a->draft_logits, a->draft_uncond, a->dtype, off, V, a->cfg_scale, a->top_k, zd, scratch);
    const int d_ok = orc_softmax(zd, V, Q);
    const double omega = (double)a->relax_schedule[level];
    /* the residual starts as the target's distribution; g, Z hold it unnormalised after a rejection */
    int have_g = 0, accepted = -1;
    double Z = 1.0;
    for (int n = first_child; n < N; ++n) {
      if (a->parent[n] != ctx - 1) continue;
      const int x_n = tok[n];
      const int tok_ok = (x_n >= 0 && x_n < V);
      double f;
      if (!t_ok || !d_ok) {
        f = 0.0;
        status |= ORC_STATUS_BADROW;
      } else if (!tok_ok) {
        f = 0.0;
        status |= ORC_STATUS_BADTOKEN;
      } else {
        f = orc_accept_prob(P[x_n], Q[x_n], omega);
      }
      const double r = (double)unif[n];
      if (a->margin_accept && t_ok && d_ok && tok_ok) a->margin_accept[(int64_t)b * N + n] = fabs(r - f);
      if (r <= f) { accepted = n; break; }
      if (!t_ok) continue; /* nothing to update: the emitted token will be -1 */
      /* rejected: the residual becomes Eq. opt_G of the current residual */
      if (d_ok) {
        Z = orc_resample_weights(P, Q, omega, V, g);
      } else { /* f == 0 for every candidate: Eq. opt_G leaves the residual as it is */
        Z = 0.0;
        for (int x = 0; x < V; ++x) { g[x] = P[x]; Z += P[x]; }
      }
      if (!(Z > 0.0)) {
        status |= ORC_STATUS_ZFALLBACK;
        Z = 0.0;
        for (int x = 0; x < V; ++x) { g[x] = P[x]; Z += P[x]; }
      }
      have_g = 1;
      /* the next sibling is tested against the normalised residual */
      int more = 0;
      for (int m = n + 1; m < N; ++m)
        if (a->parent[m] == ctx - 1) { more = 1; break; }
      if (more)
        for (int x = 0; x < V; ++x) P[x] = g[x] / Z;
    }
    if (accepted >= 0) {
      out[level] = tok[accepted];
      if (a->out_nodes) a->out_nodes[(int64_t)b * D + level] = accepted;
      ++level;
      ctx = accepted + 1;
      continue;
    }
    /* every candidate rejected: draw from the residual */
    if (!t_ok) {
      out[level] = -1;
    } else {
      double mg = INFINITY;
      (void)have_g; /* at least one candidate was rejected, so g and Z are set */
      out[level] = orc_inverse_cdf(g, V, Z, u, &mg);
      if (a->margin_cdf) a->margin_cdf[b] = mg;
      if (a->G)
        for (int x = 0; x < V; ++x) a->G[(int64_t)b * V + x] = g[x] / Z;
    }
    break;
  }
  a->out_accept_len[b] = level;
  if (a->out_status) a->out_status[b] = status;
}

/* Batched driver of the tree walk.  Returns 0, -1 on bad shapes or a malformed tree (a parent that is
 * not an earlier node, a level beyond D), -2 if memory could not be had. */
int orc_verify_tree(const orc_tree_params *a) {
  if (!a || a->B < 1 || a->N < 1 || a->V < 2 || a->D < 1 || !a->parent) return -1;
  for (int n = 0; n < a->N; ++n) {
    if (a->parent[n] < -1 || a->parent[n] >= n) return -1;
    int level = 1;
    for (int p = a->parent[n]; p >= 0; p = a->parent[p]) ++level;
    if (level > a->D) return -1;
  }
  int failed = 0;
#ifdef _OPENMP
#pragma omp parallel
#endif
  {
    const size_t V = (size_t)a->V;
    double *buf = (double *)malloc(6 * V * sizeof(double));
    if (!buf) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
      failed = 1;
    }
#ifdef _OPENMP
#pragma omp barrier
#endif
    if (!failed) {
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
      for (int b = 0; b < a->B; ++b)
        verify_tree_one(a, b, buf, buf + V, buf + 2 * V, buf + 3 * V, buf + 4 * V, buf + 5 * V);
    }
    free(buf);
  }
  return failed ? -2 : 0;
}

/* ---- Algorithm 1, drafting stage: one token per row -------------------------------------------
 * x~ ~ Q(. | prefix): for each of R rows of logits (prepared like the verification's rows: optional
 * guidance mix in fp32, optional top-k), the softmax and one inverse-CDF draw with the row's supplied
 * uniform (same convention as the verification's draws).  out_tokens[r] = -1 and status bit BADROW for
 * an unusable row.  margin[r] (optional) is the distance of u to the nearest CDF boundary of the pick.
 * Returns 0, or -1 on bad shapes, -2 if memory could not be had. */
int orc_sample_rows(const void *logits, const void *uncond, int dtype, float cfg_scale, int top_k, int R,
                    int V, int64_t row_stride, const float *uniforms, int32_t *out_tokens,
                    int32_t *out_status, double *margin) {
  if (!logits || !uniforms || !out_tokens || R < 1 || V < 2 || row_stride < V) return -1;
  double *buf = (double *)malloc(3 * (size_t)V * sizeof(double));
  if (!buf) return -2;
  double *z = buf, *P = buf + V, *scratch = buf + 2 * (size_t)V;
  for (int r = 0; r < R; ++r) {
    orc_prepare_row(logits, uncond, dtype, (int64_t)r * row_stride, V, cfg_scale, top_k, z, scratch);
    int status = 0;
    double mg = INFINITY;
    if (orc_softmax(z, V, P)) {
      double Z = 0.0;
      for (int x = 0; x < V; ++x) Z += P[x];
      out_tokens[r] = orc_inverse_cdf(P, V, Z, (double)uniforms[r], &mg);
    } else {
      out_tokens[r] = -1;
      status = ORC_STATUS_BADROW;
    }
    if (out_status) out_status[r] = status;
    if (margin) margin[r] = mg;
  }
  free(buf);
  return 0;
}

/* Batched driver: sequences are independent.  Returns 0, or -1 on bad shapes,
 * -2 if memory could not be had. */
int orc_verify(const orc_params *a) {
  if (!a || a->B < 1 || a->gamma < 1 || a->V < 2) return -1;
  if (a->target_rows != a->gamma && a->target_rows != a->gamma + 1) return -1;
  int failed = 0;
#ifdef _OPENMP
#pragma omp parallel
#endif
  {
    const size_t V = (size_t)a->V;
    double *buf = (double *)malloc(6 * V * sizeof(double));
    if (!buf) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
      failed = 1;
    }
#ifdef _OPENMP
#pragma omp barrier
#endif
    if (!failed) {
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
      for (int b = 0; b < a->B; ++b)
        verify_one(a, b, buf, buf + V, buf + 2 * V, buf + 3 * V, buf + 4 * V, buf + 5 * V);
    }
    free(buf);
  }
  return failed ? -2 : 0;
}
