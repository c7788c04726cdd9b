/*
 * SpecSteer verify + recover: plain CPU oracle (float64).
 *
 * THIS FILE IS TEST INFRASTRUCTURE, NOT PRODUCT CODE.  It is a slow, obviously
 * correct restatement of one Draft-Verify-Recover round as the paper defines
 * it, used only to check the CUDA library and as the timed CPU baseline.  It
 * shares no code, header, table or constant with the CUDA path and nothing in
 * the product may call it.
 *
 * What it follows (SpecSteer, arXiv 2603.16219):
 *   - Algorithm 1, Phase 2/3: for t = 1..K compute alpha_t, accept while
 *     Uniform(0,1) <= alpha_t, on the first rejection sample one token from
 *     Softmax(h_rec) and stop.
 *   - Eq. 7 (ratio rule):   alpha = min(1, P_LLM(y) / (lambda * P_SLM-(y))).
 *   - Eq. 6 (exact rule):   alpha = min(1, P*(y) / P_SLM+(y)) with the true Z_t.
 *   - Eq. 2-4 (fused target): P* = P_LLM * exp(r) / Z_t, r = log P+ - log P-.
 *   - Eq. 8 (recovery logits): h_rec = h_LLM + beta * (h_SLM+ - h_SLM-).
 *   - Greedy decoding (the experimental settings): ORACLE_RECOVER_ARGMAX takes the
 *     token of largest h_rec (Eq. 8, over the reals: ordered in double) instead of
 *     sampling, and reports the gap to the runner-up; the single-precision ordering
 *     the CUDA library documents as its tie-break is reported beside it, not used.
 *   - ORACLE_FLAG_ALG1_READS: the round reading exactly what Algorithm 1 reads:
 *     h_LLM and h_SLM- on the drafted rows (Eq. 7), all three tensors only on the
 *     row the new token comes from (Eq. 8).  h_SLM+ on a drafted row is never touched.
 * Every distribution is a softmax of logits divided by a per-request
 * temperature (the paper runs at temperature 1).  Logits may also be given in
 * double (ORACLE_DTYPE_F64): the LM-head oracle in __init__.py forms them as
 * x W^T in float64 and hands them to the same round.
 *
 * Pins (tests/test_oracle_pins.py, tests/golden/): special cases that reduce
 * to library log-softmax, hand-derived rational examples, the output-token law
 * by enumeration and Monte-Carlo, and the speculative-sampling theorem for the
 * EXACT_Z + RESIDUAL pair; greedy recovery by exact rationals, numpy argmax and
 * a pair that only double precision separates; the Algorithm-1-reads round by
 * equality with the full round on finite inputs and by poisoning what it must not
 * read; the float64 logit decode and the LM-head step in
 * tests/test_oracle_lmhead_pins.py.  Parts with no pin: none of the functions below.
 *
 * No blocking, fusion or reordering: each log-sum-exp is "max, then sum of
 * exp(x - max)" over the row in vocabulary order; the sampler walks the CDF in
 * vocabulary order.  OpenMP, if enabled, only runs different requests on
 * different threads.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#include "specsteer_oracle.h"

/* ---- input decoding: logits are upcast exactly to double ---- */
static double logit_at(const void *base, int dtype, int64_t idx) {
  if (dtype == ORACLE_DTYPE_F32) {
    return (double)((const float *)base)[idx];
  } else if (dtype == ORACLE_DTYPE_F64) { /* logits that were themselves computed in double (the LM-head path) */
    return ((const double *)base)[idx];
  } else { /* bf16: the upper 16 bits of an IEEE float32 */
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
  }
}

/* log(sum_i exp(x_i)), max-subtracted.  All -inf -> -inf; any NaN or +inf -> non-finite. */
double specsteer_oracle_logsumexp(const double *x, int64_t n) {
  double mx = -INFINITY;
  int has_nan = 0;
  for (int64_t i = 0; i < n; ++i) {
    if (isnan(x[i])) has_nan = 1;
    else if (x[i] > mx) mx = x[i];
  }
  if (has_nan) return NAN;
  if (mx == -INFINITY) return -INFINITY;
  if (mx == INFINITY) return INFINITY;
  double s = 0.0;
  for (int64_t i = 0; i < n; ++i) s += exp(x[i] - mx);
  return mx + log(s);
}

/* One row's tempered logits and the four normalisers.
 * ell = h_LLM/T, p = h_SLM+/T, m = h_SLM-/T, r = ell + beta*(p - m)   (Eq. 8, tempered). */
typedef struct {
  double *ell, *p, *m, *r;
  double lseL, lseP, lseM, lseR;
} row_t;

static void row_load(row_t *w, int V, int dtype, const void *hl, const void *hp, const void *hm,
                     int64_t off, double beta, double T) {
  for (int v = 0; v < V; ++v) {
    w->ell[v] = logit_at(hl, dtype, off + v) / T;
    w->p[v] = logit_at(hp, dtype, off + v) / T;
    w->m[v] = logit_at(hm, dtype, off + v) / T;
    w->r[v] = w->ell[v] + beta * (w->p[v] - w->m[v]);
  }
  w->lseL = specsteer_oracle_logsumexp(w->ell, V);
  w->lseP = specsteer_oracle_logsumexp(w->p, V);
  w->lseM = specsteer_oracle_logsumexp(w->m, V);
  w->lseR = specsteer_oracle_logsumexp(w->r, V);
}

/* What Eq. 7 reads of a drafted row: h_LLM and h_SLM- alone.  Everything that involves h_SLM+ is left NaN. */
static void row_load_ratio(row_t *w, int V, int dtype, const void *hl, const void *hm, int64_t off, double T) {
  for (int v = 0; v < V; ++v) {
    w->ell[v] = logit_at(hl, dtype, off + v) / T;
    w->m[v] = logit_at(hm, dtype, off + v) / T;
    w->p[v] = NAN;
    w->r[v] = NAN;
  }
  w->lseL = specsteer_oracle_logsumexp(w->ell, V);
  w->lseM = specsteer_oracle_logsumexp(w->m, V);
  w->lseP = NAN;
  w->lseR = NAN;
}

static int row_finite(const row_t *w) {
  return isfinite(w->lseL) && isfinite(w->lseP) && isfinite(w->lseM) && isfinite(w->lseR);
}

/* Recovery weights of one row (unnormalised), into wgt[V]; returns W = sum.
 * STEER:    w(v) = Softmax(h_rec)(v)                       (Algorithm 1 line "Sample y_new"; Eq. 8)
 * RESIDUAL: w(v) = max(0, Softmax(h_rec)(v) - P_SLM+(v))    (speculative-sampling residual over the fused target) */
static double recovery_weights(const row_t *w, int V, int mode, double *wgt) {
  double W = 0.0;
  for (int v = 0; v < V; ++v) {
    double ps = exp(w->r[v] - w->lseR);
    double x = ps;
    if (mode == ORACLE_RECOVER_RESIDUAL) {
      x = ps - exp(w->p[v] - w->lseP);
      if (!(x > 0.0)) x = 0.0;
    }
    wgt[v] = x;
    W += x;
  }
  return W;
}

/* Inverse CDF in vocabulary order: min{ v : sum_{j<=v} w(j) > target }, else the last v with w(v) > 0. */
static int cdf_pick(const double *wgt, int V, double target) {
  double c = 0.0;
  int last_pos = -1;
  for (int v = 0; v < V; ++v) {
    if (wgt[v] > 0.0) last_pos = v;
    c += wgt[v];
    if (c > target) return v;
  }
  return last_pos;
}

int specsteer_oracle_row(int V, int dtype, const void *h_llm, const void *h_plus, const void *h_minus,
                         double beta, double T, int recover_mode,
                         double *lse4, double *logp_star_full, double *weights, double *W_out) {
  row_t w;
  w.ell = (double *)malloc(sizeof(double) * 4 * (size_t)V);
  if (!w.ell) return -1;
  w.p = w.ell + V; w.m = w.p + V; w.r = w.m + V;
  row_load(&w, V, dtype, h_llm, h_plus, h_minus, 0, beta, T);
  if (lse4) { lse4[0] = w.lseL; lse4[1] = w.lseP; lse4[2] = w.lseM; lse4[3] = w.lseR; }
  if (logp_star_full) for (int v = 0; v < V; ++v) logp_star_full[v] = w.r[v] - w.lseR;
  if (weights) {
    double W = recovery_weights(&w, V, recover_mode, weights);
    if (W_out) *W_out = W;
  }
  free(w.ell);
  return 0;
}

static void one_request(const oracle_round_args *a, int b, row_t *w, double *wgt) {
  const int K = a->K, V = a->V;
  const double lam = (double)a->lambda[b], beta = (double)a->beta[b], T = (double)a->temperature[b];
  int status = 0;
  int len = a->draft_len[b];
  const int32_t *yhat = a->draft_tokens + (int64_t)b * K;

  /* defaults for every output slot of this request */
  for (int t = 0; t < K; ++t) {
    int64_t i = (int64_t)b * K + t;
    if (a->accept_flags) a->accept_flags[i] = 0;
    if (a->alpha) a->alpha[i] = 0.0;
    if (a->logp_llm) a->logp_llm[i] = NAN;
    if (a->logp_minus) a->logp_minus[i] = NAN;
    if (a->logp_plus) a->logp_plus[i] = NAN;
    if (a->logp_star) a->logp_star[i] = NAN;
    if (a->accept_margin) a->accept_margin[i] = INFINITY;
  }
  for (int t = 0; t <= K; ++t) {
    if (a->log_z) a->log_z[(int64_t)b * (K + 1) + t] = NAN;
    if (a->out_tokens) a->out_tokens[(int64_t)b * (K + 1) + t] = -1;
  }
  if (a->cdf_margin) a->cdf_margin[b] = INFINITY;
  if (a->rec_token_lo) a->rec_token_lo[b] = -1;
  if (a->rec_token_hi) a->rec_token_hi[b] = -1;
  int rec_token = -1, n_out = 0, n = 0;
  int decided = 0, stop_nonfinite = 0;
  double rec_logprob = NAN;

  /* every problem the request shows is reported: a bad length and a bad parameter give both bits */
  const int alg1 = (a->flags & ORACLE_FLAG_ALG1_READS) != 0;
  if (len < 0 || len > K) { status |= ORACLE_REQ_BAD_LEN; len = 0; }
  int params_ok = isfinite(T) && T > 0.0 && isfinite(lam) && lam > 0.0 && isfinite(beta);
  if (!params_ok) {
    status |= ORACLE_REQ_BAD_PARAM;
    goto done;
  }

  /* Algorithm 1, the for-loop over draft positions.  The decision (n) is fixed at the first
   * rejection; later drafted rows are still evaluated so that their per-position diagnostics
   * (alpha, log-probs) are defined, but they change neither n nor the status. */
  n = len;
  for (int t = 0; t < len; ++t) {
    int64_t off = (int64_t)b * a->ld_req + (int64_t)t * a->ld_row;
    int64_t i = (int64_t)b * K + t;
    int fin;
    if (alg1) {   /* Algorithm 1's verification: the cloud holds h_LLM and h_SLM- only (Eq. 7) */
      row_load_ratio(w, V, a->dtype, a->h_llm, a->h_slm_minus, off, T);
      fin = isfinite(w->lseL) && isfinite(w->lseM);
    } else {
      row_load(w, V, a->dtype, a->h_llm, a->h_slm_plus, a->h_slm_minus, off, beta, T);
      fin = row_finite(w);
    }
    if (!fin) {
      if (!decided) { status |= ORACLE_REQ_NONFINITE; n = t; decided = 1; stop_nonfinite = 1; }
      continue;
    }
    double logZ = w->lseR - w->lseL - beta * (w->lseP - w->lseM);  /* log sum_v P_LLM (P+/P-)^beta; Eq. 2 at beta=1 */
    if (a->log_z && !alg1) a->log_z[(int64_t)b * (K + 1) + t] = logZ;
    int y = yhat[t];
    double al = 0.0, rho = 0.0;
    int accept, testable = 1;   /* a bad token or an undefined ratio is a rejection whatever the uniform */
    if (y < 0 || y >= V) {
      if (!decided) status |= ORACLE_REQ_BAD_TOKEN;
      al = 0.0; rho = 0.0; testable = 0;
    } else {
      double logpL = w->ell[y] - w->lseL, logpM = w->m[y] - w->lseM;
      double logpP = w->p[y] - w->lseP, logpS = w->r[y] - w->lseR;
      if (a->logp_llm) a->logp_llm[i] = logpL;
      if (a->logp_minus) a->logp_minus[i] = logpM;
      if (a->logp_plus && !alg1) a->logp_plus[i] = logpP;
      if (a->logp_star && !alg1) a->logp_star[i] = logpS;
      double logrho = (a->accept_mode == ORACLE_ACCEPT_RATIO)
                          ? (logpL - logpM - log(lam))   /* Eq. 7 */
                          : (logpS - logpP);             /* Eq. 6 */
      if (isnan(logrho)) { rho = 0.0; al = 0.0; testable = 0; }
      else { rho = exp(logrho); al = exp(fmin(0.0, logrho)); }
    }
    double u = (double)a->u_accept[i];
    accept = testable && (u <= al);                   /* Algorithm 1: "Uniform(0,1) <= alpha_t" */
    if (a->alpha) a->alpha[i] = al;
    if (a->accept_margin)
      a->accept_margin[i] = !testable ? INFINITY : (rho < 1.0) ? fabs(u - rho) : fmax(rho - 1.0, 1.0 - u);
    if (a->force_accept && a->force_accept[i] >= 0) accept = a->force_accept[i] ? 1 : 0;
    if (a->accept_flags) a->accept_flags[i] = (uint8_t)accept;
    if (!decided && !accept) { n = t; decided = 1; }
  }

  for (int t = 0; t < n; ++t) if (a->out_tokens) a->out_tokens[(int64_t)b * (K + 1) + t] = yhat[t];
  n_out = n;
  /* diagnostic: with FLAG_BONUS row `len` belongs to the round, so its log Z_t is reported whatever n is */
  if ((a->flags & ORACLE_FLAG_BONUS) && a->log_z && !alg1) {
    row_load(w, V, a->dtype, a->h_llm, a->h_slm_plus, a->h_slm_minus,
             (int64_t)b * a->ld_req + (int64_t)len * a->ld_row, beta, T);
    if (row_finite(w)) a->log_z[(int64_t)b * (K + 1) + len] = w->lseR - w->lseL - beta * (w->lseP - w->lseM);
  }
  if (stop_nonfinite) goto done;

  /* Phase 3: recovery at the first rejection; with FLAG_BONUS also one token from row len when all were accepted. */
  if (n < len || (a->flags & ORACLE_FLAG_BONUS)) {
    int64_t off = (int64_t)b * a->ld_req + (int64_t)n * a->ld_row;
    row_load(w, V, a->dtype, a->h_llm, a->h_slm_plus, a->h_slm_minus, off, beta, T);
    if (!row_finite(w)) { status |= ORACLE_REQ_NONFINITE; goto done; }
    if (a->recover_mode == ORACLE_RECOVER_ARGMAX) {
      /* Greedy decoding (the paper's experimental setting): y_new is the token of largest h_rec (Eq. 8), the lowest
       * id among equals, on the rejection row and on the bonus row alike; the temperature does not change the order.
       * Its log-probability is the one under Softmax(h_rec / T). */
      /* The order of Eq. 8 over the reals: h_rec is formed and compared in double from the exactly upcast logits.
       * cdf_margin reports the gap between the largest and the second largest value (0 for an exact tie), so that a
       * comparison can tell a decided order from one that rounding in a narrower type may turn around. */
      double best = -INFINITY, second = -INFINITY;
      for (int v = 0; v < V; ++v) {
        double r = logit_at(a->h_llm, a->dtype, off + v) +
                   beta * (logit_at(a->h_slm_plus, a->dtype, off + v) - logit_at(a->h_slm_minus, a->dtype, off + v));
        if (rec_token < 0 || r > best) { second = best; best = r; rec_token = v; }
        else if (r > second) second = r;
      }
      double gap = best - second;
      /* Beside it, not used for anything above: the token the single-precision form of Eq. 8 would order first,
       * fl(h_LLM + beta * fl(h_SLM+ - h_SLM-)) with one fused multiply-add, lowest id among equals - the rule the CUDA
       * library documents for breaking what double precision calls a near-tie.  Reported in rec_token_lo. */
      int tie_token = rec_token;
      if (a->dtype != ORACLE_DTYPE_F64) {
        const float beta32 = a->beta[b];
        float best32 = -INFINITY;
        tie_token = -1;
        for (int v = 0; v < V; ++v) {
          float l = (float)logit_at(a->h_llm, a->dtype, off + v), pp = (float)logit_at(a->h_slm_plus, a->dtype, off + v),
                mm = (float)logit_at(a->h_slm_minus, a->dtype, off + v);
          float r = fmaf(beta32, pp - mm, l);
          if (tie_token < 0 || r > best32) { best32 = r; tie_token = v; }
        }
      }
      rec_logprob = w->r[rec_token] - w->lseR;
      if (a->out_tokens) a->out_tokens[(int64_t)b * (K + 1) + n] = rec_token;
      n_out = n + 1;
      if (a->cdf_margin) a->cdf_margin[b] = gap;   /* no uniform is involved */
      if (a->rec_token_lo) a->rec_token_lo[b] = tie_token;
      if (a->rec_token_hi) a->rec_token_hi[b] = rec_token;
      goto done;
    }
    int mode = (n < len) ? a->recover_mode : ORACLE_RECOVER_STEER;
    double W = recovery_weights(w, V, mode, wgt);
    if (mode == ORACLE_RECOVER_RESIDUAL && !(W > 0.0)) {
      status |= ORACLE_REQ_RESIDUAL_EMPTY;
      W = recovery_weights(w, V, ORACLE_RECOVER_STEER, wgt);
    }
    double u = (double)a->u_recover[b];
    double target = u * W;
    rec_token = cdf_pick(wgt, V, target);
    if (rec_token >= 0) {
      rec_logprob = log(wgt[rec_token] / W);
      if (a->out_tokens) a->out_tokens[(int64_t)b * (K + 1) + n] = rec_token;
      n_out = n + 1;
      /* distance of the target from the chosen token's CDF interval, and the tokens within margin_tol */
      double c_lo = 0.0;
      for (int v = 0; v < rec_token; ++v) c_lo += wgt[v];
      double c_hi = c_lo + wgt[rec_token];
      if (a->cdf_margin) a->cdf_margin[b] = fmin(target - c_lo, c_hi - target) / W;
      double tol = a->margin_tol * W;
      if (a->rec_token_lo) { int v = cdf_pick(wgt, V, fmax(0.0, target - tol)); a->rec_token_lo[b] = v; }
      if (a->rec_token_hi) { int v = cdf_pick(wgt, V, target + tol); a->rec_token_hi[b] = v; }
    }
  }

done:
  a->accept_len[b] = n;
  if (a->rec_token) a->rec_token[b] = rec_token;
  if (a->rec_logprob) a->rec_logprob[b] = rec_logprob;
  if (a->n_out) a->n_out[b] = n_out;
  if (a->req_status) a->req_status[b] = status;
}

int specsteer_oracle_round(const oracle_round_args *a) {
  if (!a || a->B < 0 || a->K < 0 || a->V <= 0 || a->ld_row < a->V || !a->accept_len) return -1;
  if (a->ld_req < (int64_t)(a->K + 1) * a->ld_row) return -1;
  /* Eq. 6 needs P_SLM+ and Z_t on every drafted row: it cannot be evaluated from what Algorithm 1's verification reads */
  if ((a->flags & ORACLE_FLAG_ALG1_READS) && a->accept_mode != ORACLE_ACCEPT_RATIO) return -3;
  int nthreads = a->nthreads > 0 ? a->nthreads : 1;
  int failed = 0;
#ifdef _OPENMP
#pragma omp parallel num_threads(nthreads)
#endif
  {
    row_t w;
    double *buf = (double *)malloc(sizeof(double) * 5 * (size_t)a->V);
    if (!buf) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
      failed = 1;
    } else {
      w.ell = buf; w.p = buf + a->V; w.m = buf + 2 * (size_t)a->V; w.r = buf + 3 * (size_t)a->V;
      double *wgt = buf + 4 * (size_t)a->V;
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
      for (int b = 0; b < a->B; ++b) one_request(a, b, &w, wgt);
      free(buf);
    }
  }
  (void)nthreads;
  return failed ? -2 : 0;
}

int specsteer_oracle_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
