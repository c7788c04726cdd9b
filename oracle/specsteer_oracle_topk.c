/*
 * SpecSteer top-k split recovery: plain CPU oracle.
 *
 * THIS FILE IS TEST INFRASTRUCTURE, NOT PRODUCT CODE (same rules as specsteer_oracle.c: nothing in the
 * product may call it, and it shares nothing with the CUDA path).
 *
 * What it follows (SpecSteer, arXiv 2603.16219, appendix "System Deployment and Implementation Details",
 * item "Minimal Downlink (Steering Recovery)", case "If rejected"):
 *   - the cloud forms the non-private part of the recovery logits of Eq. 8,
 *         h_cloud = h_LLM - beta * h_SLM-,
 *     and keeps only the k entries with the highest values (the paper's example: k = 32);
 *   - the edge adds its private term beta * h_SLM+ on those k entries and resamples locally.
 * Readings where the paper is silent: h_cloud is formed in float32 by ONE fused multiply-add (that is the
 * precision in which the truncation is decided and the payload is sent); ties go to the lower token id;
 * NaN entries are never selected; the list is ordered by value, highest first; the edge divides the k
 * recovery logits by the request's temperature, takes their softmax in float64 and samples by inverse CDF
 * in list order with the caller's uniform (smallest j with cumulative weight > u*W, else the last j with
 * positive weight).
 *
 * Pins (tests/test_oracle_topk_pins.py): exact rational brute force on tiny rows, numpy sorting on rows
 * where the float32 arithmetic is exact, k >= V reducing to the full softmax of Eq. 8 (library log-softmax),
 * shift invariance, tie order, and the sampling law by a dense grid of uniforms.  Parts with no pin: none.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "specsteer_oracle.h"

static float logit32(const void *base, int dtype, int64_t i) {
  if (dtype == ORACLE_DTYPE_F32) return ((const float *)base)[i];
  uint32_t bits = ((uint32_t)((const uint16_t *)base)[i]) << 16;
  float f;
  memcpy(&f, &bits, sizeof f);
  return f;
}

typedef struct { float v; int32_t i; } entry_t;

/* value descending, then token id ascending */
static int entry_cmp(const void *pa, const void *pb) {
  const entry_t *a = (const entry_t *)pa, *b = (const entry_t *)pb;
  if (a->v > b->v) return -1;
  if (a->v < b->v) return 1;
  return (a->i > b->i) - (a->i < b->i);
}

int specsteer_oracle_cloud_topk_row(int V, int dtype, const void *h_llm, const void *h_minus, float beta, int k,
                                    int32_t *idx_out, float *val_out) {
  if (V <= 0 || k <= 0) return -1;
  entry_t *e = (entry_t *)malloc(sizeof(entry_t) * (size_t)V);
  if (!e) return -2;
  int n = 0;
  for (int v = 0; v < V; ++v) {
    float h = fmaf(-beta, logit32(h_minus, dtype, v), logit32(h_llm, dtype, v)); /* h_LLM - beta h_SLM-, float32 */
    if (h != h) continue;                                                        /* NaN: never selected */
    e[n].v = h; e[n].i = v; ++n;
  }
  qsort(e, (size_t)n, sizeof(entry_t), entry_cmp);
  for (int j = 0; j < k; ++j) {
    if (j < n) { idx_out[j] = e[j].i; val_out[j] = e[j].v; }
    else { idx_out[j] = -1; val_out[j] = -INFINITY; }
  }
  free(e);
  return 0;
}

int specsteer_oracle_edge_resample_row(int V, int dtype, const void *h_plus, float beta, float T, int k,
                                       const int32_t *idx, const float *val, double u,
                                       int32_t *token, double *logprob, double *probs, double *cdf_margin) {
  if (k <= 0 || !(T > 0.0f)) return -1;
  double *w = (double *)malloc(sizeof(double) * (size_t)k);
  if (!w) return -2;
  double mx = -INFINITY;
  for (int j = 0; j < k; ++j) {
    if (idx[j] < 0 || idx[j] >= V) { w[j] = -INFINITY; continue; }
    /* recovery logit of Eq. 8 on a kept entry: the cloud's part plus the private term, tempered */
    w[j] = ((double)val[j] + (double)beta * (double)logit32(h_plus, dtype, idx[j])) / (double)T;
    if (w[j] > mx) mx = w[j];
  }
  double W = 0.0;
  for (int j = 0; j < k; ++j) { w[j] = (w[j] == -INFINITY || w[j] != w[j]) ? ((w[j] != w[j]) ? NAN : 0.0) : exp(w[j] - mx); W += w[j]; }
  *token = -1;
  *logprob = NAN;
  if (cdf_margin) *cdf_margin = INFINITY;
  if (probs) for (int j = 0; j < k; ++j) probs[j] = (W > 0.0) ? w[j] / W : NAN;
  if (!(W > 0.0) || !isfinite(W)) { free(w); return 0; }   /* nothing to sample from */
  double target = u * W, c = 0.0;
  int pick = -1, last_pos = -1;
  double c_lo = 0.0;
  for (int j = 0; j < k; ++j) {
    if (w[j] > 0.0) last_pos = j;
    if (c + w[j] > target) { pick = j; c_lo = c; break; }
    c += w[j];
  }
  if (pick < 0) {
    pick = last_pos;
    c_lo = 0.0;
    for (int j = 0; j < pick; ++j) c_lo += w[j];
  }
  *token = idx[pick];
  *logprob = log(w[pick] / W);
  if (cdf_margin) *cdf_margin = fmin(target - c_lo, c_lo + w[pick] - target) / W;
  free(w);
  return 0;
}
