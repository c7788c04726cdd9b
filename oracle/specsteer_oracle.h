/*
 * Interface of the CPU oracle (test infrastructure only; see specsteer_oracle.c).
 * Deliberately separate from the CUDA library's header: the two share nothing.
 * All pointers are HOST pointers.  Floating-point outputs are double.
 */
#ifndef SPECSTEER_ORACLE_H
#define SPECSTEER_ORACLE_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORACLE_DTYPE_F32 = 0, ORACLE_DTYPE_BF16 = 1, ORACLE_DTYPE_F64 = 2 };
enum { ORACLE_ACCEPT_RATIO = 0 /* Eq. 7 */, ORACLE_ACCEPT_EXACT_Z = 1 /* Eq. 6 */ };
enum { ORACLE_RECOVER_STEER = 0 /* Eq. 8 softmax */, ORACLE_RECOVER_RESIDUAL = 1,
       ORACLE_RECOVER_ARGMAX = 2 /* greedy decoding: the token of largest h_rec (Eq. 8) */ };
enum { ORACLE_FLAG_BONUS = 1u,
       /* read what Algorithm 1 reads: h_LLM and h_SLM- on drafted rows (Eq. 7; RATIO only), all three tensors on the row
        * the new token comes from (Eq. 8).  logp_plus, logp_star and log_z are then not defined (NaN). */
       ORACLE_FLAG_ALG1_READS = 2u };
enum {
  ORACLE_REQ_BAD_TOKEN = 1, ORACLE_REQ_BAD_LEN = 2, ORACLE_REQ_NONFINITE = 4,
  ORACLE_REQ_RESIDUAL_EMPTY = 8, ORACLE_REQ_BAD_PARAM = 16
};

typedef struct {
  int32_t B, K, V;
  int64_t ld_row, ld_req;              /* strides in elements */
  int32_t dtype, accept_mode, recover_mode;
  uint32_t flags;
  int32_t nthreads;                    /* OpenMP threads over requests (>=1) */
  double margin_tol;                   /* width used for rec_token_lo/hi (e.g. 1e-5) */
  const void *h_llm, *h_slm_plus, *h_slm_minus;   /* [B][K+1][V] logits, f32 or bf16 bits */
  const int32_t *draft_tokens;         /* [B][K] */
  const int32_t *draft_len;            /* [B] */
  const float *lambda, *beta, *temperature;       /* [B] */
  const float *u_accept;               /* [B][K] */
  const float *u_recover;              /* [B] */
  const int8_t *force_accept;          /* optional [B][K]: -1 = decide by the uniform, 0/1 = forced decision */
  /* outputs; all optional except accept_len */
  int32_t *accept_len;                 /* [B] */
  uint8_t *accept_flags;               /* [B][K] */
  double *alpha, *logp_llm, *logp_minus, *logp_plus, *logp_star;   /* [B][K] */
  double *log_z;                       /* [B][K+1] */
  int32_t *rec_token; double *rec_logprob;        /* [B] */
  int32_t *out_tokens;                 /* [B][K+1] */
  int32_t *n_out, *req_status;         /* [B] */
  double *accept_margin;               /* [B][K]: distance of u from the decision boundary */
  double *cdf_margin;                  /* [B]: distance of the CDF target from the chosen interval's ends, / W;
                                          ARGMAX: the gap between the two largest h_rec, in double */
  int32_t *rec_token_lo, *rec_token_hi;/* [B]: tokens picked at target -/+ margin_tol*W; ARGMAX: lo = the token the
                                          single-precision form of Eq. 8 orders first (a tie-break rule, reported only) */
} oracle_round_args;

/* One whole round for B requests (Algorithm 1 phases 2 and 3).  Returns 0, or <0 on bad arguments / no memory. */
int specsteer_oracle_round(const oracle_round_args *a);

/* log(sum exp(x)) of n doubles. */
double specsteer_oracle_logsumexp(const double *x, int64_t n);

/* One row: lse4 = {lse_LLM, lse_SLM+, lse_SLM-, lse_rec}; logp_star_full[V] = log Softmax(h_rec);
 * weights[V] = unnormalised recovery weights for recover_mode, *W_out their sum.  Any output may be NULL. */
int specsteer_oracle_row(int V, int dtype, const void *h_llm, const void *h_plus, const void *h_minus,
                         double beta, double T, int recover_mode,
                         double *lse4, double *logp_star_full, double *weights, double *W_out);

int specsteer_oracle_max_threads(void);

/* ---- top-k split recovery (deployment appendix; specsteer_oracle_topk.c) ---- */
/* Cloud half, one row: the k largest entries of h_LLM - beta*h_SLM- (float32, one fused multiply-add), value
 * descending then token id ascending; slots beyond the number of non-NaN entries get id -1, value -inf. */
int specsteer_oracle_cloud_topk_row(int V, int dtype, const void *h_llm, const void *h_minus, float beta, int k,
                                    int32_t *idx_out, float *val_out);
/* Edge half, one row: adds beta*h_SLM+ on the kept entries, softmax at temperature T in float64, inverse CDF in
 * list order with uniform u.  token -1 when nothing can be sampled.  probs[k] and cdf_margin are optional. */
int specsteer_oracle_edge_resample_row(int V, int dtype, const void *h_plus, float beta, float T, int k,
                                       const int32_t *idx, const float *val, double u,
                                       int32_t *token, double *logprob, double *probs, double *cdf_margin);

#ifdef __cplusplus
}
#endif
#endif
