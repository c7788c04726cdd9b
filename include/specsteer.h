/*
 * specsteer.h - C ABI of the B200 (sm_100a) verify + recover step of SpecSteer's
 * Draft-Verify-Recover loop (arXiv 2603.16219).
 *
 * One "round" takes, for B requests and K+1 positions each, three logit tensors over
 * the full vocabulary V:
 *     h_llm        h_LLM   the cloud Generalist                         (Algorithm 1, "Compute logits")
 *     h_slm_plus   h_SLM+  the Specialist with private context           (Eq. 5, the drafter Q)
 *     h_slm_minus  h_SLM-  the Specialist without private context        (Eq. 3 baseline)
 * plus the K drafted token ids per request, and produces per request the number of
 * accepted drafts and one token sampled at the first rejection.
 *
 * Conventions for every entry point
 *   - Pointers inside specsteer_round_desc are DEVICE pointers unless the entry point
 *     says otherwise; all tensors are caller-owned and never freed or retained.
 *   - Logit tensors are [B][K+1][V], V contiguous; row t of request b starts at element
 *     b*ld_req + t*ld_row.  The fast path needs 16-byte aligned rows (base pointers,
 *     ld_row and ld_req all multiples of 16 bytes); otherwise a slower generic kernel runs.
 *   - Calls only enqueue work on the given CUDA stream (a cudaStream_t passed as void*;
 *     NULL = the legacy default stream).  They never synchronise and never copy to host.
 *   - Host-checkable mistakes return an error code and launch nothing.  Problems only the
 *     device can see set bits in req_status[b] and give the defined result stated below;
 *     no kernel traps or reads out of bounds because of input values.
 *   - Same inputs give bit-identical outputs from run to run.
 *   - One round may be in flight per context; contexts are independent.
 */
#ifndef SPECSTEER_H
#define SPECSTEER_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct specsteer_ctx specsteer_ctx; /* opaque, library-owned */

typedef enum {
  SPECSTEER_OK = 0,
  SPECSTEER_ERR_INVALID_ARG = 1, /* NULL required pointer, negative size, stride < V, unknown enum */
  SPECSTEER_ERR_UNSUPPORTED = 2, /* B, K or V beyond the maxima given to specsteer_ctx_create */
  SPECSTEER_ERR_WORKSPACE = 3,   /* device allocation failed */
  SPECSTEER_ERR_CUDA = 4,        /* a CUDA runtime call failed (launch error, wrong device) */
  SPECSTEER_ERR_ORDER = 5,       /* recover_sample without a preceding verify_round of the same shape */
  SPECSTEER_ERR_TIMEOUT = 6,     /* a bounded device-side wait gave up (reported by specsteer_ctx_device_error) */
  SPECSTEER_ERR_STATIC_LIMIT = 7 /* specsteer_verify_round_static: the shape does not fit the fixed scratch */
} specsteer_status;

typedef enum { SPECSTEER_F32 = 0, SPECSTEER_BF16 = 1 } specsteer_dtype;

/* How alpha_t is formed for drafted token y at position t.
 *   RATIO    alpha = min(1, P_LLM(y) / (lambda * P_SLM-(y)))                (Eq. 7; Algorithm 1)
 *   EXACT_Z  alpha = min(1, P*(y) / P_SLM+(y)) with the true partition Z_t  (Eq. 6) */
typedef enum { SPECSTEER_ACCEPT_RATIO = 0, SPECSTEER_ACCEPT_EXACT_Z = 1 } specsteer_accept_mode;

/* What is sampled at the first rejection.
 *   STEER     y ~ Softmax(h_LLM + beta (h_SLM+ - h_SLM-))                   (Eq. 8; Algorithm 1 Phase 3)
 *   RESIDUAL  y ~ normalise(max(0, Softmax(h_rec) - P_SLM+)), the speculative-sampling residual of the
 *             fused target; not in the paper, offered so that EXACT_Z + RESIDUAL emits exactly P*. */
typedef enum {
  SPECSTEER_RECOVER_STEER = 0,    /* y ~ Softmax(h_rec / T), Eq. 8 (Algorithm 1 as printed) */
  SPECSTEER_RECOVER_RESIDUAL = 1, /* y ~ norm(max(0, Softmax(h_rec / T) - P_SLM+)), an extension */
  SPECSTEER_RECOVER_ARGMAX = 2    /* greedy decoding, the paper's experimental setting: y = the token of largest h_rec
                                     (Eq. 8), lowest id among equals, on the rejection row and on the bonus row;
                                     h_rec is compared as float32 forms it, fl(h_LLM + beta * fl(h_SLM+ - h_SLM-)) with
                                     one fused multiply-add; u_recover is not used; rec_logprob is its log-probability
                                     under Softmax(h_rec / T).  One more pass over row accept_len of every request
                                     that takes a token (in the LM-head round: none, the tensor-core pass leaves the
                                     largest h_rec of every tile; the order is then that of its float32 accumulators).
                                     In the sharded rounds: specsteer_shard_greedy_local / _finish. */
} specsteer_recover_mode;

enum {
  SPECSTEER_FLAG_BONUS = 1u,    /* when all drafts are accepted, also sample one token (STEER) from row draft_len */
  SPECSTEER_FLAG_TWO_PHASE = 2u, /* take the two-phase round (see the outputs below) whenever it is eligible, however
                                   small the batch; without it the library takes it from 128 MB of logits upwards,
                                   below which its two extra launches cost more than the bytes it saves */
  SPECSTEER_FLAG_SEPARATE_LAUNCHES = 4u, /* keep verification and recovery in launches of their own.  Without it, when
                                   recovery is the STEER sample, u_recover is given and the round is not two-phase,
                                   the launch that runs the verification epilogue also samples the recovery token:
                                   specsteer_verify_round then writes rec_token, rec_logprob, out_tokens and n_out
                                   as well, and the specsteer_recover_sample that follows launches nothing.  A round
                                   of ONE request (below 128 MB of logits, 16-byte aligned rows) runs in a single
                                   launch altogether.  Same outputs, bit for bit.
                                   Set it when something else than specsteer_recover_sample follows
                                   (specsteer_cloud_topk: the sample would be wasted work) or when the recovery outputs
                                   must not be written before that call. */
  SPECSTEER_FLAG_ONE_LAUNCH = 8u /* take the one-launch round for a small batch of several requests too (slower than three
                                   launches on the shapes measured, see above; kept for callers to whom the number of
                                   launches matters more than the time) */
};

/* bits of req_status[b].  Every problem a request shows is reported: a bad length together with a bad parameter gives
 * both bits (BAD_LEN | BAD_PARAM); BAD_TOKEN and NONFINITE are reported only for rows up to the first rejection. */
enum {
  SPECSTEER_REQ_BAD_TOKEN = 1,      /* a reached draft token outside [0,V): that position is a rejection, alpha 0 */
  SPECSTEER_REQ_BAD_LEN = 2,        /* draft_len outside [0,K]: treated as 0 */
  SPECSTEER_REQ_NONFINITE = 4,      /* a reached row has a NaN/inf normaliser: accept_len = that row, no token */
  SPECSTEER_REQ_RESIDUAL_EMPTY = 8, /* RESIDUAL had zero mass: STEER weights were used */
  SPECSTEER_REQ_BAD_PARAM = 16      /* lambda <= 0, temperature <= 0 or a non-finite parameter: nothing accepted */
};

typedef struct {
  int32_t B, K, V;        /* requests, maximum drafts per request, vocabulary size */
  int64_t ld_row, ld_req; /* strides in ELEMENTS: ld_row >= V, ld_req >= (K+1)*ld_row */
  int32_t dtype;          /* specsteer_dtype of the three logit tensors */
  int32_t accept_mode;    /* specsteer_accept_mode */
  int32_t recover_mode;   /* specsteer_recover_mode */
  uint32_t flags;         /* SPECSTEER_FLAG_* */

  /* ---- inputs ---- */
  const void *h_llm, *h_slm_plus, *h_slm_minus; /* [B][K+1][V] logits */
  const int32_t *draft_tokens;                  /* [B][K]   drafted ids y_hat (Eq. 5) */
  const int32_t *draft_len;                     /* [B]      drafts actually made, 0..K; rows > draft_len unread */
  const float *lambda;                          /* [B]      lambda of Eq. 7, > 0 */
  const float *beta;                            /* [B]      beta of Eq. 8 */
  const float *temperature;                     /* [B]      > 0; every logit is divided by it before any softmax */
  const float *u_accept;                        /* [B][K]   uniforms in [0,1) for "Uniform(0,1) <= alpha_t" */
  const float *u_recover;                       /* [B]      uniform in [0,1) for the recovery sample */

  /* ---- outputs (caller-allocated; any may be NULL except accept_len) ----
   * What is requested decides what is read.  Algorithm 1 itself needs the normalisers of h_LLM and h_SLM- on the
   * drafted rows (Eq. 7) and that of h_rec on the one row it recovers from (Eq. 8).
   *   - RATIO + STEER (or ARGMAX) with logp_plus, logp_star and log_z all NULL (and 16-byte aligned rows):
   *     verification reads h_LLM and h_SLM- alone, over the drafted rows; specsteer_recover_sample then streams row
   *     accept_len of the requests that take a token, all three tensors: the two-phase round, about a fifth fewer
   *     bytes (taken automatically for large batches, see SPECSTEER_FLAG_TWO_PHASE).  A non-finite entry of
   *     h_SLM+ on a drafted row is then not seen (REQ_NONFINITE is raised for it only on the recovery row).
   *   - logp_star wanted, logp_plus and log_z NULL: one pass over all three tensors and all rows, but the
   *     normaliser of h_SLM+ is not formed (a quarter fewer exponentials; it matters for 16-bit logits).
   *   - otherwise (logp_plus or log_z wanted, EXACT_Z, RESIDUAL): all four normalisers on every row.
   * Decisions and tokens are the same in all three; floating-point outputs may differ in the last bits. */
  int32_t *accept_len;   /* [B]      drafts accepted before the first rejection */
  uint8_t *accept_flags; /* [B][K]   1 where u <= alpha (every drafted position, also after the first rejection) */
  float *alpha;          /* [B][K]   acceptance probability; 0 beyond draft_len */
  float *logp_llm;       /* [B][K]   log P_LLM(y_hat)      NaN beyond draft_len or for a bad token */
  float *logp_minus;     /* [B][K]   log P_SLM-(y_hat) */
  float *logp_plus;      /* [B][K]   log P_SLM+(y_hat) */
  float *logp_star;      /* [B][K]   log Softmax(h_rec)(y_hat) = log P*(y_hat) at beta = 1 (Eq. 4) */
  float *log_z;          /* [B][K+1] log sum_v P_LLM (P+/P-)^beta = log Z_t at beta = 1 (Eq. 2); NaN for unread rows */
  int32_t *rec_token;    /* [B]      sampled token, -1 if none was sampled */
  float *rec_logprob;    /* [B]      log of its probability under the sampled distribution */
  int32_t *out_tokens;   /* [B][K+1] accepted drafts followed by rec_token, padded with -1 */
  int32_t *n_out;        /* [B]      number of valid entries in out_tokens */
  int32_t *req_status;   /* [B]      SPECSTEER_REQ_* bits */
} specsteer_round_desc;

/* Create a context on CUDA device `device` able to run rounds up to the given maxima.  Allocates the
 * workspace (row normalisers and per-chunk partial sums; about
 * max_B*(max_K+1)*(16 + 32*ceil(max_V/512)) bytes, plus 4 KB per request for specsteer_cloud_topk) once; no later call of the device-pointer entry points allocates.
 * Errors: INVALID_ARG (NULL out, non-positive maxima), CUDA, WORKSPACE. */
specsteer_status specsteer_ctx_create(specsteer_ctx **out, int device, int32_t max_B, int32_t max_K, int32_t max_V);

/* Free the context and its workspace.  The caller must have synchronised any stream still using it. */
specsteer_status specsteer_ctx_destroy(specsteer_ctx *ctx);

/* Verification (Algorithm 1 Phase 2; Eq. 6/7): one pass over the three logit streams of every used row
 * computes the four log-normalisers, then per position the log-probabilities, alpha and the accept flag,
 * and per request accept_len = the first t with u_accept > alpha (or draft_len).  Writes every output of
 * the descriptor except rec_token, rec_logprob, out_tokens, n_out (req_status is written here and may gain
 * bits in specsteer_recover_sample); unless SPECSTEER_FLAG_SEPARATE_LAUNCHES is set it may write those four as well
 * (see the flag).  Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
specsteer_status specsteer_verify_round(specsteer_ctx *ctx, const specsteer_round_desc *desc, void *cuda_stream);

/* Recovery (Algorithm 1 Phase 3; Eq. 8): for each request whose accept_len < draft_len (or always, with
 * FLAG_BONUS) samples one token from row accept_len by inverse CDF in vocabulary order:
 * the smallest v with sum_{j<=v} w(j) > u_recover * sum_j w(j).  Must follow specsteer_verify_round with
 * the same descriptor on the same stream (ERR_ORDER otherwise).  Writes rec_token, rec_logprob,
 * out_tokens, n_out.  With SPECSTEER_RECOVER_ARGMAX (greedy decoding) the token is the maximiser of h_rec on that
 * row instead and u_recover is not used.  Errors: INVALID_ARG, ORDER, CUDA. */
specsteer_status specsteer_recover_sample(specsteer_ctx *ctx, const specsteer_round_desc *desc, void *cuda_stream);

/* Top-k split recovery (the paper's deployment appendix, "Minimal Downlink (Steering Recovery)", case "If
 * rejected"), an alternative to specsteer_recover_sample for a deployment where h_SLM+ lives on another machine.
 * Both calls must follow specsteer_verify_round with the same descriptor on the same stream (ERR_ORDER otherwise)
 * and act on row accept_len of every request that samples (accept_len < draft_len, or always with FLAG_BONUS).
 *
 * Cloud half: h_cloud(v) = h_LLM(v) - beta*h_SLM-(v), formed in float32 by one fused multiply-add, truncated to the
 * k entries with the highest values.  topk_idx[B][k] / topk_val[B][k] (device) receive them ordered by value,
 * highest first, equal values by lower token id; NaN entries are never kept; unused slots and requests that do
 * not sample get id -1 and value -inf.  Reads h_llm, h_slm_minus, beta, draft_len, accept_len; h_slm_plus is not
 * touched.  1 <= k <= SPECSTEER_TOPK_MAX.  Errors: INVALID_ARG, UNSUPPORTED, ORDER, CUDA. */
#define SPECSTEER_TOPK_MAX 32
specsteer_status specsteer_cloud_topk(specsteer_ctx *ctx, const specsteer_round_desc *desc, int32_t k,
                                      int32_t *topk_idx, float *topk_val, void *cuda_stream);

/* Edge half: on the kept entries h_rec = topk_val + beta*h_SLM+[topk_idx] (Eq. 8), divided by the temperature;
 * their softmax is taken in float64 and one token is drawn by inverse CDF in list order with u_recover (the
 * smallest j whose cumulative weight exceeds u * total, else the last j with positive weight).  Writes rec_token,
 * rec_logprob (log of its probability among the k), out_tokens and n_out exactly like specsteer_recover_sample.
 * Reads h_slm_plus, beta, temperature, u_recover, draft_tokens, draft_len, accept_len and the two lists; h_llm and
 * h_slm_minus are not touched.  Errors: as above. */
specsteer_status specsteer_edge_resample(specsteer_ctx *ctx, const specsteer_round_desc *desc, int32_t k,
                                         const int32_t *topk_idx, const float *topk_val, void *cuda_stream);

/* Vocabulary-sharded rounds: the logits arrive split along V over n_shards GPUs (a tensor-parallel LM head), GPU g
 * holding [B][K+1][V_g] for the global token ids [vocab_offset_g, vocab_offset_g + V_g).  The paper runs its
 * Generalist and the public Specialist copy side by side on the cloud (deployment appendix) and says nothing about
 * sharding them; this is the same round (Algorithm 1 phases 2 and 3, Eq. 7 / Eq. 6, Eq. 8) with one exchange step:
 *   1. specsteer_shard_verify_local on every GPU: streams the local shard and writes, for every row, a 64-byte
 *      partial (largest exponent and float64 sum of the four normalisers over the shard, and the drafted token's
 *      three logits if the token lies in the shard) into row_partials [B][K+1][64 bytes] (device).
 *   2. the caller all-gathers the partials into gathered [n_shards][B][K+1][64 bytes] on every GPU (NCCL).
 *   3. specsteer_shard_verify_combine on every GPU: identical arithmetic everywhere; writes every output
 *      specsteer_verify_round writes.  desc is the LOCAL descriptor (V = V_g); draft_tokens hold GLOBAL ids.
 *   4. specsteer_shard_recover_local on every GPU: all GPUs place the CDF target among the shards from the
 *      gathered partials; the owner samples within its shard and writes the global token id, rec_logprob,
 *      out_tokens, n_out; the others write -1, -inf, the accepted prefix with -1 in the new slot, and accept_len,
 *      so that an element-wise MAX all-reduce of those four arrays gives every GPU the result.
 * STEER recovery only; B <= 1024; n_shards <= SPECSTEER_MAX_SHARDS.
 * Errors: INVALID_ARG, UNSUPPORTED, ORDER (step out of sequence), CUDA. */
#define SPECSTEER_MAX_SHARDS 32
#define SPECSTEER_SHARD_PARTIAL_BYTES 64
specsteer_status specsteer_shard_verify_local(specsteer_ctx *ctx, const specsteer_round_desc *desc, int32_t vocab_offset,
                                              void *row_partials, void *cuda_stream);
specsteer_status specsteer_shard_verify_combine(specsteer_ctx *ctx, const specsteer_round_desc *desc, const void *gathered,
                                                int32_t n_shards, int32_t shard_rank, int32_t vocab_offset,
                                                int32_t vocab_total, void *cuda_stream);
specsteer_status specsteer_shard_recover_local(specsteer_ctx *ctx, const specsteer_round_desc *desc, const void *gathered,
                                               int32_t n_shards, int32_t shard_rank, int32_t vocab_offset,
                                               int32_t vocab_total, void *cuda_stream);

/* The round with the three LM heads fused in front of it.  Algorithm 1's verification and recovery steps read the
 * logits of three forward passes, h = x W^T: the Generalist (h_LLM), and the Specialist with and without the private
 * context (h_SLM+, h_SLM-; the same model, hence usually the same head).  This entry point takes the hidden states and
 * the head weights instead of the logits and never stores a logit: the products are formed tile by tile on the tensor
 * cores (tcgen05, float32 accumulation in tensor memory), each tile is reduced at once to the per-chunk partial sums
 * the round needs, and the recovery step (Eq. 8) recomputes the 128 logits of the one chunk it samples from.
 *   - round: as for specsteer_verify_round + specsteer_recover_sample, except that h_llm, h_slm_plus, h_slm_minus,
 *     ld_row, ld_req and dtype are ignored.  Every output may be requested; every row of every request is computed.
 *   - x_*: DEVICE, bf16, [B][K+1][d] dense; w_*: DEVICE, bf16, [V][d] dense (row v = the head's weights of token v);
 *     all 16-byte aligned, d_llm and d_slm multiples of 8.  w_slm_plus and w_slm_minus may be the same pointer.
 *   - RATIO or EXACT_Z acceptance, STEER or ARGMAX recovery (RESIDUAL: UNSUPPORTED).
 *   - The first call allocates a second workspace for the context's maxima
 *     (max_B*(max_K+1)*(16 + 40*ceil(max_V/128)) bytes); later calls allocate nothing.
 *   - Accuracy: the logits carry the rounding of a float32 accumulation over d bf16 products, so decisions may
 *     differ from exact arithmetic where their margin is below about 1e-4.
 *   - With only Algorithm 1's outputs requested (RATIO, STEER or ARGMAX, logp_plus / logp_star / log_z NULL, and not
 *     SPECSTEER_FLAG_SEPARATE_LAUNCHES) the round is two-phase: verification forms h_LLM and h_SLM- alone (Eq. 7) in
 *     tiles twice as wide, then all three products of row accept_len of every request that takes a token (Eq. 8) from
 *     compacted hidden states.  Seven launches, about a fifth faster; a further workspace of
 *     max_B*(d_llm + 2*d_slm)*2 bytes is allocated by the first such call.  Same decisions and tokens as the one-pass
 *     round up to the accuracy stated above.
 * Three launches otherwise; stream-ordered; specsteer_ctx_time_streaming brackets the tensor-core kernel(s).
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, TIMEOUT, CUDA. */
typedef struct {
  specsteer_round_desc round;
  const void *x_llm, *w_llm;             /* [B][K+1][d_llm], [V][d_llm] */
  const void *x_slm_plus, *w_slm_plus;   /* [B][K+1][d_slm], [V][d_slm] */
  const void *x_slm_minus, *w_slm_minus; /* [B][K+1][d_slm], [V][d_slm] */
  int32_t d_llm, d_slm;
} specsteer_lmhead_desc;
specsteer_status specsteer_lmhead_round(specsteer_ctx *ctx, const specsteer_lmhead_desc *desc, void *cuda_stream);

/* The fused round with the heads split along the vocabulary over n_shards GPUs (a tensor-parallel LM head): GPU g
 * holds rows [vocab_offset_g, vocab_offset_g + V_g) of every head (desc->round.V = V_g, w_* point at those rows) and
 * all the hidden states.  Same four steps and the same two collectives as the vocabulary-sharded round above:
 *   1. specsteer_lmhead_shard_local: the tensor-core pass over the local rows of the heads, then one 64-byte partial
 *      per row into row_partials [B][K+1][64 bytes] (the drafted token's logits if the token lies in the shard);
 *   2. the caller all-gathers the partials into gathered [n_shards][B][K+1][64 bytes];
 *   3. specsteer_lmhead_shard_combine: every verification output, identical on every GPU;
 *   4. specsteer_lmhead_shard_recover: the shard that holds the CDF target recomputes its chunk and writes the global
 *      token id; the others write -1, -inf, the accepted prefix and accept_len, for an element-wise MAX all-reduce
 *      of rec_token, rec_logprob, out_tokens and n_out.
 * No logit and no head weight crosses the link.  draft_tokens hold GLOBAL ids.  B <= 1024.
 * Errors: as specsteer_lmhead_round and the sharded round. */
specsteer_status specsteer_lmhead_shard_local(specsteer_ctx *ctx, const specsteer_lmhead_desc *desc, int32_t vocab_offset,
                                              void *row_partials, void *cuda_stream);
specsteer_status specsteer_lmhead_shard_combine(specsteer_ctx *ctx, const specsteer_lmhead_desc *desc, const void *gathered,
                                                int32_t n_shards, int32_t shard_rank, int32_t vocab_offset,
                                                int32_t vocab_total, void *cuda_stream);
specsteer_status specsteer_lmhead_shard_recover(specsteer_ctx *ctx, const specsteer_lmhead_desc *desc, const void *gathered,
                                                int32_t n_shards, int32_t shard_rank, int32_t vocab_offset,
                                                int32_t vocab_total, void *cuda_stream);

/* Greedy recovery (SPECSTEER_RECOVER_ARGMAX) in the two vocabulary-sharded rounds.  Steps 1-3 are as above; in place
 * of step 4:
 *   4a. specsteer_shard_greedy_local (logit shards; after specsteer_shard_verify_combine) or
 *       specsteer_lmhead_shard_greedy_local (head shards; after specsteer_lmhead_shard_combine): best_keys[B]
 *       (device, int64) receives this shard's best entry of row accept_len as a key that orders by h_rec first and
 *       by the lower GLOBAL token id among equal values ((order-preserving float bits << 31) | (0x7fffffff - id));
 *       -1 for a request that takes no token;
 *   4b. the caller takes the element-wise MAX of best_keys over the shards (one all-reduce of B int64);
 *   4c. specsteer_shard_greedy_finish on every GPU: rec_token, rec_logprob, out_tokens and n_out from the reduced
 *       keys, identical everywhere (desc: the round descriptor, or &lmhead_desc->round).
 * Errors: INVALID_ARG, UNSUPPORTED (another recovery mode), ORDER, TIMEOUT, CUDA. */
specsteer_status specsteer_shard_greedy_local(specsteer_ctx *ctx, const specsteer_round_desc *desc, int32_t vocab_offset,
                                              int64_t *best_keys, void *cuda_stream);
specsteer_status specsteer_lmhead_shard_greedy_local(specsteer_ctx *ctx, const specsteer_lmhead_desc *desc,
                                                     int64_t *best_keys, void *cuda_stream);
specsteer_status specsteer_shard_greedy_finish(specsteer_ctx *ctx, const specsteer_round_desc *desc,
                                               const int64_t *best_keys, void *cuda_stream);

/* Whole round from HOST memory: every pointer in `desc` is a HOST pointer (pinned memory makes the copies
 * asynchronous).  Copies inputs to device staging buffers owned by the context (allocated on the first
 * call, sized for the context's maxima: 3*max_B*(max_K+1)*max_V elements of 4 bytes), runs verification and
 * recovery, copies every non-NULL output back, and returns after the stream has drained.  Requests are
 * processed in slabs so that the copy of one slab overlaps the kernels of the previous one.
 * The host-to-device link bounds this call, so when only Algorithm 1's outputs are wanted (the conditions of the
 * two-phase round: RATIO, STEER or ARGMAX, logp_plus / logp_star / log_z NULL, 16-byte aligned rows) it copies only
 * what that round reads: rows [0, K) of h_LLM and h_SLM-, then - once the accepted lengths are back on the host -
 * row accept_len of h_SLM+ for every request that takes a token (and of the other two tensors when that row is the
 * bonus row).  Nothing else of the three host tensors is touched.
 * Errors: as the two calls above, plus WORKSPACE. */
specsteer_status specsteer_round_host(specsteer_ctx *ctx, const specsteer_round_desc *desc, void *cuda_stream);

/* Verification without a context and without any allocation.  (The paper has no counterpart: this is a
 * packaging of specsteer_verify_round for hosts that cannot allocate device memory.)
 *
 * Who needs it: code that runs where a device allocation is forbidden or harmful - a plug-in inside a
 * serving process whose memory manager owns the whole device and hands out no more after start-up, a
 * latency-critical loop that cannot afford the device-wide synchronisation cudaMalloc may imply, or a
 * process so close to its memory budget that a late allocation could fail.  specsteer_ctx_create allocates
 * a workspace; this call instead keeps its workspace in a fixed 8 MiB array that is part of the library's
 * device image, so every GPU that loads the library holds those 8 MiB until the process exits.
 *
 * It runs the same two kernels as specsteer_verify_round (same descriptor, same host-side checks, same outputs,
 * device pointers, the current CUDA device; every recover_mode is accepted, since verification does not depend on
 * it, and u_recover may be NULL) and calls no cudaMalloc, cudaFree or other allocating routine.
 * specsteer_recover_sample needs a context and cannot follow it.
 *   - Limits: B <= 1024, B*(K+1) <= 16384, and B*(K+1)*ceil(V/C) <= 229376 with C = 512 for float32 and
 *     1024 for bf16 logits.  Larger shapes return SPECSTEER_ERR_STATIC_LIMIT and launch nothing.
 *   - The first call on each device resolves the array's device address (cudaGetSymbolAddress) and reads
 *     the device's attributes; make that first call outside any stream capture.
 *   - All calls on a device share the one array.  Nothing in it has to be cleared between calls (every word
 *     a call reads it has written first), but two calls whose kernels overlap on the GPU - different
 *     streams, or different host threads - race on it: serialise them.
 *   - A bounded device-side wait that gives up is not reported by this entry point.
 * Errors: INVALID_ARG, STATIC_LIMIT, UNSUPPORTED (device index >= 64), CUDA. */
specsteer_status specsteer_verify_round_static(const specsteer_round_desc *desc, void *cuda_stream);

/* Synchronise the context's device and report whether any kernel of this context gave up a bounded wait:
 * SPECSTEER_OK or SPECSTEER_ERR_TIMEOUT (sticky until the context is destroyed). */
specsteer_status specsteer_ctx_device_error(specsteer_ctx *ctx);

/* Test hook for the library's only failure detector.  Every wait inside the streaming kernel (a consumer warp for a
 * tile's bytes, a producer thread for a free stage) is bounded: after `sm_clocks` SM clocks it gives up, the CTA records
 * the error, waits for the copies it has in flight and returns, and specsteer_ctx_device_error reports
 * SPECSTEER_ERR_TIMEOUT.  The default (0 restores it) is 2^33 clocks, a few seconds, which no healthy run reaches; a
 * limit of a few hundred clocks makes the first wait for data run out, which is how the give-up path is exercised
 * without hanging or faulting anything.  Outputs of a round that gave up are undefined (but every access stays in
 * bounds).  Applies to specsteer_verify_round / _recover_sample / _round_host / the sharded logit rounds of this
 * context.  Errors: INVALID_ARG (NULL ctx, negative limit). */
specsteer_status specsteer_ctx_set_wait_limit(specsteer_ctx *ctx, int64_t sm_clocks);

/* Profiling hook: from now on specsteer_verify_round records the two caller-owned CUDA events (cudaEvent_t
 * passed as void*, created with timing enabled) on its stream just before and just after the streaming
 * kernel, the launch that reads all the logits, so that a benchmark can time that kernel alone; the per-request
 * epilogue kernel follows the second event.  With more than 1024 requests the round runs in several slabs and
 * the events bracket everything from the first slab's streaming kernel to the last one's.  Pass two NULLs to
 * switch the hook off.  Errors: INVALID_ARG (NULL ctx, or only one event given). */
specsteer_status specsteer_ctx_time_streaming(specsteer_ctx *ctx, void *ev_begin, void *ev_end);

/* Measurement aid (the paper has no counterpart): launches n_ctas CTAs of 1024 threads on the current device, each
 * thread evaluating 8 * iters ex2.approx (the special-function instruction every normaliser of the streaming kernel
 * costs once per vocabulary entry), so that a benchmark can time it with its own events and state a measured
 * special-function rate instead of an assumed one.  sink: DEVICE, n_ctas * 1024 floats, overwritten.
 * Total evaluations: n_ctas * 1024 * 8 * iters.  Errors: INVALID_ARG, CUDA. */
specsteer_status specsteer_probe_ex2(int32_t n_ctas, int32_t iters, float *sink, void *cuda_stream);

/* Bytes of device workspace owned by the context. */
size_t specsteer_ctx_workspace_bytes(const specsteer_ctx *ctx);

/* Number of kernels the context has launched since creation (for launch accounting in benchmarks). */
uint64_t specsteer_ctx_launch_count(const specsteer_ctx *ctx);

const char *specsteer_status_string(specsteer_status s);
uint32_t specsteer_version(void); /* major<<16 | minor<<8 | patch */

#ifdef __cplusplus
}
#endif
#endif /* SPECSTEER_H */
