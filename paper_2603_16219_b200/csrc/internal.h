// Host/device structures shared by the translation units of the library (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace specsteer {

// One vocabulary chunk = what one warp of the streaming pass reduces = one partial record (2 KB per stream).
// The streaming pass copies tiles of two chunks (4 KB per stream, 12 KB per stage).
constexpr int kChunkF32 = 512;
constexpr int kChunkBF16 = 1024;
constexpr int kChunkMin = 512;
// When only h_LLM and h_SLM- are streamed a stage holds two slots instead of three, so the chunks grow by half
// (3 KB per stream): fewer per-chunk set-ups and reductions per byte (measured on 3.15 GB of bf16: 570 -> 512 us).
constexpr int kChunkRatioF32 = 768;
constexpr int kChunkRatioBF16 = 1536;
// A bounded device-side wait gives up after this many SM clocks (a few seconds) unless the context says otherwise.
constexpr long long kDefaultWaitCycles = 1ll << 33;
constexpr int kMaxSlabB = 1024;  // requests handled by one launch (per-request tables live in shared memory)

// What one vocabulary shard knows about one row (64 bytes; the unit of the all-gather in the sharded path):
// for the four normalisers the largest exponent and the float64 sum relative to it (value s * 2^m), and the
// three logits of the drafted token when that token lies in the shard.
struct ShardPartial {
  float m[4];
  double s[4];
  float tok_logit[3];  // h_LLM, h_SLM+, h_SLM- at the drafted token
  int has_token;
};
static_assert(sizeof(ShardPartial) == 64, "the sharded path exchanges 64 bytes per row and shard");

enum { SUM_L = 1, SUM_P = 2, SUM_M = 4, SUM_R = 8, SUM_ALL = 15 };  // bit q = normaliser Q_q
enum {
  ROWS_ALL = 0,       // rows 0 .. draft_len (the last one only with FLAG_BONUS)
  ROWS_DRAFTED = 1,   // rows 0 .. draft_len - 1: verification alone
  ROWS_RECOVERY = 2   // row accept_len of the requests that sample (after the epilogue has run)
};

struct RoundParams {
  int B, K, V;
  long long ld_row, ld_req;  // elements
  int accept_mode, recover_mode;
  unsigned flags;
  int sums;      // SUM_* bits: which of the four normalisers the streaming pass forms (Algorithm 1 needs L, M and,
                 // on the recovery row, R; the one of h_SLM+ only serves logp_plus, log_z, EXACT_Z and RESIDUAL)
  int row_mode;  // ROWS_*: which rows of a request the streaming pass reads
  int tile;      // vocabulary entries per chunk (kChunkF32 or kChunkBF16)
  int n_chunks;  // ceil(V / tile)
  const void *h_llm, *h_plus, *h_minus;
  const int* draft_tokens;
  const int* draft_len;
  const float *lambda, *beta, *temperature, *u_accept, *u_recover;
  int* accept_len;
  uint8_t* accept_flags;
  float *alpha, *logp_llm, *logp_minus, *logp_plus, *logp_star, *log_z;
  int* rec_token;
  float* rec_logprob;
  int* out_tokens;
  int* n_out;
  int* req_status;
  // workspace
  float* part;        // [B*(K+1)][n_chunks][8]  partial records {mL,sL,mP,sP,mM,sM,mR,sR}
  float* lse2;        // [B*(K+1)][4]            base-2 log-normalisers {L,P,M,R}
  int* status_ws;     // [B]                     request status when the caller passes no req_status
  int* dev_error;     // [1]                     set when a bounded wait gave up
  int* req_done;      // [B]                     chunks retired per request (one-launch round); zero between launches
  long long wait_cycles;  // give-up limit of the streaming kernel's pipeline waits, in SM clocks
  float* row_ref;     // [B*(K+1)][4]            reference exponents per row {L,P,M,R} (row_ref_kernel), or null: the
                      //                         chunks take their references from their own first batch
  // vocabulary-sharded path (n_shards == 0: the tensors hold the whole vocabulary)
  const ShardPartial* shard_parts;  // [n_shards][B][K+1] gathered partials
  int n_shards, shard_rank;
  int vocab_offset, vocab_total;    // this shard covers global ids [vocab_offset, vocab_offset + V)
  // fused LM-head path: the logit tensors do not exist; the drafted tokens' logits were left here instead
  const float* tok_logits;          // [B*(K+1)][4] {h_LLM, h_SLM+, h_SLM-, unused} of the row's drafted token, or null
  // greedy recovery in a sharded round: the argmax kernels leave this shard's best key per request here instead of
  // writing the outputs ((order-preserving value bits << 31) | (0x7fffffff - global id); -1: no token), or null
  long long* greedy_keys;
};

// The LM heads in front of the round: h = x W^T, all operands bf16, row-major, dense.
constexpr int kLmheadChunk = 128;   // vocabulary entries per partial record on that path (one tensor-core tile)
struct LmheadOperands {
  const uint16_t *x_llm, *w_llm;      // [B*(K+1)][d_llm], [V][d_llm]
  const uint16_t *x_plus, *w_plus;    // [B*(K+1)][d_slm], [V][d_slm]
  const uint16_t *x_minus, *w_minus;  // [B*(K+1)][d_slm], [V][d_slm]
  int d_llm, d_slm;
};

}  // namespace specsteer
#include "specsteer.h"
namespace specsteer {

// Host-side checks of a round descriptor that every entry point shares: sizes, strides, enums, flags and the
// pointers verification needs.  need_u_recover: the caller will (or may) run a recovery step on this descriptor.
specsteer_status check_round_desc(const specsteer_round_desc* d, bool need_u_recover);
// Which normalisers the streaming pass forms for a descriptor (SUM_* bits), from the outputs and modes it asks for.
int sums_wanted(const specsteer_round_desc* d);
// Every row of the three logit tensors starts on a 16-byte boundary (the bulk-copy path).
bool rows_aligned(const specsteer_round_desc* d);

struct LaunchInfo {
  int device;
  int sm_count;
  int max_smem_optin;
};

// ev_begin / ev_end, when not null, are recorded on `s` just before and just after the streaming kernel.
// with_recover: the launch that runs the epilogue also draws the STEER recovery sample (see launch_epilogue).
cudaError_t launch_verify(const RoundParams& p, int dtype, bool aligned, const LaunchInfo& li, cudaStream_t s,
                          int* n_launches, cudaEvent_t ev_begin = nullptr, cudaEvent_t ev_end = nullptr,
                          bool with_recover = false);
// The tensor-core pass: partial records of every row at kLmheadChunk entries per chunk, and tok_logits.
// argmax_keys: [B*(K+1)][n_chunks] 64-bit words that receive, per tile, the key of the largest h_rec (greedy recovery),
// or null when nobody needs them.
cudaError_t launch_lmhead(const RoundParams& p, const LmheadOperands& op, float* tok_logits, void* argmax_keys,
                          const LaunchInfo& li, cudaStream_t s);
// Two-phase round on the LM-head path.  Verification alone: h_LLM and h_SLM- of every row (tiles of 128 x 256, records
// at 256 entries per chunk, slots of h_SLM+ and h_rec empty) and the drafted tokens' two logits.
constexpr int kLmheadRatioChunk = 256;
cudaError_t launch_lmhead_ratio(const RoundParams& p, const LmheadOperands& op, float* tok_logits, const LaunchInfo& li,
                                cudaStream_t s);
// the hidden states of row accept_len of every request that takes a token, compacted to [B][d] (zero rows otherwise)
cudaError_t launch_lmhead_gather_rows(const RoundParams& p, const LmheadOperands& op, uint16_t* xl, uint16_t* xp, uint16_t* xm,
                                      cudaStream_t s);
// rec_token, rec_logprob, out_tokens, n_out and the status words from the compact pass's token and status
cudaError_t launch_lmhead_finish(const RoundParams& p, const int* c_status, const int* c_token, cudaStream_t s);
// Sharded greedy rounds, last step: the outputs from the keys every shard agreed on (MAX over shards).
cudaError_t launch_greedy_finish(const RoundParams& p, const long long* keys, cudaStream_t s);
// Greedy recovery from those keys.
cudaError_t launch_lmhead_argmax(const RoundParams& p, const void* argmax_keys, cudaStream_t s);
// Recovery (Eq. 8) from those records; the logits of the one chunk that holds the CDF target are recomputed.
cudaError_t launch_lmhead_recover(const RoundParams& p, const LmheadOperands& op, cudaStream_t s);
constexpr int kTopkMaxSplit = 16;  // CTAs that may share one row in specsteer_cloud_topk
// lists_ws: [B][kTopkMaxSplit][32] 64-bit keys; count_ws: [B] counters, zero between launches
cudaError_t launch_cloud_topk(const RoundParams& p, int dtype, int k, int* topk_idx, float* topk_val,
                              void* lists_ws, int* count_ws, int sm_count, cudaStream_t s);
cudaError_t launch_edge_resample(const RoundParams& p, int dtype, int k, const int* topk_idx, const float* topk_val,
                                 cudaStream_t s);
// The whole round of a small batch in one launch: streaming, per-request epilogue and STEER recovery sample.
// p: ROWS_ALL, sums with SUM_R, 16-byte aligned rows, p.req_done set.  fused_round_fits: the vocabulary is small enough
// for the chunk weights of a row to sit in the ring.
bool fused_round_fits(const RoundParams& p, int dtype);
cudaError_t launch_verify_fused(const RoundParams& p, int dtype, const LaunchInfo& li, cudaStream_t s);
// the reference exponents of every row (p.row_ref), for the streaming kernel launched next on the same stream
cudaError_t launch_row_ref(const RoundParams& p, int dtype, cudaStream_t s);
// the streaming kernel alone (partial records into the workspace), no epilogue
cudaError_t launch_verify_stream(const RoundParams& p, int dtype, bool aligned, const LaunchInfo& li, cudaStream_t s);
// per-row ShardPartial of this shard from its partial records: out[B][K+1]
cudaError_t launch_shard_rows(const RoundParams& p, int dtype, ShardPartial* out, cudaStream_t s);
// the per-request epilogue alone (reads p.shard_parts when p.n_shards > 0); with_recover: the same CTAs go on to the
// STEER recovery sample of their request (p as for launch_recover without own_lse, records at the logit type's chunk
// size), which saves the second launch of a round whose verification read every row
cudaError_t launch_epilogue(const RoundParams& p, int dtype, cudaStream_t s, bool with_recover = false);
// own_lse: row accept_len has records but no normalisers yet (two-phase round); the STEER kernel forms them first.
cudaError_t launch_recover(const RoundParams& p, int dtype, const LaunchInfo& li, cudaStream_t s, int* n_launches,
                           bool own_lse = false);
// Greedy recovery (ARGMAX).  best_ws: [B][kTopkMaxSplit * 32] 64-bit words (the top-k selection's lists), count_ws: [B]
// counters, zero between launches.  `aligned`: every row of the three tensors starts on a 16-byte boundary.
// `own_lse`: the row has no normaliser in lse2 (two-phase round): the pass forms it, and the row's finiteness check, itself.
cudaError_t launch_recover_argmax(const RoundParams& p, int dtype, bool aligned, bool own_lse, void* best_ws, int* count_ws,
                                  int sm_count, cudaStream_t s);

}  // namespace specsteer
