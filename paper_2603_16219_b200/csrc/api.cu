// C ABI: context, argument checks, launches, and the host-buffer round.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "internal.h"
#include "specsteer.h"

using namespace specsteer;

struct specsteer_ctx {
  int device;
  int max_B, max_K, max_V;
  LaunchInfo li;
  // workspace (one allocation)
  void* ws;
  size_t ws_bytes;
  float* part;
  float* lse2;
  int* status_ws;
  int* dev_error;
  float* row_ref;     // [max_B*(max_K+1)][4] reference exponents per row for the streaming kernel of large rounds
  int* req_done;      // [max_B] chunks retired per request in the one-launch round; zero between launches
  bool v_fused;       // the last verify_round ran the whole round (recover_sample then has nothing to launch)
  void* topk_lists;   // [max_B][kTopkMaxSplit][32] keys of the split top-k selection
  int* topk_count;    // [max_B], zero between launches
  // last verified round, for the order check
  bool verified;
  int v_B, v_K, v_V, v_dtype;
  const void* v_h_llm;
  uint64_t launches;
  long long wait_cycles;   // give-up limit of the streaming kernel's waits (specsteer_ctx_set_wait_limit)
  bool poisoned;
  bool shard_streamed;   // specsteer_shard_verify_local ran for the shape in v_*
  bool v_two_phase;      // the last verify_round left the recovery rows unread (see two_phase())
  // host-round staging
  void* stage;
  size_t stage_bytes;
  cudaStream_t copy_stream;
  cudaEvent_t ev_copied[2], ev_done[2];
  bool host_ready;
  // optional timing hooks around the streaming kernel (caller-owned events)
  cudaEvent_t ev_stream_begin, ev_stream_end;
  // fused LM-head path: records at 128 entries per chunk and the drafted tokens' logits (allocated on first use)
  void* lm_ws;
  float* lm_part;
  float* lm_tok;
  void* lm_keys;      // [rows][chunks of 128] per-tile keys of the largest h_rec, for greedy recovery
  // two-phase round on that path: the recovery rows' hidden states, compacted, and three small per-request arrays
  void* lm_x2;
  size_t lm_x2_bytes;
};

static_assert(sizeof(specsteer_round_desc) == 232, "the Python mirror of the descriptor assumes this layout");
static_assert(sizeof(specsteer_lmhead_desc) == 288, "the Python mirror of the LM-head descriptor assumes this layout");

namespace specsteer {

specsteer_status check_round_desc(const specsteer_round_desc* d, bool need_u_recover) {
  if (!d) return SPECSTEER_ERR_INVALID_ARG;
  if (d->B < 0 || d->K < 0 || d->V <= 0) return SPECSTEER_ERR_INVALID_ARG;
  if (d->ld_row < d->V || d->ld_req < (int64_t)(d->K + 1) * d->ld_row) return SPECSTEER_ERR_INVALID_ARG;
  if (d->dtype != SPECSTEER_F32 && d->dtype != SPECSTEER_BF16) return SPECSTEER_ERR_INVALID_ARG;
  if (d->accept_mode != SPECSTEER_ACCEPT_RATIO && d->accept_mode != SPECSTEER_ACCEPT_EXACT_Z)
    return SPECSTEER_ERR_INVALID_ARG;
  if (d->recover_mode != SPECSTEER_RECOVER_STEER && d->recover_mode != SPECSTEER_RECOVER_RESIDUAL &&
      d->recover_mode != SPECSTEER_RECOVER_ARGMAX)
    return SPECSTEER_ERR_INVALID_ARG;
  if (d->flags & ~(uint32_t)(SPECSTEER_FLAG_BONUS | SPECSTEER_FLAG_TWO_PHASE | SPECSTEER_FLAG_SEPARATE_LAUNCHES | SPECSTEER_FLAG_ONE_LAUNCH)) return SPECSTEER_ERR_INVALID_ARG;
  if (d->B > 0) {
    if (!d->h_llm || !d->h_slm_plus || !d->h_slm_minus || !d->draft_len || !d->lambda || !d->beta ||
        !d->temperature || !d->accept_len)
      return SPECSTEER_ERR_INVALID_ARG;
    if (need_u_recover && !d->u_recover) return SPECSTEER_ERR_INVALID_ARG;
    if (d->K > 0 && (!d->draft_tokens || !d->u_accept)) return SPECSTEER_ERR_INVALID_ARG;
  }
  return SPECSTEER_OK;
}

int sums_wanted(const specsteer_round_desc* d) {
  return (d->logp_plus || d->log_z || d->accept_mode == SPECSTEER_ACCEPT_EXACT_Z ||
          d->recover_mode == SPECSTEER_RECOVER_RESIDUAL) ? SUM_ALL : (SUM_L | SUM_M | SUM_R);
}

bool rows_aligned(const specsteer_round_desc* d) {
  const size_t es = d->dtype == SPECSTEER_F32 ? 4 : 2;
  auto a16 = [](const void* p) { return ((uintptr_t)p & 15u) == 0; };
  return a16(d->h_llm) && a16(d->h_slm_plus) && a16(d->h_slm_minus) && ((size_t)d->ld_row * es) % 16 == 0 &&
         ((size_t)d->ld_req * es) % 16 == 0;
}

}  // namespace specsteer

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct DeviceGuard {
  int prev;
  bool ok;
  explicit DeviceGuard(int dev) : prev(-1), ok(false) {
    if (cudaGetDevice(&prev) != cudaSuccess) return;
    ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

int tile_of(int dtype) { return dtype == SPECSTEER_F32 ? kChunkF32 : kChunkBF16; }
int n_chunks_of(int V, int tile) { return (V + tile - 1) / tile; }

specsteer_status check_desc(const specsteer_ctx* ctx, const specsteer_round_desc* d) {
  if (!ctx || !d) return SPECSTEER_ERR_INVALID_ARG;
  specsteer_status st = check_round_desc(d, true);
  if (st != SPECSTEER_OK) return st;
  if (d->B > ctx->max_B || d->K > ctx->max_K || d->V > ctx->max_V) return SPECSTEER_ERR_UNSUPPORTED;
  // tiles of one launch are indexed with 31 bits
  const size_t slab_b = d->B < kMaxSlabB ? d->B : kMaxSlabB;
  if (slab_b * (size_t)(d->K + 1) * (size_t)n_chunks_of(d->V, kChunkMin) >= ((size_t)1 << 31)) return SPECSTEER_ERR_UNSUPPORTED;
  return SPECSTEER_OK;
}


// Parameters for the slab of requests [b0, b0 + nb).
RoundParams slab_params(const specsteer_ctx* ctx, const specsteer_round_desc* d, int b0, int nb) {
  RoundParams p;
  memset(&p, 0, sizeof p);
  const size_t es = d->dtype == SPECSTEER_F32 ? 4 : 2;
  const int K = d->K, K1 = K + 1;
  p.B = nb; p.K = K; p.V = d->V;
  p.ld_row = d->ld_row; p.ld_req = d->ld_req;
  p.accept_mode = d->accept_mode; p.recover_mode = d->recover_mode; p.flags = d->flags;
  p.sums = sums_wanted(d);
  p.row_mode = ROWS_ALL;
  p.tile = tile_of(d->dtype);
  p.n_chunks = n_chunks_of(d->V, p.tile);
  auto lg = [&](const void* base) { return (const void*)((const char*)base + (size_t)b0 * d->ld_req * es); };
  p.h_llm = lg(d->h_llm); p.h_plus = lg(d->h_slm_plus); p.h_minus = lg(d->h_slm_minus);
#define OFF(ptr, stride) ((ptr) ? (ptr) + (size_t)b0 * (stride) : nullptr)
  p.draft_tokens = OFF(d->draft_tokens, K);
  p.draft_len = OFF(d->draft_len, 1);
  p.lambda = OFF(d->lambda, 1); p.beta = OFF(d->beta, 1); p.temperature = OFF(d->temperature, 1);
  p.u_accept = OFF(d->u_accept, K); p.u_recover = OFF(d->u_recover, 1);
  p.accept_len = OFF(d->accept_len, 1); p.accept_flags = OFF(d->accept_flags, K);
  p.alpha = OFF(d->alpha, K); p.logp_llm = OFF(d->logp_llm, K); p.logp_minus = OFF(d->logp_minus, K);
  p.logp_plus = OFF(d->logp_plus, K); p.logp_star = OFF(d->logp_star, K); p.log_z = OFF(d->log_z, K1);
  p.rec_token = OFF(d->rec_token, 1); p.rec_logprob = OFF(d->rec_logprob, 1);
  p.out_tokens = OFF(d->out_tokens, K1); p.n_out = OFF(d->n_out, 1); p.req_status = OFF(d->req_status, 1);
  p.part = ctx->part + (size_t)b0 * K1 * p.n_chunks * 8;
  p.lse2 = ctx->lse2 + (size_t)b0 * K1 * 4;
  p.status_ws = ctx->status_ws + b0;
#undef OFF
  p.dev_error = ctx->dev_error;
  p.wait_cycles = ctx->wait_cycles;
  return p;
}

// Verification needs the normalisers of h_LLM and h_SLM- only (Eq. 7); when nobody asks for a quantity of the
// fused target on the drafted rows, the h_SLM+ tensor is left unread there and the recovery call forms the
// normalisers of its one row itself (Eq. 8 on the row of the first rejection).
bool large_round(const specsteer_round_desc* d) {
  const double bytes = 3.0 * d->B * (d->K + 1) * (double)d->V * (d->dtype == SPECSTEER_F32 ? 4 : 2);
  return bytes >= 128.0 * 1024 * 1024;
}

bool two_phase(const specsteer_round_desc* d) {
  const bool eligible = d->accept_mode == SPECSTEER_ACCEPT_RATIO &&
                        (d->recover_mode == SPECSTEER_RECOVER_STEER || d->recover_mode == SPECSTEER_RECOVER_ARGMAX) &&
                        !d->logp_plus && !d->logp_star && !d->log_z && rows_aligned(d);
  if (!eligible) return false;
  if (d->flags & SPECSTEER_FLAG_TWO_PHASE) return true;
  // one more launch and a short second pass (about 10 us) against a fifth of the bytes: worth it from roughly 128 MB of logits upwards
  return large_round(d);
}

// Verification of the requests [b0, b0 + nb).  lean: two tensors over the drafted rows, in the larger chunks of that
// launch shape (the two-phase round).
specsteer_status verify_slab(specsteer_ctx* ctx, const specsteer_round_desc* d, int b0, int nb, bool lean, cudaStream_t s,
                             cudaEvent_t ev_begin, cudaEvent_t ev_end, bool with_recover) {
  RoundParams p = slab_params(ctx, d, b0, nb);
  if (lean) {
    p.sums = SUM_L | SUM_M;
    p.row_mode = ROWS_DRAFTED;
    p.tile = d->dtype == SPECSTEER_F32 ? kChunkRatioF32 : kChunkRatioBF16;
    p.n_chunks = n_chunks_of(d->V, p.tile);
  }
  // Large rounds take the reference exponents of a row from its drafted token (one small launch in front of the
  // streaming kernel), so that heavy-tailed rows at low temperature stay on the streaming kernel's fast path; below
  // about 128 MB of logits the extra launch costs more than it can save.
  if (large_round(d) && rows_aligned(d)) p.row_ref = ctx->row_ref + (size_t)b0 * (d->K + 1) * 4;
  int nl = 0;
  if (launch_verify(p, d->dtype, rows_aligned(d), ctx->li, s, &nl, ev_begin, ev_end, with_recover) != cudaSuccess)
    return SPECSTEER_ERR_CUDA;
  ctx->launches += nl;
  return SPECSTEER_OK;
}

// Recovery of the requests [b0, b0 + nb).  lean: the verification left row accept_len unread.
specsteer_status recover_slab(specsteer_ctx* ctx, const specsteer_round_desc* d, int b0, int nb, bool lean, cudaStream_t s) {
  RoundParams p = slab_params(ctx, d, b0, nb);
  int nl = 0;
  if (lean && d->recover_mode != SPECSTEER_RECOVER_ARGMAX) {   // the recovery rows have no records yet: one more streaming pass over them alone
    p.sums = SUM_ALL;
    p.row_mode = ROWS_RECOVERY;
    if (launch_verify_stream(p, d->dtype, true, ctx->li, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
    ctx->launches += 1;
  }
  if (d->recover_mode == SPECSTEER_RECOVER_ARGMAX) {
    if (launch_recover_argmax(p, d->dtype, rows_aligned(d), lean, (char*)ctx->topk_lists + (size_t)b0 * kTopkMaxSplit * 32 * 8,
                              ctx->topk_count + b0, ctx->li.sm_count, s) != cudaSuccess)
      return SPECSTEER_ERR_CUDA;
    nl = 1;
  } else if (launch_recover(p, d->dtype, ctx->li, s, &nl, lean) != cudaSuccess) {
    return SPECSTEER_ERR_CUDA;
  }
  ctx->launches += nl;
  return SPECSTEER_OK;
}

// A round of a single request (the paper's own regime: one user, one drafted block per round) with STEER recovery
// runs in one launch: the streaming kernel also does the request's epilogue and its recovery sample.  With more
// requests the one launch loses: the requests' last chunks are retired by whichever CTAs run last, a few CTAs end up
// with most of the epilogues and run them one after the other (measured on 16 requests: 113 us against 38 us in three
// launches), so those rounds keep their three launches unless SPECSTEER_FLAG_ONE_LAUNCH asks otherwise.
bool fused_round(const specsteer_ctx* ctx, const specsteer_round_desc* d) {
  if (d->flags & SPECSTEER_FLAG_SEPARATE_LAUNCHES) return false;
  if (large_round(d) || two_phase(d) || !rows_aligned(d) || d->recover_mode != SPECSTEER_RECOVER_STEER) return false;
  if (d->B > kMaxSlabB || !d->u_recover) return false;
  if (d->B != 1 && !(d->flags & SPECSTEER_FLAG_ONE_LAUNCH)) return false;
  RoundParams p = slab_params(ctx, d, 0, d->B);
  return fused_round_fits(p, d->dtype);
}

bool tail_in_one_launch(const specsteer_round_desc* d, bool lean) {
  return !lean && d->recover_mode == SPECSTEER_RECOVER_STEER && d->u_recover != nullptr &&
         !(d->flags & SPECSTEER_FLAG_SEPARATE_LAUNCHES);
}

specsteer_status do_verify(specsteer_ctx* ctx, const specsteer_round_desc* d, cudaStream_t s) {
  ctx->v_fused = false;
  if (fused_round(ctx, d)) {
    RoundParams p = slab_params(ctx, d, 0, d->B);
    p.req_done = ctx->req_done;
    if (ctx->ev_stream_begin && cudaEventRecord(ctx->ev_stream_begin, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
    if (launch_verify_fused(p, d->dtype, ctx->li, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
    if (ctx->ev_stream_end && cudaEventRecord(ctx->ev_stream_end, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
    ctx->launches += 1;
    ctx->v_fused = true;
    return SPECSTEER_OK;
  }
  const bool lean = two_phase(d);
  // A round whose verification reads every row and whose recovery is the STEER sample needs nothing between its
  // epilogue and that sample: one launch does both (same device code, same bits), and the recovery call that follows
  // finds its work done.
  const bool tail = tail_in_one_launch(d, lean);
  for (int b0 = 0; b0 < d->B; b0 += kMaxSlabB) {
    const int nb = d->B - b0 < kMaxSlabB ? d->B - b0 : kMaxSlabB;
    const bool first = b0 == 0, last = b0 + nb >= d->B;
    specsteer_status st = verify_slab(ctx, d, b0, nb, lean, s, first ? ctx->ev_stream_begin : nullptr,
                                      last ? ctx->ev_stream_end : nullptr, tail);
    if (st != SPECSTEER_OK) return st;
  }
  ctx->v_fused = tail;
  return SPECSTEER_OK;
}

specsteer_status do_recover(specsteer_ctx* ctx, const specsteer_round_desc* d, cudaStream_t s) {
  if (ctx->v_fused && d->recover_mode == SPECSTEER_RECOVER_STEER) return SPECSTEER_OK;   // the one launch did it
  const bool lean = ctx->v_two_phase;   // what the verification of this round did, not what this descriptor says
  for (int b0 = 0; b0 < d->B; b0 += kMaxSlabB) {
    const int nb = d->B - b0 < kMaxSlabB ? d->B - b0 : kMaxSlabB;
    specsteer_status st = recover_slab(ctx, d, b0, nb, lean, s);
    if (st != SPECSTEER_OK) return st;
  }
  return SPECSTEER_OK;
}

}  // namespace

extern "C" {

specsteer_status specsteer_ctx_create(specsteer_ctx** out, int device, int32_t max_B, int32_t max_K, int32_t max_V) {
  if (!out) return SPECSTEER_ERR_INVALID_ARG;
  *out = nullptr;
  if (max_B <= 0 || max_K < 0 || max_V <= 0 || device < 0) return SPECSTEER_ERR_INVALID_ARG;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device >= ndev) return SPECSTEER_ERR_CUDA;
  DeviceGuard g(device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  specsteer_ctx* c = new (std::nothrow) specsteer_ctx();
  if (!c) return SPECSTEER_ERR_WORKSPACE;
  memset(c, 0, sizeof *c);
  c->device = device; c->max_B = max_B; c->max_K = max_K; c->max_V = max_V;
  c->wait_cycles = kDefaultWaitCycles;
  c->li.device = device;
  if (cudaDeviceGetAttribute(&c->li.sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
      cudaDeviceGetAttribute(&c->li.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess) {
    delete c;
    return SPECSTEER_ERR_CUDA;
  }
  const size_t rows = (size_t)max_B * (max_K + 1);
  const size_t nch = (size_t)n_chunks_of(max_V, kChunkMin);
  const size_t b_part = align_up(rows * nch * 8 * sizeof(float), 256);
  const size_t b_lse = align_up(rows * 4 * sizeof(float), 256);
  const size_t b_st = align_up((size_t)max_B * sizeof(int), 256);
  const size_t b_tl = align_up((size_t)max_B * kTopkMaxSplit * 32 * sizeof(unsigned long long), 256);
  const size_t b_tc = align_up((size_t)max_B * sizeof(int), 256);
  c->ws_bytes = b_part + 2 * b_lse + 2 * b_st + 256 + b_tl + b_tc;
  if (cudaMalloc(&c->ws, c->ws_bytes) != cudaSuccess) {
    cudaGetLastError();
    delete c;
    return SPECSTEER_ERR_WORKSPACE;
  }
  char* w = (char*)c->ws;
  c->part = (float*)w; w += b_part;
  c->lse2 = (float*)w; w += b_lse;
  c->row_ref = (float*)w; w += b_lse;
  c->status_ws = (int*)w; w += b_st;
  c->req_done = (int*)w; w += b_st;
  c->dev_error = (int*)w; w += 256;
  c->topk_lists = (void*)w; w += b_tl;
  c->topk_count = (int*)w;
  if (cudaMemset(c->ws, 0, c->ws_bytes) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
    cudaFree(c->ws);
    delete c;
    return SPECSTEER_ERR_CUDA;
  }
  *out = c;
  return SPECSTEER_OK;
}

specsteer_status specsteer_ctx_destroy(specsteer_ctx* ctx) {
  if (!ctx) return SPECSTEER_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (ctx->host_ready) {
    for (int i = 0; i < 2; ++i) { cudaEventDestroy(ctx->ev_copied[i]); cudaEventDestroy(ctx->ev_done[i]); }
    cudaStreamDestroy(ctx->copy_stream);
  }
  if (ctx->stage) cudaFree(ctx->stage);
  if (ctx->lm_ws) cudaFree(ctx->lm_ws);
  if (ctx->lm_x2) cudaFree(ctx->lm_x2);
  if (ctx->ws) cudaFree(ctx->ws);
  delete ctx;
  return SPECSTEER_OK;
}

specsteer_status specsteer_verify_round(specsteer_ctx* ctx, const specsteer_round_desc* d, void* cuda_stream) {
  specsteer_status st = check_desc(ctx, d);
  if (st != SPECSTEER_OK) return st;
  if (ctx->poisoned) return SPECSTEER_ERR_TIMEOUT;
  ctx->verified = false;
  ctx->shard_streamed = false;
  if (d->B == 0) { ctx->verified = true; ctx->v_B = 0; ctx->v_K = d->K; ctx->v_V = d->V; ctx->v_dtype = d->dtype; ctx->v_h_llm = d->h_llm; return SPECSTEER_OK; }
  DeviceGuard g(ctx->device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  st = do_verify(ctx, d, (cudaStream_t)cuda_stream);
  if (st != SPECSTEER_OK) return st;
  ctx->v_two_phase = two_phase(d);
  ctx->verified = true;
  ctx->v_B = d->B; ctx->v_K = d->K; ctx->v_V = d->V; ctx->v_dtype = d->dtype; ctx->v_h_llm = d->h_llm;
  return SPECSTEER_OK;
}

specsteer_status specsteer_recover_sample(specsteer_ctx* ctx, const specsteer_round_desc* d, void* cuda_stream) {
  specsteer_status st = check_desc(ctx, d);
  if (st != SPECSTEER_OK) return st;
  if (ctx->poisoned) return SPECSTEER_ERR_TIMEOUT;
  if (!ctx->verified || ctx->v_B != d->B || ctx->v_K != d->K || ctx->v_V != d->V || ctx->v_dtype != d->dtype ||
      ctx->v_h_llm != d->h_llm)
    return SPECSTEER_ERR_ORDER;
  if (d->B == 0) return SPECSTEER_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  return do_recover(ctx, d, (cudaStream_t)cuda_stream);
}

// ---- vocabulary-sharded path -------------------------------------------------------------------------
namespace {
bool same_round(const specsteer_ctx* ctx, const specsteer_round_desc* d) {
  return ctx->v_B == d->B && ctx->v_K == d->K && ctx->v_V == d->V && ctx->v_dtype == d->dtype && ctx->v_h_llm == d->h_llm;
}
void remember_round(specsteer_ctx* ctx, const specsteer_round_desc* d) {
  ctx->v_B = d->B; ctx->v_K = d->K; ctx->v_V = d->V; ctx->v_dtype = d->dtype; ctx->v_h_llm = d->h_llm;
}
specsteer_status check_shard_args(const specsteer_round_desc* d, const void* gathered, int32_t n_shards, int32_t rank,
                                  int32_t vocab_offset, int32_t vocab_total) {
  if (!gathered || n_shards < 1 || n_shards > SPECSTEER_MAX_SHARDS || rank < 0 || rank >= n_shards) return SPECSTEER_ERR_INVALID_ARG;
  if (vocab_offset < 0 || vocab_total < d->V || (int64_t)vocab_offset + d->V > vocab_total) return SPECSTEER_ERR_INVALID_ARG;
  if (d->B > kMaxSlabB) return SPECSTEER_ERR_UNSUPPORTED;
  return SPECSTEER_OK;
}
}  // namespace

specsteer_status specsteer_shard_verify_local(specsteer_ctx* ctx, const specsteer_round_desc* d, int32_t vocab_offset,
                                              void* row_partials, void* cuda_stream) {
  specsteer_status st = check_desc(ctx, d);
  if (st != SPECSTEER_OK) return st;
  if (!row_partials || vocab_offset < 0 || d->B > kMaxSlabB) return SPECSTEER_ERR_INVALID_ARG;
  if (ctx->poisoned) return SPECSTEER_ERR_TIMEOUT;
  ctx->verified = false;
  ctx->shard_streamed = false;
  if (d->B > 0) {
    DeviceGuard g(ctx->device);
    if (!g.ok) return SPECSTEER_ERR_CUDA;
    RoundParams p = slab_params(ctx, d, 0, d->B);
    p.sums = SUM_ALL;
    p.vocab_offset = vocab_offset;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (launch_verify_stream(p, d->dtype, rows_aligned(d), ctx->li, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
    if (launch_shard_rows(p, d->dtype, (ShardPartial*)row_partials, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
    ctx->launches += 2;
  }
  remember_round(ctx, d);
  ctx->shard_streamed = true;
  return SPECSTEER_OK;
}

specsteer_status specsteer_shard_verify_combine(specsteer_ctx* ctx, const specsteer_round_desc* d, const void* gathered,
                                                int32_t n_shards, int32_t shard_rank, int32_t vocab_offset,
                                                int32_t vocab_total, void* cuda_stream) {
  specsteer_status st = check_desc(ctx, d);
  if (st != SPECSTEER_OK) return st;
  if ((st = check_shard_args(d, gathered, n_shards, shard_rank, vocab_offset, vocab_total)) != SPECSTEER_OK) return st;
  if (ctx->poisoned) return SPECSTEER_ERR_TIMEOUT;
  if (!ctx->shard_streamed || !same_round(ctx, d)) return SPECSTEER_ERR_ORDER;
  if (d->B > 0) {
    DeviceGuard g(ctx->device);
    if (!g.ok) return SPECSTEER_ERR_CUDA;
    RoundParams p = slab_params(ctx, d, 0, d->B);
    p.sums = SUM_ALL;
    p.shard_parts = (const ShardPartial*)gathered;
    p.n_shards = n_shards; p.shard_rank = shard_rank;
    p.vocab_offset = vocab_offset; p.vocab_total = vocab_total;
    if (launch_epilogue(p, d->dtype, (cudaStream_t)cuda_stream) != cudaSuccess) return SPECSTEER_ERR_CUDA;
    ctx->launches += 1;
  }
  ctx->v_two_phase = false;
  ctx->verified = true;
  return SPECSTEER_OK;
}

specsteer_status specsteer_shard_recover_local(specsteer_ctx* ctx, const specsteer_round_desc* d, const void* gathered,
                                               int32_t n_shards, int32_t shard_rank, int32_t vocab_offset,
                                               int32_t vocab_total, void* cuda_stream) {
  specsteer_status st = check_desc(ctx, d);
  if (st != SPECSTEER_OK) return st;
  if ((st = check_shard_args(d, gathered, n_shards, shard_rank, vocab_offset, vocab_total)) != SPECSTEER_OK) return st;
  if (d->recover_mode != SPECSTEER_RECOVER_STEER) return SPECSTEER_ERR_UNSUPPORTED;
  if (ctx->poisoned) return SPECSTEER_ERR_TIMEOUT;
  if (!ctx->verified || !ctx->shard_streamed || !same_round(ctx, d)) return SPECSTEER_ERR_ORDER;
  if (d->B == 0) return SPECSTEER_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  RoundParams p = slab_params(ctx, d, 0, d->B);
  p.sums = SUM_ALL;
  p.shard_parts = (const ShardPartial*)gathered;
  p.n_shards = n_shards; p.shard_rank = shard_rank;
  p.vocab_offset = vocab_offset; p.vocab_total = vocab_total;
  int nl = 0;
  if (launch_recover(p, d->dtype, ctx->li, (cudaStream_t)cuda_stream, &nl) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  ctx->launches += nl;
  return SPECSTEER_OK;
}

// Greedy recovery in the vocabulary-sharded round: this shard's best key per request (see the header).
specsteer_status specsteer_shard_greedy_local(specsteer_ctx* ctx, const specsteer_round_desc* d, int32_t vocab_offset,
                                              int64_t* best_keys, void* cuda_stream) {
  specsteer_status st = check_desc(ctx, d);
  if (st != SPECSTEER_OK) return st;
  if (!best_keys || vocab_offset < 0 || d->B > kMaxSlabB) return SPECSTEER_ERR_INVALID_ARG;
  if (d->recover_mode != SPECSTEER_RECOVER_ARGMAX) return SPECSTEER_ERR_UNSUPPORTED;
  if (ctx->poisoned) return SPECSTEER_ERR_TIMEOUT;
  if (!ctx->verified || !ctx->shard_streamed || !same_round(ctx, d)) return SPECSTEER_ERR_ORDER;
  if (d->B == 0) return SPECSTEER_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  RoundParams p = slab_params(ctx, d, 0, d->B);
  p.vocab_offset = vocab_offset;
  p.greedy_keys = (long long*)best_keys;
  if (launch_recover_argmax(p, d->dtype, rows_aligned(d), false, ctx->topk_lists, ctx->topk_count, ctx->li.sm_count,
                            (cudaStream_t)cuda_stream) != cudaSuccess)
    return SPECSTEER_ERR_CUDA;
  ctx->launches += 1;
  return SPECSTEER_OK;
}

// Last step of a sharded greedy round, the same on every GPU.  Only the per-request arrays of the descriptor are used
// (the LM-head rounds pass their embedded round descriptor, whose logit pointers are NULL).
specsteer_status specsteer_shard_greedy_finish(specsteer_ctx* ctx, const specsteer_round_desc* d, const int64_t* best_keys,
                                               void* cuda_stream) {
  if (!ctx || !d || !best_keys) return SPECSTEER_ERR_INVALID_ARG;
  if (d->B < 0 || d->K < 0 || d->B > ctx->max_B || d->K > ctx->max_K || d->B > kMaxSlabB) return SPECSTEER_ERR_INVALID_ARG;
  if (d->recover_mode != SPECSTEER_RECOVER_ARGMAX) return SPECSTEER_ERR_UNSUPPORTED;
  if (d->B > 0 && (!d->draft_len || !d->temperature || !d->accept_len || (d->K > 0 && !d->draft_tokens))) return SPECSTEER_ERR_INVALID_ARG;
  if (ctx->poisoned) return SPECSTEER_ERR_TIMEOUT;
  if (d->B == 0) return SPECSTEER_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  specsteer_round_desc dd = *d;
  dd.dtype = SPECSTEER_F32; dd.ld_row = d->V > 0 ? d->V : 1; dd.ld_req = (int64_t)(d->K + 1) * dd.ld_row;
  RoundParams p = slab_params(ctx, &dd, 0, d->B);
  if (launch_greedy_finish(p, (const long long*)best_keys, (cudaStream_t)cuda_stream) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  ctx->launches += 1;
  return SPECSTEER_OK;
}

namespace {
// Checks an LM-head descriptor, makes sure the second workspace exists and fills the kernels' parameters.
specsteer_status prep_lmhead(specsteer_ctx* ctx, const specsteer_lmhead_desc* ld, RoundParams* p, LmheadOperands* op) {
  if (!ctx || !ld) return SPECSTEER_ERR_INVALID_ARG;
  const specsteer_round_desc* d = &ld->round;
  if (d->B < 0 || d->K < 0 || d->V <= 0) return SPECSTEER_ERR_INVALID_ARG;
  if (d->accept_mode != SPECSTEER_ACCEPT_RATIO && d->accept_mode != SPECSTEER_ACCEPT_EXACT_Z) return SPECSTEER_ERR_INVALID_ARG;
  if (d->recover_mode != SPECSTEER_RECOVER_STEER && d->recover_mode != SPECSTEER_RECOVER_ARGMAX) return SPECSTEER_ERR_UNSUPPORTED;
  if (d->flags & ~(uint32_t)(SPECSTEER_FLAG_BONUS | SPECSTEER_FLAG_TWO_PHASE | SPECSTEER_FLAG_SEPARATE_LAUNCHES | SPECSTEER_FLAG_ONE_LAUNCH)) return SPECSTEER_ERR_INVALID_ARG;
  if (ld->d_llm <= 0 || ld->d_slm <= 0) return SPECSTEER_ERR_INVALID_ARG;
  if (ld->d_llm % 8 || ld->d_slm % 8) return SPECSTEER_ERR_UNSUPPORTED;   // rows of the operands must be 16-byte multiples
  if (d->B > 0) {
    if (!ld->x_llm || !ld->w_llm || !ld->x_slm_plus || !ld->w_slm_plus || !ld->x_slm_minus || !ld->w_slm_minus ||
        !d->draft_len || !d->lambda || !d->beta || !d->temperature || !d->u_recover || !d->accept_len)
      return SPECSTEER_ERR_INVALID_ARG;
    if (d->K > 0 && (!d->draft_tokens || !d->u_accept)) return SPECSTEER_ERR_INVALID_ARG;
    const void* ops[6] = {ld->x_llm, ld->w_llm, ld->x_slm_plus, ld->w_slm_plus, ld->x_slm_minus, ld->w_slm_minus};
    for (const void* o : ops)
      if ((uintptr_t)o & 15u) return SPECSTEER_ERR_UNSUPPORTED;
  }
  if (d->B > ctx->max_B || d->K > ctx->max_K || d->V > ctx->max_V) return SPECSTEER_ERR_UNSUPPORTED;
  if ((size_t)(ld->d_llm + 2 * ld->d_slm) * 2 + (size_t)n_chunks_of(d->V, kLmheadChunk) * 8 + 64 > 200 * 1024)
    return SPECSTEER_ERR_UNSUPPORTED;   // the recovery kernel keeps the row's hidden states and chunk weights in shared memory
  if (ctx->poisoned) return SPECSTEER_ERR_TIMEOUT;
  if (d->B == 0) return SPECSTEER_OK;
  const int K1 = d->K + 1;
  if (!ctx->lm_ws) {   // sized for the context's maxima, once
    const size_t rows = (size_t)ctx->max_B * (ctx->max_K + 1);
    const size_t part_bytes = align_up(rows * (size_t)n_chunks_of(ctx->max_V, kLmheadChunk) * 32, 256);
    const size_t tok_bytes = align_up(rows * 16, 256);
    const size_t key_bytes = align_up(rows * (size_t)n_chunks_of(ctx->max_V, kLmheadChunk) * 8, 256);
    if (cudaMalloc(&ctx->lm_ws, part_bytes + tok_bytes + key_bytes) != cudaSuccess) { ctx->lm_ws = nullptr; (void)cudaGetLastError(); return SPECSTEER_ERR_WORKSPACE; }
    ctx->lm_part = (float*)ctx->lm_ws;
    ctx->lm_tok = (float*)((char*)ctx->lm_ws + part_bytes);
    ctx->lm_keys = (char*)ctx->lm_ws + part_bytes + tok_bytes;
    ctx->ws_bytes += part_bytes + tok_bytes + key_bytes;
  }
  specsteer_round_desc dd = *d;
  dd.dtype = SPECSTEER_F32; dd.ld_row = d->V; dd.ld_req = (int64_t)K1 * d->V;   // no logit tensor exists
  *p = slab_params(ctx, &dd, 0, d->B);
  p->h_llm = p->h_plus = p->h_minus = nullptr;
  p->sums = SUM_ALL;
  p->row_mode = ROWS_ALL;
  p->tile = kLmheadChunk;
  p->n_chunks = n_chunks_of(d->V, kLmheadChunk);
  p->part = ctx->lm_part;
  p->tok_logits = ctx->lm_tok;
  op->x_llm = (const uint16_t*)ld->x_llm; op->w_llm = (const uint16_t*)ld->w_llm;
  op->x_plus = (const uint16_t*)ld->x_slm_plus; op->w_plus = (const uint16_t*)ld->w_slm_plus;
  op->x_minus = (const uint16_t*)ld->x_slm_minus; op->w_minus = (const uint16_t*)ld->w_slm_minus;
  op->d_llm = ld->d_llm; op->d_slm = ld->d_slm;
  return SPECSTEER_OK;
}
}  // namespace

namespace {
// The two-phase round on the LM-head path (only Algorithm 1's outputs wanted: the ratio rule, STEER or ARGMAX recovery,
// none of logp_plus, logp_star, log_z): verification forms h_LLM and h_SLM- alone, in tiles twice as wide (Eq. 7);
// then the hidden states of row accept_len of every request that takes a token are compacted and the three-product
// kernel forms all three logit rows of just those positions (Eq. 8), from which the token is sampled (or the argmax
// taken) exactly as in the one-pass round.
bool lmhead_two_phase(const specsteer_round_desc* d) {
  return d->accept_mode == SPECSTEER_ACCEPT_RATIO &&
         (d->recover_mode == SPECSTEER_RECOVER_STEER || d->recover_mode == SPECSTEER_RECOVER_ARGMAX) && !d->logp_plus &&
         !d->logp_star && !d->log_z && !(d->flags & SPECSTEER_FLAG_SEPARATE_LAUNCHES);
}

specsteer_status lmhead_round_two_phase(specsteer_ctx* ctx, const specsteer_lmhead_desc* ld, RoundParams p, LmheadOperands op,
                                        cudaStream_t s) {
  const specsteer_round_desc* d = &ld->round;
  const int B = d->B;
  // compact operands and per-request scratch (grown when a call needs more)
  const size_t x_bytes = align_up((size_t)ctx->max_B * (size_t)(op.d_llm + 2 * op.d_slm) * 2, 256);
  const size_t need = x_bytes + 3 * align_up((size_t)ctx->max_B * sizeof(int), 256);
  if (need > ctx->lm_x2_bytes) {
    if (ctx->lm_x2) { cudaStreamSynchronize(s); cudaFree(ctx->lm_x2); ctx->lm_x2 = nullptr; ctx->lm_x2_bytes = 0; }
    if (cudaMalloc(&ctx->lm_x2, need) != cudaSuccess) { (void)cudaGetLastError(); return SPECSTEER_ERR_WORKSPACE; }
    ctx->lm_x2_bytes = need;
    ctx->ws_bytes += need;
  }
  uint16_t* xl = (uint16_t*)ctx->lm_x2;
  uint16_t* xp = xl + (size_t)ctx->max_B * op.d_llm;
  uint16_t* xm = xp + (size_t)ctx->max_B * op.d_slm;
  int* c_n = (int*)((char*)ctx->lm_x2 + x_bytes);
  int* c_status = c_n + align_up((size_t)ctx->max_B * sizeof(int), 256) / sizeof(int);
  int* c_token = c_status + align_up((size_t)ctx->max_B * sizeof(int), 256) / sizeof(int);
  const bool greedy = d->recover_mode == SPECSTEER_RECOVER_ARGMAX;

  // 1. verification alone: h_LLM, h_SLM- of every row; 2. the per-request epilogue over the drafted rows
  RoundParams pv = p;
  pv.sums = SUM_L | SUM_M;
  pv.row_mode = ROWS_DRAFTED;
  pv.tile = kLmheadRatioChunk;
  pv.n_chunks = n_chunks_of(d->V, kLmheadRatioChunk);
  if (ctx->ev_stream_begin && cudaEventRecord(ctx->ev_stream_begin, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  if (launch_lmhead_ratio(pv, op, ctx->lm_tok, ctx->li, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  if (launch_epilogue(pv, SPECSTEER_F32, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  // 3. the recovery rows, compacted; 4. all three products on them (one row per request: a round with K = 0)
  if (launch_lmhead_gather_rows(p, op, xl, xp, xm, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  RoundParams pc = p;
  pc.K = 0;
  pc.flags = p.flags | SPECSTEER_FLAG_BONUS;
  pc.sums = SUM_ALL;
  pc.row_mode = ROWS_ALL;
  pc.accept_len = c_n; pc.status_ws = c_status; pc.req_status = nullptr;
  pc.accept_flags = nullptr; pc.alpha = nullptr; pc.logp_llm = nullptr; pc.logp_minus = nullptr; pc.logp_plus = nullptr;
  pc.logp_star = nullptr; pc.log_z = nullptr; pc.out_tokens = nullptr; pc.n_out = nullptr;
  pc.rec_token = c_token;
  LmheadOperands oc = op;
  oc.x_llm = xl; oc.x_plus = xp; oc.x_minus = xm;
  if (launch_lmhead(pc, oc, ctx->lm_tok, greedy ? ctx->lm_keys : nullptr, ctx->li, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  if (ctx->ev_stream_end && cudaEventRecord(ctx->ev_stream_end, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  // 5. the normalisers of those rows (and whether they are finite); 6. the token; 7. the round's outputs
  if (launch_epilogue(pc, SPECSTEER_F32, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  if ((greedy ? launch_lmhead_argmax(pc, ctx->lm_keys, s) : launch_lmhead_recover(pc, oc, s)) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  if (launch_lmhead_finish(p, c_status, c_token, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  ctx->launches += 7;
  (void)B;
  return SPECSTEER_OK;
}
}  // namespace

specsteer_status specsteer_lmhead_round(specsteer_ctx* ctx, const specsteer_lmhead_desc* ld, void* cuda_stream) {
  RoundParams p;
  LmheadOperands op;
  specsteer_status st = prep_lmhead(ctx, ld, &p, &op);
  if (st != SPECSTEER_OK) return st;
  ctx->verified = false;
  ctx->shard_streamed = false;
  if (ld->round.B == 0) return SPECSTEER_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  if (lmhead_two_phase(&ld->round)) return lmhead_round_two_phase(ctx, ld, p, op, s);
  if (ctx->ev_stream_begin && cudaEventRecord(ctx->ev_stream_begin, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  const bool greedy = ld->round.recover_mode == SPECSTEER_RECOVER_ARGMAX;
  if (launch_lmhead(p, op, ctx->lm_tok, greedy ? ctx->lm_keys : nullptr, ctx->li, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  if (ctx->ev_stream_end && cudaEventRecord(ctx->ev_stream_end, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  if (launch_epilogue(p, SPECSTEER_F32, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  if ((greedy ? launch_lmhead_argmax(p, ctx->lm_keys, s) : launch_lmhead_recover(p, op, s)) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  ctx->launches += 3;
  return SPECSTEER_OK;
}

// The same round with the heads split along the vocabulary over several GPUs (a tensor-parallel LM head).
specsteer_status specsteer_lmhead_shard_local(specsteer_ctx* ctx, const specsteer_lmhead_desc* ld, int32_t vocab_offset,
                                              void* row_partials, void* cuda_stream) {
  RoundParams p;
  LmheadOperands op;
  specsteer_status st = prep_lmhead(ctx, ld, &p, &op);
  if (st != SPECSTEER_OK) return st;
  if (!row_partials || vocab_offset < 0 || ld->round.B > kMaxSlabB) return SPECSTEER_ERR_INVALID_ARG;
  ctx->verified = false;
  ctx->shard_streamed = false;
  if (ld->round.B == 0) return SPECSTEER_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  p.vocab_offset = vocab_offset;
  p.vocab_total = vocab_offset + ld->round.V;
  // the "token met" words must start at zero: a token outside this shard leaves its row untouched
  if (cudaMemsetAsync(ctx->lm_tok, 0, (size_t)ld->round.B * (ld->round.K + 1) * 16, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  if (ctx->ev_stream_begin && cudaEventRecord(ctx->ev_stream_begin, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  const bool greedy = ld->round.recover_mode == SPECSTEER_RECOVER_ARGMAX;   // the per-tile keys carry global ids
  if (launch_lmhead(p, op, ctx->lm_tok, greedy ? ctx->lm_keys : nullptr, ctx->li, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  if (ctx->ev_stream_end && cudaEventRecord(ctx->ev_stream_end, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  if (launch_shard_rows(p, SPECSTEER_F32, (ShardPartial*)row_partials, s) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  ctx->launches += 2;
  return SPECSTEER_OK;
}

specsteer_status specsteer_lmhead_shard_combine(specsteer_ctx* ctx, const specsteer_lmhead_desc* ld, const void* gathered,
                                                int32_t n_shards, int32_t shard_rank, int32_t vocab_offset,
                                                int32_t vocab_total, void* cuda_stream) {
  RoundParams p;
  LmheadOperands op;
  specsteer_status st = prep_lmhead(ctx, ld, &p, &op);
  if (st != SPECSTEER_OK) return st;
  if ((st = check_shard_args(&ld->round, gathered, n_shards, shard_rank, vocab_offset, vocab_total)) != SPECSTEER_OK) return st;
  if (ld->round.B == 0) return SPECSTEER_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  p.shard_parts = (const ShardPartial*)gathered;
  p.n_shards = n_shards; p.shard_rank = shard_rank;
  p.vocab_offset = vocab_offset; p.vocab_total = vocab_total;
  p.tok_logits = nullptr;   // the tokens' logits travel inside the partials
  if (launch_epilogue(p, SPECSTEER_F32, (cudaStream_t)cuda_stream) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  ctx->launches += 1;
  return SPECSTEER_OK;
}

specsteer_status specsteer_lmhead_shard_recover(specsteer_ctx* ctx, const specsteer_lmhead_desc* ld, const void* gathered,
                                                int32_t n_shards, int32_t shard_rank, int32_t vocab_offset,
                                                int32_t vocab_total, void* cuda_stream) {
  RoundParams p;
  LmheadOperands op;
  specsteer_status st = prep_lmhead(ctx, ld, &p, &op);
  if (st != SPECSTEER_OK) return st;
  if ((st = check_shard_args(&ld->round, gathered, n_shards, shard_rank, vocab_offset, vocab_total)) != SPECSTEER_OK) return st;
  if (ld->round.recover_mode != SPECSTEER_RECOVER_STEER) return SPECSTEER_ERR_UNSUPPORTED;
  if (ld->round.B == 0) return SPECSTEER_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  p.shard_parts = (const ShardPartial*)gathered;
  p.n_shards = n_shards; p.shard_rank = shard_rank;
  p.vocab_offset = vocab_offset; p.vocab_total = vocab_total;
  if (launch_lmhead_recover(p, op, (cudaStream_t)cuda_stream) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  ctx->launches += 1;
  return SPECSTEER_OK;
}

// Greedy recovery with the heads split along the vocabulary: this shard's best key per request, from the per-tile
// keys the tensor-core pass of specsteer_lmhead_shard_local left (after specsteer_lmhead_shard_combine).
specsteer_status specsteer_lmhead_shard_greedy_local(specsteer_ctx* ctx, const specsteer_lmhead_desc* ld, int64_t* best_keys,
                                                     void* cuda_stream) {
  RoundParams p;
  LmheadOperands op;
  specsteer_status st = prep_lmhead(ctx, ld, &p, &op);
  if (st != SPECSTEER_OK) return st;
  if (!best_keys || ld->round.B > kMaxSlabB) return SPECSTEER_ERR_INVALID_ARG;
  if (ld->round.recover_mode != SPECSTEER_RECOVER_ARGMAX) return SPECSTEER_ERR_UNSUPPORTED;
  if (ld->round.B == 0) return SPECSTEER_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  p.greedy_keys = (long long*)best_keys;
  if (launch_lmhead_argmax(p, ctx->lm_keys, (cudaStream_t)cuda_stream) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  ctx->launches += 1;
  return SPECSTEER_OK;
}

specsteer_status specsteer_cloud_topk(specsteer_ctx* ctx, const specsteer_round_desc* d, int32_t k, int32_t* topk_idx,
                                      float* topk_val, void* cuda_stream) {
  specsteer_status st = check_desc(ctx, d);
  if (st != SPECSTEER_OK) return st;
  if (k < 1 || k > SPECSTEER_TOPK_MAX || !topk_idx || !topk_val) return SPECSTEER_ERR_INVALID_ARG;
  if (ctx->poisoned) return SPECSTEER_ERR_TIMEOUT;
  if (!ctx->verified || ctx->v_B != d->B || ctx->v_K != d->K || ctx->v_V != d->V || ctx->v_dtype != d->dtype ||
      ctx->v_h_llm != d->h_llm)
    return SPECSTEER_ERR_ORDER;
  if (d->B == 0) return SPECSTEER_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  RoundParams p = slab_params(ctx, d, 0, d->B);
  if (launch_cloud_topk(p, d->dtype, k, topk_idx, topk_val, ctx->topk_lists, ctx->topk_count, ctx->li.sm_count,
                        (cudaStream_t)cuda_stream) != cudaSuccess)
    return SPECSTEER_ERR_CUDA;
  ctx->launches += 1;
  return SPECSTEER_OK;
}

specsteer_status specsteer_edge_resample(specsteer_ctx* ctx, const specsteer_round_desc* d, int32_t k,
                                         const int32_t* topk_idx, const float* topk_val, void* cuda_stream) {
  specsteer_status st = check_desc(ctx, d);
  if (st != SPECSTEER_OK) return st;
  if (k < 1 || k > SPECSTEER_TOPK_MAX || !topk_idx || !topk_val) return SPECSTEER_ERR_INVALID_ARG;
  if (ctx->poisoned) return SPECSTEER_ERR_TIMEOUT;
  if (!ctx->verified || ctx->v_B != d->B || ctx->v_K != d->K || ctx->v_V != d->V || ctx->v_dtype != d->dtype ||
      ctx->v_h_llm != d->h_llm)
    return SPECSTEER_ERR_ORDER;
  if (d->B == 0) return SPECSTEER_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  RoundParams p = slab_params(ctx, d, 0, d->B);
  if (launch_edge_resample(p, d->dtype, k, topk_idx, topk_val, (cudaStream_t)cuda_stream) != cudaSuccess)
    return SPECSTEER_ERR_CUDA;
  ctx->launches += 1;
  return SPECSTEER_OK;
}

specsteer_status specsteer_round_host(specsteer_ctx* ctx, const specsteer_round_desc* h, void* cuda_stream) {
  specsteer_status st = check_desc(ctx, h);
  if (st != SPECSTEER_OK) return st;
  if (ctx->poisoned) return SPECSTEER_ERR_TIMEOUT;
  if (h->B == 0) return SPECSTEER_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const int B = h->B, K = h->K, K1 = K + 1;
  const size_t es = h->dtype == SPECSTEER_F32 ? 4 : 2;
  if (!ctx->host_ready) {
    if (cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return SPECSTEER_ERR_CUDA;
    for (int i = 0; i < 2; ++i) {
      if (cudaEventCreateWithFlags(&ctx->ev_copied[i], cudaEventDisableTiming) != cudaSuccess ||
          cudaEventCreateWithFlags(&ctx->ev_done[i], cudaEventDisableTiming) != cudaSuccess)
        return SPECSTEER_ERR_CUDA;
    }
    ctx->host_ready = true;
  }
  // device staging: the three logit tensors (as strided as the caller's) + the small per-request arrays
  const size_t logit_bytes = align_up((size_t)B * h->ld_req * es, 256);
  const size_t small = align_up((size_t)B * (size_t)(K1 * 64 + 128) + 1024, 256);
  const size_t need = 3 * logit_bytes + small;
  if (need > ctx->stage_bytes) {
    if (ctx->stage) { cudaStreamSynchronize(s); cudaFree(ctx->stage); ctx->stage = nullptr; ctx->stage_bytes = 0; }
    if (cudaMalloc(&ctx->stage, need) != cudaSuccess) { cudaGetLastError(); return SPECSTEER_ERR_WORKSPACE; }
    ctx->stage_bytes = need;
  }
  char* base = (char*)ctx->stage;
  specsteer_round_desc d = *h;
  d.h_llm = base; d.h_slm_plus = base + logit_bytes; d.h_slm_minus = base + 2 * logit_bytes;
  char* w = base + 3 * logit_bytes;
  auto carve = [&](size_t bytes) { char* r = w; w += align_up(bytes, 16); return r; };
  int32_t* tok = (int32_t*)carve((size_t)B * K * 4); int32_t* len = (int32_t*)carve((size_t)B * 4);
  float* lam = (float*)carve((size_t)B * 4); float* beta = (float*)carve((size_t)B * 4);
  float* tmp = (float*)carve((size_t)B * 4); float* ua = (float*)carve((size_t)B * K * 4);
  float* ur = (float*)carve((size_t)B * 4);
  d.draft_tokens = tok; d.draft_len = len; d.lambda = lam; d.beta = beta; d.temperature = tmp;
  d.u_accept = ua; d.u_recover = ur;
  d.accept_len = (int32_t*)carve((size_t)B * 4);
  d.accept_flags = h->accept_flags ? (uint8_t*)carve((size_t)B * K) : nullptr;
  d.alpha = h->alpha ? (float*)carve((size_t)B * K * 4) : nullptr;
  d.logp_llm = h->logp_llm ? (float*)carve((size_t)B * K * 4) : nullptr;
  d.logp_minus = h->logp_minus ? (float*)carve((size_t)B * K * 4) : nullptr;
  d.logp_plus = h->logp_plus ? (float*)carve((size_t)B * K * 4) : nullptr;
  d.logp_star = h->logp_star ? (float*)carve((size_t)B * K * 4) : nullptr;
  d.log_z = h->log_z ? (float*)carve((size_t)B * K1 * 4) : nullptr;
  d.rec_token = h->rec_token ? (int32_t*)carve((size_t)B * 4) : nullptr;
  d.rec_logprob = h->rec_logprob ? (float*)carve((size_t)B * 4) : nullptr;
  d.out_tokens = h->out_tokens ? (int32_t*)carve((size_t)B * K1 * 4) : nullptr;
  d.n_out = h->n_out ? (int32_t*)carve((size_t)B * 4) : nullptr;
  d.req_status = h->req_status ? (int32_t*)carve((size_t)B * 4) : nullptr;

  bool fail = false;
#define CK(x) do { if ((x) != cudaSuccess) fail = true; } while (0)
  // small inputs first, on the compute stream
  if (K > 0) { CK(cudaMemcpyAsync(tok, h->draft_tokens, (size_t)B * K * 4, cudaMemcpyHostToDevice, s));
               CK(cudaMemcpyAsync(ua, h->u_accept, (size_t)B * K * 4, cudaMemcpyHostToDevice, s)); }
  CK(cudaMemcpyAsync(len, h->draft_len, (size_t)B * 4, cudaMemcpyHostToDevice, s));
  CK(cudaMemcpyAsync(lam, h->lambda, (size_t)B * 4, cudaMemcpyHostToDevice, s));
  CK(cudaMemcpyAsync(beta, h->beta, (size_t)B * 4, cudaMemcpyHostToDevice, s));
  CK(cudaMemcpyAsync(tmp, h->temperature, (size_t)B * 4, cudaMemcpyHostToDevice, s));
  CK(cudaMemcpyAsync(ur, h->u_recover, (size_t)B * 4, cudaMemcpyHostToDevice, s));
  // the copy stream must not overwrite staging still in use by work queued earlier on `s`
  CK(cudaEventRecord(ctx->ev_done[0], s));
  CK(cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_done[0], 0));

  const size_t req_bytes = (size_t)h->ld_req * es;
  const size_t row_bytes = (size_t)h->ld_row * es;
  specsteer_round_desc forced = d;
  forced.flags |= SPECSTEER_FLAG_TWO_PHASE;
  if (two_phase(&forced)) {
    // Only Algorithm 1's outputs are wanted: the link, not the GPU, bounds this call, so copy only what the two-phase
    // round reads.  First rows [0, K) of h_LLM and h_SLM-, slab by slab, each slab verified while the next one is
    // copied; then, with the accepted lengths on the host, row accept_len of h_SLM+ for every request that takes a token
    // (and of the other two tensors when that row is the bonus row, which verification did not need); then recovery.
    size_t per2 = (size_t)(96u << 20) / (2 * req_bytes);
    const int slab2 = (int)(per2 < 1 ? 1 : (per2 > (size_t)kMaxSlabB ? (size_t)kMaxSlabB : per2));
    int idx2 = 0;
    for (int b0 = 0; b0 < B && !fail; b0 += slab2, idx2 ^= 1) {
      const int nb = B - b0 < slab2 ? B - b0 : slab2;
      if (K > 0) {   // rows [0, K) of every request of the slab: one strided copy per tensor (rows beyond draft_len ride along)
        const size_t o = (size_t)b0 * req_bytes;
        CK(cudaMemcpy2DAsync((char*)d.h_llm + o, req_bytes, (const char*)h->h_llm + o, req_bytes, (size_t)K * row_bytes, nb,
                             cudaMemcpyHostToDevice, ctx->copy_stream));
        CK(cudaMemcpy2DAsync((char*)d.h_slm_minus + o, req_bytes, (const char*)h->h_slm_minus + o, req_bytes,
                             (size_t)K * row_bytes, nb, cudaMemcpyHostToDevice, ctx->copy_stream));
      }
      CK(cudaEventRecord(ctx->ev_copied[idx2], ctx->copy_stream));
      CK(cudaStreamWaitEvent(s, ctx->ev_copied[idx2], 0));
      if (verify_slab(ctx, &forced, b0, nb, true, s, nullptr, nullptr, false) != SPECSTEER_OK) fail = true;
    }
    int32_t* n_host = (int32_t*)malloc((size_t)B * 8);
    if (!n_host) fail = true;
    if (!fail) {
      int32_t* st_host = n_host + B;
      CK(cudaMemcpyAsync(n_host, d.accept_len, (size_t)B * 4, cudaMemcpyDeviceToHost, s));
      CK(cudaMemcpyAsync(st_host, ctx->status_ws, (size_t)B * 4, cudaMemcpyDeviceToHost, s));
      CK(cudaStreamSynchronize(s));
      // single rows, many of them: spread over both streams so that one copy's set-up hides behind another's transfer
      int turn = 0;
      auto row_copy = [&](void* dst, const void* src) {
        CK(cudaMemcpyAsync(dst, src, row_bytes, cudaMemcpyHostToDevice, (turn++ & 1) ? ctx->copy_stream : s));
      };
      for (int b = 0; b < B && !fail; ++b) {
        int ln = h->draft_len[b];
        if (ln < 0 || ln > K) ln = 0;
        const int n = n_host[b];
        const bool bad = (st_host[b] & (SPECSTEER_REQ_BAD_PARAM | SPECSTEER_REQ_NONFINITE)) != 0;
        if (bad || n < 0 || n > ln || !(n < ln || (h->flags & SPECSTEER_FLAG_BONUS))) continue;
        const size_t o = (size_t)b * req_bytes + (size_t)n * row_bytes;
        row_copy((char*)d.h_slm_plus + o, (const char*)h->h_slm_plus + o);
        if (n >= K) {   // the bonus row of a request with K drafts: the first copies stopped before it
          row_copy((char*)d.h_llm + o, (const char*)h->h_llm + o);
          row_copy((char*)d.h_slm_minus + o, (const char*)h->h_slm_minus + o);
        }
      }
      CK(cudaEventRecord(ctx->ev_copied[0], ctx->copy_stream));
      CK(cudaStreamWaitEvent(s, ctx->ev_copied[0], 0));
      for (int b0 = 0; b0 < B && !fail; b0 += kMaxSlabB) {
        const int nb = B - b0 < kMaxSlabB ? B - b0 : kMaxSlabB;
        if (recover_slab(ctx, &forced, b0, nb, true, s) != SPECSTEER_OK) fail = true;
      }
    }
    free(n_host);
  } else {
  // slabs of requests: copy slab i+1 on the copy stream while slab i computes on `s`
  size_t per = (size_t)(96u << 20) / (3 * req_bytes);
  int slab = (int)(per < 1 ? 1 : (per > (size_t)kMaxSlabB ? (size_t)kMaxSlabB : per));
  int idx = 0;
  for (int b0 = 0; b0 < B && !fail; b0 += slab, idx ^= 1) {
    const int nb = B - b0 < slab ? B - b0 : slab;
    const size_t o = (size_t)b0 * req_bytes, nbytes = (size_t)nb * req_bytes;
    CK(cudaMemcpyAsync((char*)d.h_llm + o, (const char*)h->h_llm + o, nbytes, cudaMemcpyHostToDevice, ctx->copy_stream));
    CK(cudaMemcpyAsync((char*)d.h_slm_plus + o, (const char*)h->h_slm_plus + o, nbytes, cudaMemcpyHostToDevice, ctx->copy_stream));
    CK(cudaMemcpyAsync((char*)d.h_slm_minus + o, (const char*)h->h_slm_minus + o, nbytes, cudaMemcpyHostToDevice, ctx->copy_stream));
    CK(cudaEventRecord(ctx->ev_copied[idx], ctx->copy_stream));
    CK(cudaStreamWaitEvent(s, ctx->ev_copied[idx], 0));
    RoundParams p = slab_params(ctx, &d, b0, nb);
    int nl = 0;
    const bool tail = tail_in_one_launch(&d, false);   // epilogue and STEER sample in one launch
    CK(launch_verify(p, d.dtype, rows_aligned(&d), ctx->li, s, &nl, nullptr, nullptr, tail)); ctx->launches += nl;
    if (tail) {
    } else if (d.recover_mode == SPECSTEER_RECOVER_ARGMAX) {
      CK(launch_recover_argmax(p, d.dtype, rows_aligned(&d), false, (char*)ctx->topk_lists + (size_t)b0 * kTopkMaxSplit * 32 * 8,
                               ctx->topk_count + b0, ctx->li.sm_count, s));
      ctx->launches += 1;
    } else {
      CK(launch_recover(p, d.dtype, ctx->li, s, &nl)); ctx->launches += nl;
    }
  }
  }
  auto back = [&](void* hp, const void* dp, size_t bytes) {
    if (hp && dp && bytes) CK(cudaMemcpyAsync(hp, dp, bytes, cudaMemcpyDeviceToHost, s));
  };
  back(h->accept_len, d.accept_len, (size_t)B * 4); back(h->accept_flags, d.accept_flags, (size_t)B * K);
  back(h->alpha, d.alpha, (size_t)B * K * 4); back(h->logp_llm, d.logp_llm, (size_t)B * K * 4);
  back(h->logp_minus, d.logp_minus, (size_t)B * K * 4); back(h->logp_plus, d.logp_plus, (size_t)B * K * 4);
  back(h->logp_star, d.logp_star, (size_t)B * K * 4); back(h->log_z, d.log_z, (size_t)B * K1 * 4);
  back(h->rec_token, d.rec_token, (size_t)B * 4); back(h->rec_logprob, d.rec_logprob, (size_t)B * 4);
  back(h->out_tokens, d.out_tokens, (size_t)B * K1 * 4); back(h->n_out, d.n_out, (size_t)B * 4);
  back(h->req_status, d.req_status, (size_t)B * 4);
#undef CK
  if (cudaStreamSynchronize(s) != cudaSuccess) fail = true;
  ctx->verified = false;
  if (fail) { cudaGetLastError(); return SPECSTEER_ERR_CUDA; }
  return SPECSTEER_OK;
}

specsteer_status specsteer_ctx_device_error(specsteer_ctx* ctx) {
  if (!ctx) return SPECSTEER_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SPECSTEER_ERR_CUDA;
  int flag = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return SPECSTEER_ERR_CUDA;
  if (cudaMemcpy(&flag, ctx->dev_error, sizeof flag, cudaMemcpyDeviceToHost) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  if (flag) ctx->poisoned = true;
  return flag ? SPECSTEER_ERR_TIMEOUT : SPECSTEER_OK;
}

specsteer_status specsteer_ctx_set_wait_limit(specsteer_ctx* ctx, int64_t sm_clocks) {
  if (!ctx || sm_clocks < 0) return SPECSTEER_ERR_INVALID_ARG;
  ctx->wait_cycles = sm_clocks == 0 ? kDefaultWaitCycles : (long long)sm_clocks;
  return SPECSTEER_OK;
}

specsteer_status specsteer_ctx_time_streaming(specsteer_ctx* ctx, void* ev_begin, void* ev_end) {
  if (!ctx || ((ev_begin == nullptr) != (ev_end == nullptr))) return SPECSTEER_ERR_INVALID_ARG;
  ctx->ev_stream_begin = (cudaEvent_t)ev_begin;
  ctx->ev_stream_end = (cudaEvent_t)ev_end;
  return SPECSTEER_OK;
}

size_t specsteer_ctx_workspace_bytes(const specsteer_ctx* ctx) { return ctx ? ctx->ws_bytes : 0; }
uint64_t specsteer_ctx_launch_count(const specsteer_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* specsteer_status_string(specsteer_status s) {
  switch (s) {
    case SPECSTEER_OK: return "ok";
    case SPECSTEER_ERR_INVALID_ARG: return "invalid argument";
    case SPECSTEER_ERR_UNSUPPORTED: return "shape exceeds the context's maxima";
    case SPECSTEER_ERR_WORKSPACE: return "device allocation failed";
    case SPECSTEER_ERR_CUDA: return "CUDA runtime error";
    case SPECSTEER_ERR_ORDER: return "recover_sample without a matching verify_round";
    case SPECSTEER_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    case SPECSTEER_ERR_STATIC_LIMIT:
      return "shape exceeds the fixed scratch of specsteer_verify_round_static "
             "(B <= 1024, B*(K+1) <= 16384, B*(K+1)*ceil(V/chunk) <= 229376)";
  }
  return "unknown status";
}

uint32_t specsteer_version(void) { return (0u << 16) | (1u << 8) | 0u; }

}  // extern "C"
