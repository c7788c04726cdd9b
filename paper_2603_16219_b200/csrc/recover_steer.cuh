// Recovery by inverse CDF from the per-chunk partial records (Algorithm 1 Phase 3; Eq. 8): the pieces that both the
// stand-alone recovery kernel and the one-launch round of the streaming kernel use.
#pragma once
#include "common.cuh"
#include "internal.h"
#include "records.cuh"
#include "specsteer.h"

namespace specsteer {

constexpr int kRecThreads = 256;
constexpr int kRecWarps = kRecThreads / 32;

struct PickShared {
  double warp_tot[kRecWarps];
  double base, target, W;
  int jstar, jlast;
  int tok_min, tok_max_pos;
  int plan_owner;            // sharded vocabulary: the shard that holds the CDF target, -1 if nothing can be sampled
  double plan_target, plan_W;  // the target within that shard, and the weight of the whole row
};

// The barrier of the kRecThreads threads that work on one request: the whole CTA (BAR = 0) or, inside a kernel
// whose other warps do something else, the named barrier BAR.
template <int BAR>
__device__ __forceinline__ void rec_sync() {
  if (BAR == 0) __syncthreads();
  else asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(kRecThreads) : "memory");
}

// Exclusive prefix of one double per thread over the kRecThreads threads, in thread order.
template <int BAR>
__device__ __forceinline__ double block_excl_scan(double v, double* warp_tot, int tid) {
  const int lane = tid & 31, warp = tid >> 5;
  double inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    double u = __shfl_up_sync(kFullMask, inc, o);
    if (lane >= o) inc += u;
  }
  if (lane == 31) warp_tot[warp] = inc;
  rec_sync<BAR>();
  double off = 0.0;
  for (int w = 0; w < warp; ++w) off += warp_tot[w];
  rec_sync<BAR>();
  return off + inc - v;
}

// Walk chunk `jstar`: the smallest v with base + sum_{chunk start..v} w > target, else the last v with w > 0.
// w[] are this thread's PER weights for entries v0 .. v0+PER-1 (0 beyond V).
template <int PER, int BAR>
__device__ __forceinline__ int pick_in_chunk(const double (&w)[PER], int v0, PickShared* sh, int tid) {
  constexpr int kPerThread = PER;
  double local = 0.0;
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) local += w[i];
  const double excl = block_excl_scan<BAR>(local, sh->warp_tot, tid);
  double run = sh->base + excl;
  int cand = 0x7fffffff, lastpos = -1;
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    run += w[i];
    if (w[i] > 0.0) lastpos = v0 + i;
    if (run > sh->target && cand == 0x7fffffff) cand = v0 + i;
  }
  if (cand != 0x7fffffff) atomicMin(&sh->tok_min, cand);
  if (lastpos >= 0) atomicMax(&sh->tok_max_pos, lastpos);
  rec_sync<BAR>();
  return sh->tok_min != 0x7fffffff ? sh->tok_min : sh->tok_max_pos;
}


// Chunk search over the chunk weights cw[0..n): W = sum, target = u*W, the first chunk j whose inclusive
// cumulative weight exceeds the target (else the last chunk with positive weight) and the cumulative
// weight before it.  Each thread owns a contiguous run of chunks; a block-wide scan joins the runs.
// Every thread must call it; on return sh->{jstar, base, target, W} are set and visible to all.
// With fixed_target >= 0 (sharded vocabulary) the target and the total are given instead: the search then runs
// for that absolute target over this shard's chunks, and sh->W is set to W_given.
template <int BAR>
__device__ __forceinline__ void find_chunk(const double* cw, int n, double u, PickShared* sh, int tid,
                                           double fixed_target = -1.0, double W_given = 0.0) {
  const int per = (n + kRecThreads - 1) / kRecThreads;
  const int j0 = min(tid * per, n), j1 = min(j0 + per, n);
  double local = 0.0;
  for (int j = j0; j < j1; ++j) local += cw[j];
  if (tid == 0) { sh->jstar = 0x7fffffff; sh->jlast = -1; }
  const double excl = block_excl_scan<BAR>(local, sh->warp_tot, tid);  // two barriers inside
  if (tid == kRecThreads - 1) {
    sh->W = fixed_target >= 0.0 ? W_given : excl + local;
    sh->target = fixed_target >= 0.0 ? fixed_target : u * (excl + local);
  }
  rec_sync<BAR>();
  const double target = sh->target;
  double c = excl;
  int mine = 0x7fffffff, lastpos = -1;
  for (int j = j0; j < j1; ++j) {
    if (cw[j] > 0.0) lastpos = j;
    if (mine == 0x7fffffff && c + cw[j] > target) mine = j;
    c += cw[j];
  }
  if (mine != 0x7fffffff) atomicMin(&sh->jstar, mine);
  if (lastpos >= 0) atomicMax(&sh->jlast, lastpos);
  rec_sync<BAR>();
  const int jstar = sh->jstar != 0x7fffffff ? sh->jstar : max(sh->jlast, 0);
  // the owner of jstar publishes the cumulative weight before it
  if (jstar >= j0 && jstar < j1) {
    double base = excl;
    for (int j = j0; j < jstar; ++j) base += cw[j];
    sh->base = base;
  }
  rec_sync<BAR>();
  if (tid == 0) sh->jstar = jstar;
  rec_sync<BAR>();
}

struct ReqState {
  int n, len, status;
  bool sample;  // a token is to be drawn from row n
};

__device__ __forceinline__ ReqState request_state(const RoundParams& p, int b) {
  ReqState s;
  s.n = p.accept_len[b];
  s.status = p.status_ws[b];
  s.len = p.draft_len[b];
  if (s.len < 0 || s.len > p.K) s.len = 0;
  const bool bad = (s.status & (SPECSTEER_REQ_BAD_PARAM | SPECSTEER_REQ_NONFINITE)) != 0;
  s.sample = !bad && (s.n < s.len || (p.flags & SPECSTEER_FLAG_BONUS));
  return s;
}

// OWN_LSE: the two-phase round.  Row accept_len has just been streamed on its own and has records but no
// normalisers yet: warp 0 combines them first (all four, as the epilogue would have), stores them, and flags a
// non-finite row, after which nothing is sampled.
// One request, kRecThreads threads (tid = 0 .. kRecThreads - 1), cw: [n_chunks] doubles of shared memory, sh and
// lse_fin ([2] doubles) shared memory of the group.  Every thread of the group must call it.
template <typename T, int TILE, bool OWN_LSE, int BAR>
__device__ __forceinline__ void recover_steer_request(const RoundParams& p, int b, int tid, double* cw, PickShared& sh,
                                                      double* lse_fin) {
  constexpr int kPerThread = TILE / kRecThreads;  // consecutive vocabulary entries per thread
  constexpr int kTile = TILE;
  const int K = p.K, K1 = K + 1;
  const ReqState st = request_state(p, b);

  if (p.out_tokens)
    for (int t = tid; t <= K; t += kRecThreads)
      p.out_tokens[(long long)b * K1 + t] = (t < st.n) ? p.draft_tokens[(long long)b * K + t] : -1;
  if (!st.sample) {
    if (tid == 0) {
      if (p.rec_token) p.rec_token[b] = -1;
      if (p.rec_logprob) p.rec_logprob[b] = __int_as_float(0x7fc00000);
      if (p.n_out) p.n_out[b] = st.n;
    }
    return;
  }
  const long long row = (long long)b * K1 + st.n;
  const float* rec = p.part + row * p.n_chunks * 8;
  if (OWN_LSE) {
    double& s_lse = lse_fin[0];
    double& s_fin = lse_fin[1];
    if (tid < 32) {
      float M[4];
      double S[4];
      row_sums_from_records(p, rec, tid, M, S);
      const double lg = log2_pos(tid == 0 ? S[0] : (tid == 1 ? S[1] : (tid == 2 ? S[2] : S[3])));
      bool fin = true;
      float lse[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const double v = (double)M[q] + __shfl_sync(kFullMask, lg, q);
        fin = fin && isfinite(v);
        lse[q] = (float)v;
      }
      if (tid == 0) {
        *reinterpret_cast<float4*>(p.lse2 + row * 4) = make_float4(lse[0], lse[1], lse[2], lse[3]);
        s_lse = (double)lse[Q_R];
        s_fin = fin ? 1.0 : 0.0;
        if (!fin) {
          p.status_ws[b] = st.status | SPECSTEER_REQ_NONFINITE;
          if (p.req_status) p.req_status[b] = st.status | SPECSTEER_REQ_NONFINITE;
          if (p.rec_token) p.rec_token[b] = -1;
          if (p.rec_logprob) p.rec_logprob[b] = __int_as_float(0x7fc00000);
          if (p.n_out) p.n_out[b] = st.n;
        }
      }
    }
    rec_sync<BAR>();
    if (s_fin == 0.0) return;
  }
  const double lseR = OWN_LSE ? (double)__ldcg(p.lse2 + row * 4 + Q_R) : (double)p.lse2[row * 4 + Q_R];
  for (int j = tid; j < p.n_chunks; j += kRecThreads) {
    const float2 ms = __ldcg(reinterpret_cast<const float2*>(rec + j * 8 + 6));   // records may come from other SMs
    const float m = ms.x, s = ms.y;
    cw[j] = (m == kNegInf) ? 0.0 : (double)s * exp2((double)m - lseR);
  }
  if (tid == 0) { sh.tok_min = 0x7fffffff; sh.tok_max_pos = -1; }
  if (p.n_shards > 0 && tid == 0) {
    // every rank holds every shard's partial of this row, so all of them place the target identically, without
    // talking: shard weights in shard order, the target u*W, the first shard whose cumulative weight exceeds it
    double Wg[32], W = 0.0;
    for (int g = 0; g < p.n_shards; ++g) {
      const ShardPartial& sp = p.shard_parts[((long long)g * p.B + b) * K1 + st.n];
      Wg[g] = (sp.m[Q_R] == kNegInf) ? 0.0 : sp.s[Q_R] * exp2((double)sp.m[Q_R] - lseR);
      W += Wg[g];
    }
    const double target = (double)p.u_recover[b] * W;
    double c = 0.0, base = 0.0, base_last = 0.0;
    int owner = -1, last = -1;
    for (int g = 0; g < p.n_shards; ++g) {
      if (Wg[g] > 0.0) { last = g; base_last = c; }
      if (c + Wg[g] > target) { owner = g; base = c; break; }
      c += Wg[g];
    }
    if (owner < 0) { owner = last; base = base_last; }
    sh.plan_owner = (W > 0.0 && W == W) ? owner : -1;
    sh.plan_target = target - base;
    sh.plan_W = W;
  }
  rec_sync<BAR>();
  if (p.n_shards > 0) {
    if (sh.plan_owner != p.shard_rank) {   // another shard (or nobody) samples: leave values a MAX-reduce ignores
      if (tid == 0) {
        if (p.rec_token) p.rec_token[b] = -1;
        if (p.rec_logprob) p.rec_logprob[b] = sh.plan_owner < 0 ? __int_as_float(0x7fc00000) : kNegInf;
        if (p.n_out) p.n_out[b] = st.n;
      }
      return;
    }
    find_chunk<BAR>(cw, p.n_chunks, 0.0, &sh, tid, fmax(sh.plan_target, 0.0), sh.plan_W);
  } else {
    find_chunk<BAR>(cw, p.n_chunks, (double)p.u_recover[b], &sh, tid);
  }

  const T* hl = reinterpret_cast<const T*>(p.h_llm);
  const T* hp = reinterpret_cast<const T*>(p.h_plus);
  const T* hm = reinterpret_cast<const T*>(p.h_minus);
  const double beta = (double)p.beta[b];
  const double cd = (double)(kLog2e / p.temperature[b]);
  const long long off = (long long)b * p.ld_req + (long long)st.n * p.ld_row;
  const int v0 = sh.jstar * kTile + tid * kPerThread;
  double w[kPerThread], y2[kPerThread];
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    const int v = v0 + i;
    w[i] = 0.0; y2[i] = 0.0;
    if (v < p.V) {
      const double l = (double)load_logit<T>(hl, off + v), pp = (double)load_logit<T>(hp, off + v),
                   m = (double)load_logit<T>(hm, off + v);
      y2[i] = (l + beta * (pp - m)) * cd - lseR;  // log2 of Softmax(h_rec)(v)
      w[i] = exp2(y2[i]);
    }
  }
  const int tok = pick_in_chunk<kPerThread, BAR>(w, v0, &sh, tid);
  if (tok >= v0 && tok < v0 + kPerThread) {
    if (p.rec_token) p.rec_token[b] = tok + p.vocab_offset;
    if (p.rec_logprob) p.rec_logprob[b] = (float)(y2[tok - v0] * 0.6931471805599453 - log(sh.W));
    if (p.out_tokens) p.out_tokens[(long long)b * K1 + st.n] = tok + p.vocab_offset;
    if (p.n_out) p.n_out[b] = st.n + 1;
  }
  if (tok < 0 && tid == 0) {  // no positive weight anywhere in the chunk: nothing can be sampled
    if (p.rec_token) p.rec_token[b] = -1;
    if (p.rec_logprob) p.rec_logprob[b] = __int_as_float(0x7fc00000);
    if (p.n_out) p.n_out[b] = st.n;
  }
}

}  // namespace specsteer
