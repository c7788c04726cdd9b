// Top-k split recovery (the paper's deployment appendix, "Minimal Downlink", case "If rejected"):
// the cloud keeps the k largest entries of h_cloud = h_LLM - beta * h_SLM- on the row of the first rejection,
// the edge adds beta * h_SLM+ on those entries and resamples among them.
//
// cloud_topk_kernel: one CTA per request streams the two rows once (128-bit loads).  Every warp keeps the 32
// best entries of its share as one sorted 64-bit key per lane (value in an order-preserving encoding, then the
// complemented token id, so that "larger key" means "higher value, then lower id"); an entry is compared with
// the warp's 32nd value and only the rare better ones go through a ballot-and-shift insertion.  Warp 0 then
// merges the sixteen lists.  edge_resample_kernel: one warp per request.
#include "common.cuh"
#include "internal.h"
#include "specsteer.h"

namespace specsteer {

constexpr int kTopThreads = 512;
constexpr int kTopWarps = kTopThreads / 32;


// Insert `nk` into the warp's descending list (one key per lane, 0 = empty slot) if it beats the last entry.
__device__ __forceinline__ void warp_insert(u64& mykey, u64 nk, int lane) {
  const int pos = __popc(__ballot_sync(kFullMask, mykey > nk));
  const u64 up = __shfl_up_sync(kFullMask, mykey, 1);
  if (pos < 32) {
    if (lane > pos) mykey = up;
    else if (lane == pos) mykey = nk;
  }
}

__device__ __forceinline__ u64 umax64(u64 a, u64 b) { return a > b ? a : b; }
__device__ __forceinline__ u64 umin64(u64 a, u64 b) { return a < b ? a : b; }

// Sort a bitonic sequence held one key per lane into descending order (five compare-exchange stages).
__device__ __forceinline__ u64 bitonic_merge_desc(u64 x, int lane) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const u64 y = __shfl_xor_sync(kFullMask, x, o);
    x = (lane & o) ? umin64(x, y) : umax64(x, y);
  }
  return x;
}
// Sort 32 arbitrary keys, one per lane, into descending order.
__device__ __forceinline__ u64 bitonic_sort_desc(u64 x, int lane) {
#pragma unroll
  for (int sz = 2; sz <= 32; sz <<= 1) {
    const bool up = (lane & sz) != 0 && sz < 32;   // direction of this lane's block: alternate, final pass descending
#pragma unroll
    for (int o = sz >> 1; o > 0; o >>= 1) {
      const u64 y = __shfl_xor_sync(kFullMask, x, o);
      const bool take_min = ((lane & o) != 0) != up;
      x = take_min ? umin64(x, y) : umax64(x, y);
    }
  }
  return x;
}
// The 32 largest of two descending lists: `other_rev` is the second list read back to front.
__device__ __forceinline__ u64 merge_top32(u64 mine, u64 other_rev, int lane) {
  return bitonic_merge_desc(umax64(mine, other_rev), lane);
}

struct TopState {
  u64 key;      // this lane's list entry
  float tau;    // value of the 32nd entry, -inf while the list is not full
};

// The threshold only ever rises: it may already sit above the list's own 32nd value (CTA-wide bound).
__device__ __forceinline__ void refresh_tau_floor(TopState& st) {
  const u64 last = __shfl_sync(kFullMask, st.key, 31);
  if (last) st.tau = fmaxf(st.tau, order_val((uint32_t)(last >> 32)));
}
__device__ __forceinline__ void refresh_tau(TopState& st) { refresh_tau_floor(st); }

// One candidate value per lane (NaN = none): those not below the warp's threshold are inserted one by one.
__device__ __forceinline__ void offer(TopState& st, float h, int idx, int lane) {
  unsigned cand = __ballot_sync(kFullMask, h >= st.tau);
  if (!cand) return;
  const u64 mine = entry_key(h, idx);
  while (cand) {
    const int src = __ffs(cand) - 1;
    cand &= cand - 1;
    warp_insert(st.key, __shfl_sync(kFullMask, mine, src), lane);
  }
  refresh_tau(st);
}

// h_cloud of one entry: one fused multiply-add in float32; -0 becomes +0 so that equal values have equal keys
__device__ __forceinline__ float h_cloud(float l, float m, float nbeta) { return fmaf(nbeta, m, l) + 0.f; }

template <typename T> struct Vec;
template <> struct Vec<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ void unpack(const uint4& v, float (&x)[4]) {
    x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
  }
};
template <> struct Vec<uint16_t> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void unpack(const uint4& v, float (&x)[8]) {
    x[0] = bf16lo(v.x); x[1] = bf16hi(v.x); x[2] = bf16lo(v.y); x[3] = bf16hi(v.y);
    x[4] = bf16lo(v.z); x[5] = bf16hi(v.z); x[6] = bf16lo(v.w); x[7] = bf16hi(v.w);
  }
};
// the four 16-byte vectors a lane holds for one step: two of h_LLM, two of h_SLM-
struct StepRegs { uint4 l0, m0, l1, m1; };

struct TopReq {
  int n;        // row to recover from
  bool sample;  // a token is to be drawn from it
};
__device__ __forceinline__ TopReq top_request(const RoundParams& p, int b) {
  TopReq r;
  r.n = p.accept_len[b];
  int len = p.draft_len[b];
  if (len < 0 || len > p.K) len = 0;
  const int status = p.status_ws[b];
  const bool bad = (status & (SPECSTEER_REQ_BAD_PARAM | SPECSTEER_REQ_NONFINITE)) != 0;
  r.sample = !bad && (r.n < len || (p.flags & SPECSTEER_FLAG_BONUS));
  return r;
}

// The 32 largest keys of all sixteen warps' lists, left sorted in lists[0][*].  Every thread of the CTA calls it.
__device__ __forceinline__ void cta_merge(u64 (*lists)[32], u64 mykey, int warp, int lane) {
  lists[warp][lane] = mykey;
  __syncthreads();
  u64 cur = mykey;
#pragma unroll
  for (int stride = 1; stride < kTopWarps; stride <<= 1) {
    if ((warp & (2 * stride - 1)) == 0) {
      cur = merge_top32(cur, lists[warp + stride][31 - lane], lane);
      lists[warp][lane] = cur;
    }
    __syncthreads();
  }
}

// Grid (B, S): CTA (b, s) selects over the s-th slice of the row.  With S > 1 the CTAs of a request leave their
// lists in `lists_ws` [B][S][32] and the one that finishes last (a counter per request in `count_ws`, which it
// puts back to zero) merges them; nobody waits for anybody.
template <typename T>
__global__ void __launch_bounds__(kTopThreads, 2) cloud_topk_kernel(const RoundParams p, int k, int* topk_idx,
                                                                  float* topk_val, u64* lists_ws, int* count_ws) {
  constexpr int NE = Vec<T>::N;
  __shared__ u64 lists[kTopWarps][32];
  __shared__ int is_last;
  const int b = blockIdx.x, split = blockIdx.y, S = gridDim.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  pdl_wait();
  const TopReq rq = top_request(p, b);
  if (!rq.sample) {
    if (split == 0 && tid < k) { topk_idx[(long long)b * k + tid] = -1; topk_val[(long long)b * k + tid] = kNegInf; }
    return;
  }
  const long long off = (long long)b * p.ld_req + (long long)rq.n * p.ld_row;
  const T* hl = reinterpret_cast<const T*>(p.h_llm) + off;
  const T* hm = reinterpret_cast<const T*>(p.h_minus) + off;
  const float nbeta = -p.beta[b];
  const float qnan = __int_as_float(0x7fc00000);
  TopState st;
  st.key = 0ull;
  st.tau = kNegInf;

  const bool aligned = ((reinterpret_cast<uintptr_t>(hl) | reinterpret_cast<uintptr_t>(hm)) & 15u) == 0;
  const int nvec = aligned ? p.V / NE : 0;
  const int per = (nvec + S - 1) / S;
  const int vbeg = min(split * per, nvec), vend = min(vbeg + per, nvec);
  // main part: warp w takes vectors vbeg + [w*32, w*32+32) + j*512, two per stream and lane per step; the loads
  // of the next step are issued before this step's entries are looked at
  constexpr int kStep = 2 * kTopThreads;   // vectors the CTA consumes per step
  // a lane without a vector holds NaN patterns: they never pass a comparison, so the loop needs no range tests
  const uint32_t nanw = sizeof(T) == 4 ? 0x7fc00000u : 0x7fc07fc0u;
  const uint4 nan4 = make_uint4(nanw, nanw, nanw, nanw);
  auto fetch = [&](int bs, StepRegs& r) {
    const int v0 = bs + lane, v1 = v0 + kTopThreads;
    if (v0 < vend) {
      r.l0 = __ldcs(reinterpret_cast<const uint4*>(hl + (size_t)v0 * NE));
      r.m0 = __ldcs(reinterpret_cast<const uint4*>(hm + (size_t)v0 * NE));
    } else {
      r.l0 = nan4; r.m0 = nan4;
    }
    if (v1 < vend) {
      r.l1 = __ldcs(reinterpret_cast<const uint4*>(hl + (size_t)v1 * NE));
      r.m1 = __ldcs(reinterpret_cast<const uint4*>(hm + (size_t)v1 * NE));
    } else {
      r.l1 = nan4; r.m1 = nan4;
    }
  };
  // all warps run the same number of steps (a warp without vectors offers nothing) so that they can meet at the
  // steps 1, 7, 31, ... to raise the common threshold to the 32nd value of everything the CTA has seen
  const int steps = (vend - vbeg + kStep - 1) / kStep;
  int next_sync = 1;
  // one step: the loads run two steps ahead (`refill`), the arithmetic looks at `use`.  Hot part: one fused
  // multiply-add and one compare per entry; only a warp in which some entry reaches the threshold goes on.
  auto step = [&](int it, const StepRegs& use, StepRegs& refill) {
    const int bs = vbeg + warp * 32 + it * kStep;
    fetch(bs + 2 * kStep, refill);
    float l0[NE], m0[NE], l1[NE], m1[NE];
    Vec<T>::unpack(use.l0, l0); Vec<T>::unpack(use.m0, m0);
    Vec<T>::unpack(use.l1, l1); Vec<T>::unpack(use.m1, m1);
    bool hit = false;
#pragma unroll
    for (int e = 0; e < NE; ++e) {
      hit |= fmaf(nbeta, m0[e], l0[e]) >= st.tau;
      hit |= fmaf(nbeta, m1[e], l1[e]) >= st.tau;
    }
    if (__any_sync(kFullMask, hit)) {
      const int v0 = bs + lane, v1 = v0 + kTopThreads;
#pragma unroll
      for (int e = 0; e < NE; ++e) offer(st, h_cloud(l0[e], m0[e], nbeta), v0 * NE + e, lane);
#pragma unroll
      for (int e = 0; e < NE; ++e) offer(st, h_cloud(l1[e], m1[e], nbeta), v1 * NE + e, lane);
    }
    if (it == next_sync && it + 1 < steps) {
      next_sync = 4 * next_sync + 3;
      cta_merge(lists, st.key, warp, lane);
      const u64 last = lists[0][31];
      if (last) st.tau = fmaxf(st.tau, order_val((uint32_t)(last >> 32)));
      __syncthreads();   // lists[] is reused by the next merge
    }
  };
  StepRegs ra, rb, rc;
  fetch(vbeg + warp * 32, ra);
  fetch(vbeg + warp * 32 + kStep, rb);
  {
    // Bootstrap of the threshold: every lane's maximum over its first entries is an entry of the row, so the
    // 32nd largest of the CTA's 512 lane maxima has at least 32 entries at or above it.  Step 0 then starts with a
    // threshold almost as tight as the exact one and only a few dozen entries per CTA take the insertion path.
    float l0[NE], m0[NE], l1[NE], m1[NE];
    Vec<T>::unpack(ra.l0, l0); Vec<T>::unpack(ra.m0, m0);
    Vec<T>::unpack(ra.l1, l1); Vec<T>::unpack(ra.m1, m1);
    float lm = kNegInf;
#pragma unroll
    for (int e = 0; e < NE; ++e) lm = fmaxf(lm, fmaxf(h_cloud(l0[e], m0[e], nbeta), h_cloud(l1[e], m1[e], nbeta)));
    const u64 mk = bitonic_sort_desc((u64)order_key(lm) << 32, lane);
    cta_merge(lists, mk, warp, lane);
    st.tau = order_val((uint32_t)(lists[0][31] >> 32));
    __syncthreads();
  }
#pragma unroll 1
  for (int it = 0; it < steps; ++it) {
    step(it, ra, rc);
    ra = rb;   // rotate: sixteen register moves per step keep the loop body single (it is large)
    rb = rc;
  }
  // what the vectors did not cover (the tail, or the whole row when it is not 16-byte aligned): last slice
  if (split == S - 1) {
    for (int bs = nvec * NE + warp * 32; bs < p.V; bs += kTopThreads) {
      const int v = bs + lane;
      const float h = v < p.V ? h_cloud(load_logit<T>(hl, v), load_logit<T>(hm, v), nbeta) : qnan;
      offer(st, h, v, lane);
    }
  }
  cta_merge(lists, st.key, warp, lane);
  if (warp != 0) return;
  st.key = lists[0][lane];
  if (S > 1) {
    u64* mine = lists_ws + ((size_t)b * S + split) * 32;
    mine[lane] = st.key;
    __threadfence();
    __syncwarp();
    if (lane == 0) is_last = (atomicAdd(count_ws + b, 1) == S - 1) ? 1 : 0;
    __syncwarp();
    if (!is_last) return;
    __threadfence();
    for (int s2 = 0; s2 < S; ++s2) {
      if (s2 == split) continue;
      st.key = merge_top32(st.key, __ldcg(lists_ws + ((size_t)b * S + s2) * 32 + (31 - lane)), lane);
    }
    if (lane == 0) count_ws[b] = 0;
  }
  if (lane < k) {
    const bool have = st.key != 0ull;
    topk_idx[(long long)b * k + lane] = have ? (int)(0xffffffffu - (uint32_t)(st.key & 0xffffffffull)) : -1;
    topk_val[(long long)b * k + lane] = have ? order_val((uint32_t)(st.key >> 32)) : kNegInf;
  }
}

template <typename T>
__global__ void __launch_bounds__(32) edge_resample_kernel(const RoundParams p, int k, const int* topk_idx,
                                                           const float* topk_val) {
  const int b = blockIdx.x, lane = threadIdx.x;
  const int K = p.K, K1 = K + 1;
  pdl_wait();
  const TopReq rq = top_request(p, b);
  if (p.out_tokens)
    for (int t = lane; t <= K; t += 32)
      p.out_tokens[(long long)b * K1 + t] = (t < rq.n) ? p.draft_tokens[(long long)b * K + t] : -1;
  int token = -1;
  double logprob = __longlong_as_double(0x7ff8000000000000ll);
  if (rq.sample) {
    const T* hp = reinterpret_cast<const T*>(p.h_plus) + (long long)b * p.ld_req + (long long)rq.n * p.ld_row;
    const double beta = (double)p.beta[b], Tm = (double)p.temperature[b];
    const int idx = lane < k ? topk_idx[(long long)b * k + lane] : -1;
    const bool have = idx >= 0 && idx < p.V;
    const double ninf = -__longlong_as_double(0x7ff0000000000000ll);
    // recovery logit of Eq. 8 on a kept entry, tempered
    const double hr = have ? ((double)topk_val[(long long)b * k + lane] + beta * (double)load_logit<T>(hp, idx)) / Tm : ninf;
    double mx = hr;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(kFullMask, mx, o));
    const bool any_nan = __any_sync(kFullMask, hr != hr);
    const double w = (hr == ninf) ? 0.0 : exp(hr - mx);
    double cum = w;   // inclusive scan in list order
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double u = __shfl_up_sync(kFullMask, cum, o);
      if (lane >= o) cum += u;
    }
    const double W = __shfl_sync(kFullMask, cum, 31);
    if (!any_nan && W > 0.0 && isfinite(W)) {
      const double target = (double)p.u_recover[b] * W;
      const unsigned over = __ballot_sync(kFullMask, cum > target);
      const unsigned pos = __ballot_sync(kFullMask, w > 0.0);
      const int pick = over ? __ffs(over) - 1 : 31 - __clz(pos);
      token = __shfl_sync(kFullMask, idx, pick);
      logprob = log(__shfl_sync(kFullMask, w, pick) / W);
    }
  }
  if (lane == 0) {
    if (p.rec_token) p.rec_token[b] = token;
    if (p.rec_logprob) p.rec_logprob[b] = (float)logprob;
    if (token >= 0 && p.out_tokens) p.out_tokens[(long long)b * K1 + rq.n] = token;
    if (p.n_out) p.n_out[b] = rq.n + (token >= 0 ? 1 : 0);
  }
}

cudaError_t launch_cloud_topk(const RoundParams& p, int dtype, int k, int* topk_idx, float* topk_val,
                              void* lists_ws, int* count_ws, int sm_count, cudaStream_t s) {
  // Two CTAs fit on an SM.  Few requests: split each row over as many CTAs as still fit at once (one wave), but
  // keep at least 4096 vectors (64 KB per stream) per slice.  Otherwise one CTA per row: splitting further only
  // multiplies the fixed work per CTA (measured on 512 rows of 256000 bf16 entries: 98 us unsplit, 135 us split in 4).
  const int nvec = p.V / (dtype == SPECSTEER_F32 ? 4 : 8);
  const int slots = 2 * sm_count;
  int s_cap = nvec / 4096 > 1 ? nvec / 4096 : 1;
  if (s_cap > kTopkMaxSplit) s_cap = kTopkMaxSplit;
  int S = 1;
  if (p.B * 2 <= slots) S = slots / p.B;
  if (S > s_cap) S = s_cap;
  if (S < 1 || !lists_ws || !count_ws) S = 1;
  const dim3 grid(p.B, S);
  if (dtype == SPECSTEER_F32)
    cloud_topk_kernel<float><<<grid, kTopThreads, 0, s>>>(p, k, topk_idx, topk_val, (u64*)lists_ws, count_ws);
  else
    cloud_topk_kernel<uint16_t><<<grid, kTopThreads, 0, s>>>(p, k, topk_idx, topk_val, (u64*)lists_ws, count_ws);
  return cudaGetLastError();
}

cudaError_t launch_edge_resample(const RoundParams& p, int dtype, int k, const int* topk_idx, const float* topk_val,
                                 cudaStream_t s) {
  if (dtype == SPECSTEER_F32) edge_resample_kernel<float><<<p.B, 32, 0, s>>>(p, k, topk_idx, topk_val);
  else edge_resample_kernel<uint16_t><<<p.B, 32, 0, s>>>(p, k, topk_idx, topk_val);
  return cudaGetLastError();
}

}  // namespace specsteer
