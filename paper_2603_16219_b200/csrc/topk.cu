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

typedef unsigned long long u64;

__device__ __forceinline__ uint32_t order_key(float h) {
  const uint32_t b = __float_as_uint(h);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float order_val(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
__device__ __forceinline__ u64 entry_key(float h, int idx) {
  return ((u64)order_key(h) << 32) | (u64)(0xffffffffu - (uint32_t)idx);
}

// Insert `nk` into the warp's descending list (one key per lane, 0 = empty slot) if it beats the last entry.
__device__ __forceinline__ void warp_insert(u64& mykey, u64 nk, int lane) {
  const int pos = __popc(__ballot_sync(kFullMask, mykey > nk));
  const u64 up = __shfl_up_sync(kFullMask, mykey, 1);
  if (pos < 32) {
    if (lane > pos) mykey = up;
    else if (lane == pos) mykey = nk;
  }
}

struct TopState {
  u64 key;      // this lane's list entry
  float tau;    // value of the 32nd entry, -inf while the list is not full
};

__device__ __forceinline__ void refresh_tau(TopState& st) {
  const u64 last = __shfl_sync(kFullMask, st.key, 31);
  st.tau = last ? order_val((uint32_t)(last >> 32)) : kNegInf;
}

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
  static __device__ __forceinline__ void load(const float* p, float (&x)[4]) {
    const float4 v = __ldcs(reinterpret_cast<const float4*>(p));
    x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
  }
};
template <> struct Vec<uint16_t> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void load(const uint16_t* p, float (&x)[8]) {
    const uint4 v = __ldcs(reinterpret_cast<const uint4*>(p));
    x[0] = bf16lo(v.x); x[1] = bf16hi(v.x); x[2] = bf16lo(v.y); x[3] = bf16hi(v.y);
    x[4] = bf16lo(v.z); x[5] = bf16hi(v.z); x[6] = bf16lo(v.w); x[7] = bf16hi(v.w);
  }
};

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

template <typename T>
__global__ void __launch_bounds__(kTopThreads) cloud_topk_kernel(const RoundParams p, int k, int* topk_idx,
                                                                  float* topk_val) {
  constexpr int NE = Vec<T>::N;
  __shared__ u64 lists[kTopWarps][32];
  const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  pdl_wait();
  const TopReq rq = top_request(p, b);
  if (!rq.sample) {
    if (tid < k) { topk_idx[(long long)b * k + tid] = -1; topk_val[(long long)b * k + tid] = kNegInf; }
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
  // main part: warp w takes vectors [w*32, w*32+32) + j*512; two vectors per stream in flight per lane
  for (int base = warp * 32; base < nvec; base += 2 * kTopThreads) {
    const int v0 = base + lane, v1 = v0 + kTopThreads;
    float l0[NE], m0[NE], l1[NE], m1[NE];
    const bool ok0 = v0 < nvec, ok1 = v1 < nvec;
    if (ok0) { Vec<T>::load(hl + (size_t)v0 * NE, l0); Vec<T>::load(hm + (size_t)v0 * NE, m0); }
    if (ok1) { Vec<T>::load(hl + (size_t)v1 * NE, l1); Vec<T>::load(hm + (size_t)v1 * NE, m1); }
    float h0[NE], h1[NE];
    float best = kNegInf;
#pragma unroll
    for (int e = 0; e < NE; ++e) {
      h0[e] = ok0 ? h_cloud(l0[e], m0[e], nbeta) : qnan;
      h1[e] = ok1 ? h_cloud(l1[e], m1[e], nbeta) : qnan;
      best = fmaxf(best, fmaxf(h0[e], h1[e]));   // fmaxf drops NaN
    }
    if (!__any_sync(kFullMask, best >= st.tau)) continue;
#pragma unroll
    for (int e = 0; e < NE; ++e) offer(st, h0[e], v0 * NE + e, lane);
#pragma unroll
    for (int e = 0; e < NE; ++e) offer(st, h1[e], v1 * NE + e, lane);
  }
  // what the vectors did not cover (the tail, or the whole row when it is not 16-byte aligned)
  for (int base = nvec * NE + warp * 32; base < p.V; base += kTopThreads) {
    const int v = base + lane;
    const float h = v < p.V ? h_cloud(load_logit<T>(hl, v), load_logit<T>(hm, v), nbeta) : qnan;
    offer(st, h, v, lane);
  }
  lists[warp][lane] = st.key;
  __syncthreads();
  if (warp != 0) return;
  for (int w = 1; w < kTopWarps; ++w) {
    const u64 nk = lists[w][lane];
    const u64 last = __shfl_sync(kFullMask, st.key, 31);
    unsigned cand = __ballot_sync(kFullMask, nk > last);   // an empty slot (0) never beats anything
    while (cand) {
      const int src = __ffs(cand) - 1;
      cand &= cand - 1;
      warp_insert(st.key, __shfl_sync(kFullMask, nk, src), lane);
    }
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

cudaError_t launch_cloud_topk(const RoundParams& p, int dtype, int k, int* topk_idx, float* topk_val, cudaStream_t s) {
  if (dtype == SPECSTEER_F32) cloud_topk_kernel<float><<<p.B, kTopThreads, 0, s>>>(p, k, topk_idx, topk_val);
  else cloud_topk_kernel<uint16_t><<<p.B, kTopThreads, 0, s>>>(p, k, topk_idx, topk_val);
  return cudaGetLastError();
}

cudaError_t launch_edge_resample(const RoundParams& p, int dtype, int k, const int* topk_idx, const float* topk_val,
                                 cudaStream_t s) {
  if (dtype == SPECSTEER_F32) edge_resample_kernel<float><<<p.B, 32, 0, s>>>(p, k, topk_idx, topk_val);
  else edge_resample_kernel<uint16_t><<<p.B, 32, 0, s>>>(p, k, topk_idx, topk_val);
  return cudaGetLastError();
}

}  // namespace specsteer
