// Recovery kernels (Algorithm 1 Phase 3; Eq. 8): one CTA per request samples one token from the row of
// the first rejection by inverse CDF in vocabulary order.  The STEER kernel finds the chunk from the
// per-chunk partial sums the verification pass left in the workspace and re-reads only that chunk.
// The RESIDUAL kernel makes two extra passes over the row in double precision.
#include "common.cuh"
#include "internal.h"
#include "records.cuh"
#include "recover_steer.cuh"
#include "specsteer.h"

namespace specsteer {

// The stand-alone STEER kernel: one CTA per request (see recover_steer.cuh).
template <typename T, int TILE, bool OWN_LSE>
__global__ void __launch_bounds__(kRecThreads) recover_steer_kernel(const RoundParams p) {
  extern __shared__ double cw[];  // [n_chunks] chunk weights
  __shared__ PickShared sh;
  __shared__ double lse_fin[2];
  pdl_wait();  // launched behind the epilogue kernel: nothing is read before that one has finished
  recover_steer_request<T, TILE, OWN_LSE, 0>(p, blockIdx.x, threadIdx.x, cw, sh, lse_fin);
}

// RESIDUAL: w(v) = max(0, Softmax(h_rec)(v) - P_SLM+(v)) on the rejection row, all in double.
// Runs after the STEER kernel and overrides its result unless the residual has no mass.
template <typename T, int TILE>
__global__ void __launch_bounds__(kRecThreads) recover_residual_kernel(const RoundParams p) {
  constexpr int kPerThread = TILE / kRecThreads;
  constexpr int kTile = TILE;
  extern __shared__ double cw[];  // [n_chunks]
  __shared__ PickShared sh;
  __shared__ double red[2][kRecWarps];
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K1 = p.K + 1;
  const ReqState st = request_state(p, b);
  if (!st.sample || st.n >= st.len) return;  // the bonus row is always STEER

  const T* hl = reinterpret_cast<const T*>(p.h_llm);
  const T* hp = reinterpret_cast<const T*>(p.h_plus);
  const T* hm = reinterpret_cast<const T*>(p.h_minus);
  const double beta = (double)p.beta[b];
  const double cd = (double)(kLog2e / p.temperature[b]);
  const long long off = (long long)b * p.ld_req + (long long)st.n * p.ld_row;
  const long long row = (long long)b * K1 + st.n;
  const double refR = (double)p.lse2[row * 4 + Q_R], refP = (double)p.lse2[row * 4 + Q_P];

  // pass 1: the two normalisers in double, using the single-precision ones as reference exponents
  double sR = 0.0, sP = 0.0;
  for (int v = tid; v < p.V; v += kRecThreads) {
    const double l = (double)load_logit<T>(hl, off + v), pp = (double)load_logit<T>(hp, off + v),
                 m = (double)load_logit<T>(hm, off + v);
    sR += exp2((l + beta * (pp - m)) * cd - refR);
    sP += exp2(pp * cd - refP);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    sR += __shfl_xor_sync(kFullMask, sR, o);
    sP += __shfl_xor_sync(kFullMask, sP, o);
  }
  if (lane == 0) { red[0][warp] = sR; red[1][warp] = sP; }
  if (tid == 0) { sh.tok_min = 0x7fffffff; sh.tok_max_pos = -1; }
  __syncthreads();
  sR = 0.0; sP = 0.0;
  for (int w = 0; w < kRecWarps; ++w) { sR += red[0][w]; sP += red[1][w]; }
  const double lseR = refR + log2(sR), lseP = refP + log2(sP);

  // pass 2: residual mass per chunk, one warp per chunk
  for (int j = warp; j < p.n_chunks; j += kRecWarps) {
    double acc = 0.0;
    const int vend = min(p.V, (j + 1) * kTile);
    for (int v = j * kTile + lane; v < vend; v += 32) {
      const double l = (double)load_logit<T>(hl, off + v), pp = (double)load_logit<T>(hp, off + v),
                   m = (double)load_logit<T>(hm, off + v);
      const double d = exp2((l + beta * (pp - m)) * cd - lseR) - exp2(pp * cd - lseP);
      if (d > 0.0) acc += d;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(kFullMask, acc, o);
    if (lane == 0) cw[j] = acc;
  }
  __syncthreads();
  find_chunk<0>(cw, p.n_chunks, (double)p.u_recover[b], &sh, tid);
  if (!(sh.W > 0.0)) {  // no residual mass: keep the STEER sample already written
    if (tid == 0) {
      p.status_ws[b] = st.status | SPECSTEER_REQ_RESIDUAL_EMPTY;
      if (p.req_status) p.req_status[b] = st.status | SPECSTEER_REQ_RESIDUAL_EMPTY;
    }
    return;
  }
  const int v0 = sh.jstar * kTile + tid * kPerThread;
  double w[kPerThread];
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    const int v = v0 + i;
    w[i] = 0.0;
    if (v < p.V) {
      const double l = (double)load_logit<T>(hl, off + v), pp = (double)load_logit<T>(hp, off + v),
                   m = (double)load_logit<T>(hm, off + v);
      const double d = exp2((l + beta * (pp - m)) * cd - lseR) - exp2(pp * cd - lseP);
      w[i] = d > 0.0 ? d : 0.0;
    }
  }
  const int tok = pick_in_chunk<kPerThread, 0>(w, v0, &sh, tid);
  if (tok >= v0 && tok < v0 + kPerThread) {
    if (p.rec_token) p.rec_token[b] = tok;
    if (p.rec_logprob) p.rec_logprob[b] = (float)log(w[tok - v0] / sh.W);
    if (p.out_tokens) p.out_tokens[(long long)b * K1 + st.n] = tok;
    if (p.n_out) p.n_out[b] = st.n + 1;
  }
}

// ARGMAX (greedy decoding): the token of largest h_rec = fl(h_LLM + beta * fl(h_SLM+ - h_SLM-)) (Eq. 8) on row
// accept_len, the lowest id among equals.  Grid (B, S): S CTAs share a row, each leaves the best key of its part of the
// vocabulary in the workspace, and the last one to finish (a counter per request, left at zero) writes the outputs.
template <typename T> struct Vec8;
template <> struct Vec8<float> {
  static __device__ __forceinline__ void load(const float* p, long long i, float (&x)[8]) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(p + i)), b = __ldcs(reinterpret_cast<const float4*>(p + i + 4));   // read once: streaming loads
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
  }
};
template <> struct Vec8<uint16_t> {
  static __device__ __forceinline__ void load(const uint16_t* p, long long i, float (&x)[8]) {
    const uint4 a = __ldcs(reinterpret_cast<const uint4*>(p + i));
    x[0] = bf16lo(a.x); x[1] = bf16hi(a.x); x[2] = bf16lo(a.y); x[3] = bf16hi(a.y);
    x[4] = bf16lo(a.z); x[5] = bf16hi(a.z); x[6] = bf16lo(a.w); x[7] = bf16hi(a.w);
  }
};

// max that hands a NaN on: the running maxima of the three streams then show a NaN or +inf entry by themselves
__device__ __forceinline__ float fmax_nan(float a, float b) {
  float d;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}

// An online (maximum, sum of 2^(x - maximum)) pair and its merge; empty = (-inf, 0).
struct OnlineLse {
  float m, s;
};
__device__ __forceinline__ OnlineLse lse_merge(OnlineLse a, OnlineLse b) {
  const float m = fmaxf(a.m, b.m);
  OnlineLse r;
  r.m = m;
  r.s = (a.m == kNegInf ? 0.f : a.s * ex2(a.m - m)) + (b.m == kNegInf ? 0.f : b.s * ex2(b.m - m));
  if (a.s != a.s || b.s != b.s) r.s = a.s + b.s;   // a NaN sum stays NaN whatever the maxima are
  return r;
}

// LSE: the row has no normaliser yet (verification read only h_LLM and h_SLM- and not this row's h_SLM+): the pass
// also forms log2 sum 2^(h_rec c) online for rec_logprob, and checks what the streaming pass would have checked -
// a NaN or +inf anywhere in the three streams of the row, or a stream that is -inf throughout, raises REQ_NONFINITE.
template <typename T, bool VEC, bool LSE>
__global__ void __launch_bounds__(kRecThreads) recover_argmax_kernel(const RoundParams p, u64* best_ws, int* count_ws) {
  __shared__ u64 wbest[kRecWarps];
  __shared__ OnlineLse wlse[kRecWarps];
  __shared__ float wmax[kRecWarps][3];
  const int b = blockIdx.x, sp = blockIdx.y, S = gridDim.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K = p.K, K1 = K + 1;
  pdl_wait();
  const ReqState st = request_state(p, b);
  if (sp == 0 && p.out_tokens && !p.greedy_keys)
    for (int t = tid; t <= K; t += kRecThreads)
      p.out_tokens[(long long)b * K1 + t] = (t < st.n) ? p.draft_tokens[(long long)b * K + t] : -1;
  if (!st.sample) {
    if (sp == 0 && tid == 0) {
      if (p.greedy_keys) {
        p.greedy_keys[b] = -1;
      } else {
        if (p.rec_token) p.rec_token[b] = -1;
        if (p.rec_logprob) p.rec_logprob[b] = __int_as_float(0x7fc00000);
        if (p.n_out) p.n_out[b] = st.n;
      }
    }
    return;
  }
  const T* hl = reinterpret_cast<const T*>(p.h_llm);
  const T* hp = reinterpret_cast<const T*>(p.h_plus);
  const T* hm = reinterpret_cast<const T*>(p.h_minus);
  const long long off = (long long)b * p.ld_req + (long long)st.n * p.ld_row;
  const float beta = p.beta[b];
  const float c = kLog2e / p.temperature[b];
  const int per = (((p.V + S - 1) / S) + 7) & ~7;
  const int v0 = sp * per, v1 = min(p.V, v0 + per);
  float best_r = 0.f;   // the thread walks its entries in ascending id order, so "strictly larger" keeps the lowest id
  int best_v = -1;
  OnlineLse acc = {kNegInf, 0.f};
  float mx[3] = {kNegInf, kNegInf, kNegInf};   // largest entry of each stream; NaN once the stream held a NaN
#pragma unroll 2   // two iterations' loads in flight: 16-bit rows otherwise keep too few bytes outstanding per SM
  for (int v = v0 + tid * 8; v < v1; v += kRecThreads * 8) {
    float l[8], q[8], m[8], r[8];
    int n = 8;
    if (VEC && v + 8 <= v1) {
      Vec8<T>::load(hl, off + v, l); Vec8<T>::load(hp, off + v, q); Vec8<T>::load(hm, off + v, m);
    } else {
      n = min(8, v1 - v);
      for (int i = 0; i < 8; ++i) {
        const bool in = i < n;
        l[i] = in ? load_logit<T>(hl, off + v + i) : kNegInf;
        q[i] = in ? load_logit<T>(hp, off + v + i) : 0.f;
        m[i] = in ? load_logit<T>(hm, off + v + i) : 0.f;
      }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      r[i] = fmaf(beta, q[i] - m[i], l[i]);   // Eq. 8
      if (i < n && (best_v < 0 || r[i] > best_r)) { best_r = r[i]; best_v = v + i; }
    }
    if (LSE) {
      float x[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        x[i] = r[i] * c;
        if (i < n) {
          mx[0] = fmax_nan(mx[0], l[i]); mx[1] = fmax_nan(mx[1], q[i]); mx[2] = fmax_nan(mx[2], m[i]);
        } else {
          x[i] = kNegInf;
        }
      }
      const float m8 = max8(x);
      if (m8 > acc.m) {
        acc.s = (acc.m == kNegInf) ? 0.f : acc.s * ex2(acc.m - m8);
        acc.m = m8;
      }
      if (acc.m > kNegInf) {
#pragma unroll
        for (int i = 0; i < 8; ++i) acc.s += ex2(x[i] - acc.m);
      }
    }
  }
  u64 best = best_v >= 0 ? entry_key(best_r, best_v) : 0;   // 0 is below every key of a real entry
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const u64 other = __shfl_xor_sync(kFullMask, best, o);
    best = other > best ? other : best;
    if (LSE) {
      OnlineLse t;
      t.m = __shfl_xor_sync(kFullMask, acc.m, o);
      t.s = __shfl_xor_sync(kFullMask, acc.s, o);
      acc = lse_merge(acc, t);
#pragma unroll
      for (int q = 0; q < 3; ++q) mx[q] = fmax_nan(mx[q], __shfl_xor_sync(kFullMask, mx[q], o));
    }
  }
  if (lane == 0) {
    wbest[warp] = best;
    if (LSE) { wlse[warp] = acc; wmax[warp][0] = mx[0]; wmax[warp][1] = mx[1]; wmax[warp][2] = mx[2]; }
  }
  __syncthreads();
  if (tid != 0) return;
  for (int w = 1; w < kRecWarps; ++w) {
    best = wbest[w] > best ? wbest[w] : best;
    if (LSE) {
      acc = lse_merge(acc, wlse[w]);
      for (int q = 0; q < 3; ++q) mx[q] = fmax_nan(mx[q], wmax[w][q]);
    }
  }
  // workspace of the request: [0, 16) keys, [16, 32) {maximum, sum}, [32, 48) {max h_LLM, max h_SLM+}, [48, 64) max h_SLM-
  u64* mine = best_ws + (long long)b * kTopkMaxSplit * 32;
  auto pack = [](float a, float b2) { return ((u64)__float_as_uint(a) << 32) | (u64)__float_as_uint(b2); };
  if (S > 1) {
    mine[sp] = best;
    if (LSE) { mine[16 + sp] = pack(acc.m, acc.s); mine[32 + sp] = pack(mx[0], mx[1]); mine[48 + sp] = pack(mx[2], 0.f); }
    __threadfence();
    if (atomicAdd(&count_ws[b], 1) != S - 1) return;
    __threadfence();
    // merge all parts in index order, this CTA's own included, so that the sums do not depend on who finished last
    best = 0;
    acc.m = kNegInf; acc.s = 0.f;
    mx[0] = mx[1] = mx[2] = kNegInf;
    for (int j = 0; j < S; ++j) {
      const u64 k = __ldcg(mine + j);
      best = k > best ? k : best;
      if (LSE) {
        const u64 a = __ldcg(mine + 16 + j), b2 = __ldcg(mine + 32 + j), c2 = __ldcg(mine + 48 + j);
        OnlineLse t = {__uint_as_float((uint32_t)(a >> 32)), __uint_as_float((uint32_t)a)};
        acc = lse_merge(acc, t);
        mx[0] = fmax_nan(mx[0], __uint_as_float((uint32_t)(b2 >> 32)));
        mx[1] = fmax_nan(mx[1], __uint_as_float((uint32_t)b2));
        mx[2] = fmax_nan(mx[2], __uint_as_float((uint32_t)(c2 >> 32)));
      }
    }
    count_ws[b] = 0;
  }
  if (p.greedy_keys) {   // sharded round: leave the key (with the global id) for the reduction over shards
    const long long id = (long long)(0xffffffffu - (uint32_t)(best & 0xffffffffu)) + p.vocab_offset;
    p.greedy_keys[b] = best ? (long long)(((best >> 32) << 31) | (u64)(0x7fffffffll - id)) : -1;
    return;
  }
  const long long row = (long long)b * K1 + st.n;
  double lseR;
  bool fin = best != 0;
  if (LSE) {
    lseR = (double)acc.m + log2((double)acc.s);
    // every stream's largest entry finite: no NaN, no +inf, and not -inf throughout
    fin = fin && isfinite(lseR) && isfinite(mx[0]) && isfinite(mx[1]) && isfinite(mx[2]);
    if (!fin) {
      p.status_ws[b] = st.status | SPECSTEER_REQ_NONFINITE;
      if (p.req_status) p.req_status[b] = st.status | SPECSTEER_REQ_NONFINITE;
    }
  } else {
    lseR = (double)p.lse2[row * 4 + Q_R];
  }
  if (!fin) {
    if (p.rec_token) p.rec_token[b] = -1;
    if (p.rec_logprob) p.rec_logprob[b] = __int_as_float(0x7fc00000);
    if (p.n_out) p.n_out[b] = st.n;
    return;
  }
  const int tok = (int)(0xffffffffu - (uint32_t)(best & 0xffffffffu));
  const double r = (double)order_val((uint32_t)(best >> 32));
  if (p.rec_token) p.rec_token[b] = tok;
  if (p.rec_logprob) p.rec_logprob[b] = (float)((r * (double)c - lseR) * 0.6931471805599453);
  if (p.out_tokens) p.out_tokens[(long long)b * K1 + st.n] = tok;
  if (p.n_out) p.n_out[b] = st.n + 1;
}

// Sharded greedy rounds, last step (identical on every GPU): outputs from the keys reduced over the shards.
__global__ void __launch_bounds__(128) greedy_finish_kernel(const RoundParams p, const long long* keys) {
  const int b = blockIdx.x * 128 + threadIdx.x;
  if (b >= p.B) return;
  const int K = p.K, K1 = K + 1;
  const ReqState st = request_state(p, b);
  if (p.out_tokens)
    for (int t = 0; t <= K; ++t)
      p.out_tokens[(long long)b * K1 + t] = (t < st.n) ? p.draft_tokens[(long long)b * K + t] : -1;
  const long long key = keys[b];
  if (!st.sample || key < 0) {
    if (p.rec_token) p.rec_token[b] = -1;
    if (p.rec_logprob) p.rec_logprob[b] = __int_as_float(0x7fc00000);
    if (p.n_out) p.n_out[b] = st.n;
    return;
  }
  const int tok = (int)(0x7fffffffll - (key & 0x7fffffffll));
  const double r = (double)order_val((uint32_t)((unsigned long long)key >> 31));
  const long long row = (long long)b * K1 + st.n;
  const double lseR = (double)p.lse2[row * 4 + Q_R];
  if (p.rec_token) p.rec_token[b] = tok;
  if (p.rec_logprob) p.rec_logprob[b] = (float)((r * (double)(kLog2e / p.temperature[b]) - lseR) * 0.6931471805599453);
  if (p.out_tokens) p.out_tokens[(long long)b * K1 + st.n] = tok;
  if (p.n_out) p.n_out[b] = st.n + 1;
}

cudaError_t launch_greedy_finish(const RoundParams& p, const long long* keys, cudaStream_t s) {
  if (p.B == 0) return cudaSuccess;
  greedy_finish_kernel<<<(p.B + 127) / 128, 128, 0, s>>>(p, keys);
  return cudaGetLastError();
}

template <typename T>
static cudaError_t launch_argmax_t(const cudaLaunchConfig_t& cfg, bool aligned, bool own_lse, const RoundParams& p, u64* ws,
                                   int* count_ws) {
  if (aligned) return own_lse ? cudaLaunchKernelEx(&cfg, recover_argmax_kernel<T, true, true>, p, ws, count_ws)
                              : cudaLaunchKernelEx(&cfg, recover_argmax_kernel<T, true, false>, p, ws, count_ws);
  return own_lse ? cudaLaunchKernelEx(&cfg, recover_argmax_kernel<T, false, true>, p, ws, count_ws)
                 : cudaLaunchKernelEx(&cfg, recover_argmax_kernel<T, false, false>, p, ws, count_ws);
}

cudaError_t launch_recover_argmax(const RoundParams& p, int dtype, bool aligned, bool own_lse, void* best_ws, int* count_ws,
                                  int sm_count, cudaStream_t s) {
  if (p.B == 0) return cudaSuccess;
  int S = (2 * sm_count + p.B - 1) / p.B;   // about two CTAs per SM in total
  S = S < 1 ? 1 : (S > kTopkMaxSplit ? kTopkMaxSplit : S);
  while (S > 1 && (p.V + S - 1) / S < 4096) --S;   // a part below 4096 entries is not worth a CTA
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.B, S);
  cfg.blockDim = dim3(kRecThreads);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  u64* ws = reinterpret_cast<u64*>(best_ws);
  return dtype == SPECSTEER_F32 ? launch_argmax_t<float>(cfg, aligned, own_lse, p, ws, count_ws)
                                : launch_argmax_t<uint16_t>(cfg, aligned, own_lse, p, ws, count_ws);
}

cudaError_t launch_recover(const RoundParams& p, int dtype, const LaunchInfo& li, cudaStream_t s, int* n_launches,
                           bool own_lse) {
  (void)li;
  const size_t smem = (size_t)p.n_chunks * sizeof(double);
  *n_launches = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.B);
  cfg.blockDim = dim3(kRecThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e;
  if (own_lse)
    e = dtype == SPECSTEER_F32 ? cudaLaunchKernelEx(&cfg, recover_steer_kernel<float, kChunkF32, true>, p)
                               : cudaLaunchKernelEx(&cfg, recover_steer_kernel<uint16_t, kChunkBF16, true>, p);
  else
    e = dtype == SPECSTEER_F32 ? cudaLaunchKernelEx(&cfg, recover_steer_kernel<float, kChunkF32, false>, p)
                               : cudaLaunchKernelEx(&cfg, recover_steer_kernel<uint16_t, kChunkBF16, false>, p);
  if (e != cudaSuccess || p.recover_mode != SPECSTEER_RECOVER_RESIDUAL) return e;
  *n_launches = 2;
  if (dtype == SPECSTEER_F32) recover_residual_kernel<float, kChunkF32><<<p.B, kRecThreads, smem, s>>>(p);
  else recover_residual_kernel<uint16_t, kChunkBF16><<<p.B, kRecThreads, smem, s>>>(p);
  return cudaGetLastError();
}

}  // namespace specsteer
