// Verification: one streaming pass over the three logit tensors, then a small per-request epilogue.
//
// Streaming kernel.  Work unit: a tile = one chunk of TILE vocabulary entries of one used row, all
// three streams.  A persistent CTA per SM owns a ring of shared-memory stages.  One producer thread
// fills stages with 1-D bulk (TMA) copies signalled on mbarriers; each consumer warp owns whole tiles
// (two stages per warp, so that one loads while the other is reduced), keeps four running
// (reference exponent, scaled sum) pairs per lane, and writes one 32-byte partial record per tile.
// Epilogue kernel.  One CTA per request: each warp combines the records of one row in chunk order and
// forms the log-probabilities and alpha; the accept flags are then scanned for accept_len
// (Algorithm 1 Phase 2; Eq. 6 / Eq. 7).
#include "common.cuh"
#include "internal.h"
#include "specsteer.h"

namespace specsteer {

constexpr float kSlack = 16.f;  // a lane's reference exponent may lag its running maximum by this much

struct TileMeta {
  int row, chunk, n_valid;  // padded row index b*(K+1)+t, chunk within the row, valid entries
  float beta, c;            // beta_b and log2(e)/T_b of the owning request
};

struct Acc {
  float ref[4];   // integer-valued reference exponent (base 2), -inf while nothing was seen
  float nref[4];  // -ref, or 0 while empty: the addend of the exponent FMA
  float s[4];     // sum of 2^(x*c - ref)
};

__device__ __forceinline__ void acc_init(Acc& a) {
#pragma unroll
  for (int q = 0; q < 4; ++q) { a.ref[q] = kNegInf; a.nref[q] = 0.f; a.s[q] = 0.f; }
}

// 2^d for an integer-valued d <= 0 (exact); 0 below the normal range.
__device__ __forceinline__ float pow2_nonpos_int(float d) {
  return (d < -126.f) ? 0.f : __int_as_float(((int)d + 127) << 23);
}

__device__ __forceinline__ void acc_raise(Acc& a, int q, float cand) {
  float nr = fmaxf(a.ref[q], ceilf(cand));
  if (nr > a.ref[q]) {
    float f = (a.ref[q] == kNegInf || nr == -kNegInf) ? 0.f : pow2_nonpos_int(a.ref[q] - nr);
    a.s[q] *= f;
    a.ref[q] = nr;
    a.nref[q] = -nr;
  }
}

__device__ __forceinline__ float sum8(const float (&e)[8]) {
  return ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]));
}

// Eight vocabulary entries of the three streams: r = l + beta (p - m)  (Eq. 8), then the four sums.
template <bool MASKED>
__device__ __forceinline__ void accum8(Acc& a, float (&l)[8], float (&p)[8], float (&m)[8], float beta, float c,
                                       unsigned vmask) {
  float r[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) r[i] = fmaf(beta, p[i] - m[i], l[i]);
  if (MASKED) {
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (!((vmask >> i) & 1u)) { l[i] = kNegInf; p[i] = kNegInf; m[i] = kNegInf; r[i] = kNegInf; }
  }
  const float cl = max8(l) * c, cp = max8(p) * c, cm = max8(m) * c, cr = max8(r) * c;
  const bool upd = (cl > a.ref[Q_L] + kSlack) | (cp > a.ref[Q_P] + kSlack) | (cm > a.ref[Q_M] + kSlack) |
                   (cr > a.ref[Q_R] + kSlack);
  if (__any_sync(kFullMask, upd)) {
    acc_raise(a, Q_L, cl); acc_raise(a, Q_P, cp); acc_raise(a, Q_M, cm); acc_raise(a, Q_R, cr);
  }
  float e[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) e[i] = ex2(fmaf(l[i], c, a.nref[Q_L]));
  a.s[Q_L] += sum8(e);
#pragma unroll
  for (int i = 0; i < 8; ++i) e[i] = ex2(fmaf(p[i], c, a.nref[Q_P]));
  a.s[Q_P] += sum8(e);
#pragma unroll
  for (int i = 0; i < 8; ++i) e[i] = ex2(fmaf(m[i], c, a.nref[Q_M]));
  a.s[Q_M] += sum8(e);
#pragma unroll
  for (int i = 0; i < 8; ++i) e[i] = ex2(fmaf(r[i], c, a.nref[Q_R]));
  a.s[Q_R] += sum8(e);
}

// ---- one tile from shared memory, one warp ---------------------------------------------------
template <typename T, int TILE, bool MASKED> struct TilePass;

template <int TILE, bool MASKED> struct TilePass<float, TILE, MASKED> {
  static __device__ __forceinline__ void run(Acc& a, const float* sl, const float* sp, const float* sm, int lane,
                                             int n_valid, float beta, float c) {
    const float4* vl = reinterpret_cast<const float4*>(sl);
    const float4* vp = reinterpret_cast<const float4*>(sp);
    const float4* vm = reinterpret_cast<const float4*>(sm);
#pragma unroll 2
    for (int it = 0; it < TILE / 256; ++it) {
      const int i0 = it * 64 + lane, i1 = i0 + 32;  // two conflict-free 16-byte vectors per stream
      if (MASKED && it * 256 >= n_valid) break;       // warp-uniform: nothing left for any lane
      float4 a0 = vl[i0], a1 = vl[i1], b0 = vp[i0], b1 = vp[i1], c0 = vm[i0], c1 = vm[i1];
      float l[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      float p[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
      float m[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
      unsigned vmask = 0xffu;
      if (MASKED) {
        vmask = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (i0 * 4 + i < n_valid) vmask |= 1u << i;
          if (i1 * 4 + i < n_valid) vmask |= 1u << (4 + i);
        }
      }
      accum8<MASKED>(a, l, p, m, beta, c, vmask);
    }
  }
};

template <int TILE, bool MASKED> struct TilePass<uint16_t, TILE, MASKED> {
  static __device__ __forceinline__ void run(Acc& a, const uint16_t* sl, const uint16_t* sp, const uint16_t* sm,
                                             int lane, int n_valid, float beta, float c) {
    const uint4* vl = reinterpret_cast<const uint4*>(sl);
    const uint4* vp = reinterpret_cast<const uint4*>(sp);
    const uint4* vm = reinterpret_cast<const uint4*>(sm);
#pragma unroll 2
    for (int it = 0; it < TILE / 256; ++it) {
      const int i0 = it * 32 + lane;
      if (MASKED && it * 256 >= n_valid) break;
      uint4 a0 = vl[i0], b0 = vp[i0], c0 = vm[i0];
      float l[8] = {bf16lo(a0.x), bf16hi(a0.x), bf16lo(a0.y), bf16hi(a0.y), bf16lo(a0.z), bf16hi(a0.z), bf16lo(a0.w), bf16hi(a0.w)};
      float p[8] = {bf16lo(b0.x), bf16hi(b0.x), bf16lo(b0.y), bf16hi(b0.y), bf16lo(b0.z), bf16hi(b0.z), bf16lo(b0.w), bf16hi(b0.w)};
      float m[8] = {bf16lo(c0.x), bf16hi(c0.x), bf16lo(c0.y), bf16hi(c0.y), bf16lo(c0.z), bf16hi(c0.z), bf16lo(c0.w), bf16hi(c0.w)};
      unsigned vmask = 0xffu;
      if (MASKED) {
        vmask = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (i0 * 8 + i < n_valid) vmask |= 1u << i;
      }
      accum8<MASKED>(a, l, p, m, beta, c, vmask);
    }
  }
};

// Combine the lanes' pairs into one (reference, sum) per normaliser; every lane gets the result.
__device__ __forceinline__ void warp_combine(Acc& a) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float M = warp_max(a.ref[q]);
    float s = a.s[q];
    if (a.ref[q] != M) s = (a.ref[q] == kNegInf || M == -kNegInf) ? 0.f : s * pow2_nonpos_int(a.ref[q] - M);
    a.s[q] = warp_sum(s);
    a.ref[q] = M;
  }
}

// ---- per-request epilogue: Eq. 6/7 and the accepted length ------------------------------------------
constexpr int kEpiWarps = 8;
constexpr int kEpiMaxRows = 64;  // rows of one request held in shared memory; more run in several rounds

struct RowResult {
  double lse[4];
  double logz;
  float alpha;
  float lp[4];      // log-probabilities L, P, M, R(star) of the drafted token
  int8_t fin;       // all four normalisers finite
  int8_t testable;  // token in range and ratio defined
  int8_t accept;
  int8_t tok_ok;
};

// One warp: combine the partial records of `row` in chunk order (exact power-of-two rescale, sums in
// double) and, for a drafted row, the log-probabilities, alpha and the accept decision.
template <typename T>
__device__ void epilogue_row(const RoundParams& p, int b, int t, int len, float beta, float lam, float c, int lane,
                             RowResult* out) {
  const int K = p.K, K1 = K + 1;
  const long long row = (long long)b * K1 + t;
  const float* rec = p.part + row * p.n_chunks * 8;
  float M[4] = {kNegInf, kNegInf, kNegInf, kNegInf};
  for (int ch = lane; ch < p.n_chunks; ch += 32) {
    float4 x = ld_cg_f4(rec + ch * 8), y = ld_cg_f4(rec + ch * 8 + 4);
    M[0] = fmaxf(M[0], x.x); M[1] = fmaxf(M[1], x.z); M[2] = fmaxf(M[2], y.x); M[3] = fmaxf(M[3], y.z);
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) M[q] = warp_max(M[q]);
  double S[4] = {0.0, 0.0, 0.0, 0.0};
  for (int ch = lane; ch < p.n_chunks; ch += 32) {
    float4 x = ld_cg_f4(rec + ch * 8), y = ld_cg_f4(rec + ch * 8 + 4);
    const float mm[4] = {x.x, x.z, y.x, y.z}, ss[4] = {x.y, x.w, y.y, y.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float w = ss[q];
      if (mm[q] != M[q]) w = (mm[q] == kNegInf || M[q] == -kNegInf) ? 0.f : w * pow2_nonpos_int(mm[q] - M[q]);
      S[q] += (double)w;
    }
  }
  RowResult r;
  bool fin = true;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    double s = S[q];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(kFullMask, s, o);
    r.lse[q] = (double)M[q] + log2(s);
    fin = fin && isfinite(r.lse[q]);
  }
  const double ln2 = 0.6931471805599453;
  r.logz = (r.lse[Q_R] - r.lse[Q_L] - (double)beta * (r.lse[Q_P] - r.lse[Q_M])) * ln2;
  r.fin = fin; r.testable = 0; r.accept = 0; r.tok_ok = 0; r.alpha = 0.f;
  r.lp[0] = r.lp[1] = r.lp[2] = r.lp[3] = __int_as_float(0x7fc00000);
  if (lane == 0)
    *reinterpret_cast<float4*>(p.lse2 + row * 4) =
        make_float4((float)r.lse[0], (float)r.lse[1], (float)r.lse[2], (float)r.lse[3]);
  if (fin && t < len) {
    const long long i = (long long)b * K + t;
    const int y = p.draft_tokens[i];
    if (y >= 0 && y < p.V) {
      const T* hl = reinterpret_cast<const T*>(p.h_llm);
      const T* hp = reinterpret_cast<const T*>(p.h_plus);
      const T* hm = reinterpret_cast<const T*>(p.h_minus);
      const long long off = (long long)b * p.ld_req + (long long)t * p.ld_row + y;
      const double cd = (double)c;
      const double l = (double)load_logit<T>(hl, off), pp = (double)load_logit<T>(hp, off),
                   m = (double)load_logit<T>(hm, off);
      const double rr = l + (double)beta * (pp - m);  // Eq. 8
      const double lpL = (l * cd - r.lse[Q_L]) * ln2, lpP = (pp * cd - r.lse[Q_P]) * ln2,
                   lpM = (m * cd - r.lse[Q_M]) * ln2, lpS = (rr * cd - r.lse[Q_R]) * ln2;
      r.lp[Q_L] = (float)lpL; r.lp[Q_P] = (float)lpP; r.lp[Q_M] = (float)lpM; r.lp[Q_R] = (float)lpS;
      r.tok_ok = 1;
      const double logrho = (p.accept_mode == SPECSTEER_ACCEPT_RATIO) ? (lpL - lpM - log((double)lam))  // Eq. 7
                                                                      : (lpS - lpP);                    // Eq. 6
      if (!isnan(logrho)) {
        const double ald = exp(fmin(0.0, logrho));
        r.alpha = (float)ald;
        r.testable = 1;
        r.accept = ((double)p.u_accept[i] <= ald) ? 1 : 0;  // "Uniform(0,1) <= alpha_t", decided in double
      }
    }
  }
  if (lane == 0) *out = r;
}

template <typename T>
__global__ void __launch_bounds__(kEpiWarps * 32) epilogue_kernel(const RoundParams p) {
  __shared__ RowResult res[kEpiMaxRows];
  const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int K = p.K, K1 = K + 1;
  int status = 0;
  int len = p.draft_len[b];
  const float Tmp = p.temperature[b], lam = p.lambda[b], beta = p.beta[b];
  const bool params_ok = isfinite(Tmp) && Tmp > 0.f && isfinite(lam) && lam > 0.f && isfinite(beta);
  if (len < 0 || len > K) { status |= SPECSTEER_REQ_BAD_LEN; len = 0; }
  const bool bonus = (p.flags & SPECSTEER_FLAG_BONUS) != 0;
  const int R = params_ok ? len + (bonus ? 1 : 0) : 0;
  const float c = kLog2e / Tmp;
  const float qnan = __int_as_float(0x7fc00000);

  for (int t = tid; t < K; t += kEpiWarps * 32) {
    const long long i = (long long)b * K + t;
    if (p.accept_flags) p.accept_flags[i] = 0;
    if (p.alpha) p.alpha[i] = 0.f;
    if (p.logp_llm) p.logp_llm[i] = qnan;
    if (p.logp_minus) p.logp_minus[i] = qnan;
    if (p.logp_plus) p.logp_plus[i] = qnan;
    if (p.logp_star) p.logp_star[i] = qnan;
  }
  for (int t = tid; t <= K; t += kEpiWarps * 32)
    if (p.log_z) p.log_z[(long long)b * K1 + t] = qnan;

  int n = len;
  bool decided = false;
  if (!params_ok) { status |= SPECSTEER_REQ_BAD_PARAM; n = 0; }
  for (int t0 = 0; t0 < R; t0 += kEpiMaxRows) {
    const int nr = min(kEpiMaxRows, R - t0);
    __syncthreads();  // defaults written / previous round consumed
    for (int k = warp; k < nr; k += kEpiWarps) epilogue_row<T>(p, b, t0 + k, len, beta, lam, c, lane, &res[k]);
    __syncthreads();
    // outputs of these rows (any thread), then the sequential scan (every thread, same result)
    for (int k = tid; k < nr; k += kEpiWarps * 32) {
      const int t = t0 + k;
      const RowResult& r = res[k];
      if (r.fin && p.log_z) p.log_z[(long long)b * K1 + t] = (float)r.logz;
      if (t < len && r.fin) {
        const long long i = (long long)b * K + t;
        if (p.alpha) p.alpha[i] = r.alpha;
        if (p.accept_flags) p.accept_flags[i] = (uint8_t)r.accept;
        if (r.tok_ok) {
          if (p.logp_llm) p.logp_llm[i] = r.lp[Q_L];
          if (p.logp_minus) p.logp_minus[i] = r.lp[Q_M];
          if (p.logp_plus) p.logp_plus[i] = r.lp[Q_P];
          if (p.logp_star) p.logp_star[i] = r.lp[Q_R];
        }
      }
    }
    for (int k = 0; k < nr; ++k) {
      const int t = t0 + k;
      const RowResult& r = res[k];
      if (t >= len) {  // the bonus row, reached only when every draft was accepted
        if (!r.fin && !decided) status |= SPECSTEER_REQ_NONFINITE;
        continue;
      }
      if (!r.fin) {
        if (!decided) { status |= SPECSTEER_REQ_NONFINITE; n = t; decided = true; }
        continue;
      }
      if (!r.tok_ok && !decided) status |= SPECSTEER_REQ_BAD_TOKEN;
      if (!decided && !r.accept) { n = t; decided = true; }
    }
  }
  if (tid == 0) {
    p.accept_len[b] = n;
    p.status_ws[b] = status;
    if (p.req_status) p.req_status[b] = status;
  }
}

// ---- the persistent streaming kernel --------------------------------------------------------------
// Warps [0, NCW) consume tiles; warps [NCW, NCW+NPW) each run one elected producer thread that owns the
// stages congruent to its index modulo NPW (one thread cannot issue tiles fast enough for a whole SM).
template <typename T, int TILE, int STAGES, int NCW, int NPW, bool BULK>
__global__ void __launch_bounds__((NCW + NPW) * 32, 1) verify_kernel(const RoundParams p) {
  static_assert(STAGES % NPW == 0, "each producer owns a fixed subset of the stages");
  extern __shared__ __align__(128) unsigned char smem_raw[];
  constexpr int kStageBytes = 3 * TILE * (int)sizeof(T);
  T* tiles = reinterpret_cast<T*>(smem_raw);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw + (size_t)STAGES * kStageBytes);
  uint64_t* empty = full + STAGES;
  TileMeta* meta = reinterpret_cast<TileMeta*>(empty + STAGES);
  int* abort_flag = reinterpret_cast<int*>(meta + STAGES);
  int* row_start = abort_flag + 4;                           // [B + 1]
  float* beta_s = reinterpret_cast<float*>(row_start + p.B + 1);  // [B]
  float* c_s = beta_s + p.B;                                 // [B]  log2(e) / T_b

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int nthreads = (NCW + NPW) * 32;
  const bool bonus = (p.flags & SPECSTEER_FLAG_BONUS) != 0;
  const int K = p.K;

  // ---- prologue: barriers, per-request constants, and the prefix of used rows per request
  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    *abort_flag = 0;
    row_start[0] = 0;
    fence_barrier_init();
  }
  for (int b = tid; b < p.B; b += nthreads) {
    int len = p.draft_len[b];
    if (len < 0 || len > K) len = 0;
    row_start[b + 1] = len + (bonus ? 1 : 0);
    beta_s[b] = p.beta[b];
    c_s[b] = kLog2e / p.temperature[b];
  }
  __syncthreads();
  if (warp == 0) {  // inclusive scan, 32 entries at a time
    int carry = 0;
    for (int b0 = 0; b0 < p.B; b0 += 32) {
      int v = (b0 + lane < p.B) ? row_start[b0 + lane + 1] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int u = __shfl_up_sync(kFullMask, v, o);
        if (lane >= o) v += u;
      }
      v += carry;
      if (b0 + lane < p.B) row_start[b0 + lane + 1] = v;
      carry = __shfl_sync(kFullMask, v, 31);
    }
  }
  __syncthreads();
  const int total_tiles = row_start[p.B] * p.n_chunks;  // the host guarantees this fits in 31 bits
  const int cta = blockIdx.x, G = gridDim.x;

  if (warp >= NCW) {
    // ================= producer warps =================
    const int pw = warp - NCW;
    const T* hl = reinterpret_cast<const T*>(p.h_llm);
    const T* hp = reinterpret_cast<const T*>(p.h_plus);
    const T* hm = reinterpret_cast<const T*>(p.h_minus);
    int issued = 0;
    // tile g = cta + j*G  ->  (compact row cr, chunk); advanced incrementally, no division in the loop
    const int g0 = cta + pw * G, gstep = NPW * G;
    const int step_rows = gstep / p.n_chunks, step_chunks = gstep % p.n_chunks;
    int cr = g0 / p.n_chunks, chunk = g0 % p.n_chunks;
    int b = 0;
    const int K1 = K + 1;
    for (int j = pw, g = g0; g < total_tiles; j += NPW, g += gstep) {
      const int stage = j % STAGES;
      const uint32_t phase = (uint32_t)((j / STAGES) & 1);
      bool ok = true;
      if (BULK) {
        if (lane == 0) ok = mbar_wait(&empty[stage], phase ^ 1u);
        ok = __shfl_sync(kFullMask, ok ? 1 : 0, 0) != 0;
      } else {
        ok = __all_sync(kFullMask, mbar_wait(&empty[stage], phase ^ 1u));
      }
      if (!ok || *reinterpret_cast<volatile int*>(abort_flag)) {
        if (lane == 0) { *reinterpret_cast<volatile int*>(abort_flag) = 1; atomicExch(p.dev_error, 1); }
        break;
      }
      while (row_start[b + 1] <= cr) ++b;  // cr < row_start[B], so b stays below B
      const int t = cr - row_start[b];
      const int n_valid = min(TILE, p.V - chunk * TILE);
      const long long off = (long long)b * p.ld_req + (long long)t * p.ld_row + (long long)chunk * TILE;
      T* dst = tiles + (size_t)stage * 3 * TILE;
      if (BULK) {
        if (lane == 0) {
          meta[stage] = TileMeta{b * K1 + t, chunk, n_valid, beta_s[b], c_s[b]};
          const int n_bulk = (int)(((size_t)n_valid * sizeof(T)) & ~(size_t)15) / (int)sizeof(T);
          for (int e = n_bulk; e < n_valid; ++e) {  // ragged end of the last chunk: < 16 bytes per stream
            dst[e] = hl[off + e]; dst[TILE + e] = hp[off + e]; dst[2 * TILE + e] = hm[off + e];
          }
          const uint32_t bytes = (uint32_t)(n_bulk * sizeof(T));
          if (bytes) {
            mbar_arrive_expect_tx(&full[stage], 3 * bytes);
            bulk_g2s(dst, hl + off, bytes, &full[stage]);
            bulk_g2s(dst + TILE, hp + off, bytes, &full[stage]);
            bulk_g2s(dst + 2 * TILE, hm + off, bytes, &full[stage]);
          } else {
            mbar_arrive(&full[stage]);
          }
        }
      } else {
        // rows that are not 16-byte aligned: the warp copies element by element
        for (int e = lane; e < n_valid; e += 32) {
          dst[e] = hl[off + e]; dst[TILE + e] = hp[off + e]; dst[2 * TILE + e] = hm[off + e];
        }
        __syncwarp();
        if (lane == 0) {
          meta[stage] = TileMeta{b * K1 + t, chunk, n_valid, beta_s[b], c_s[b]};
          mbar_arrive(&full[stage]);
        }
      }
      ++issued;
      cr += step_rows; chunk += step_chunks;
      if (chunk >= p.n_chunks) { chunk -= p.n_chunks; ++cr; }
    }
    // On an abort, copies already issued may still be landing: wait for them (bounded) before the CTA exits.
    __syncwarp();
    if (BULK && lane == 0 && *reinterpret_cast<volatile int*>(abort_flag)) {
      constexpr int kOwn = STAGES / NPW;
      const int first = issued > kOwn ? issued - kOwn : 0;
      for (int i = first; i < issued; ++i) {
        const int j = pw + i * NPW;
        mbar_wait(&full[j % STAGES], (uint32_t)((j / STAGES) & 1));
      }
    }
  } else {
    // ================= consumer warps =================
    for (int j = warp, g = cta + warp * G; g < total_tiles; j += NCW, g += NCW * G) {
      const int stage = j % STAGES;
      const uint32_t phase = (uint32_t)((j / STAGES) & 1);
      // every lane observes the phase itself: that is what makes the copied bytes visible to it
      bool ok = !*reinterpret_cast<volatile int*>(abort_flag) && mbar_wait(&full[stage], phase);
      ok = __all_sync(kFullMask, ok);
      if (!ok) {
        if (lane == 0) { *reinterpret_cast<volatile int*>(abort_flag) = 1; atomicExch(p.dev_error, 1); }
        break;
      }
      const TileMeta mt = meta[stage];
      const T* sl = tiles + (size_t)stage * 3 * TILE;
      Acc a;
      acc_init(a);
      if (mt.n_valid == TILE) TilePass<T, TILE, false>::run(a, sl, sl + TILE, sl + 2 * TILE, lane, TILE, mt.beta, mt.c);
      else TilePass<T, TILE, true>::run(a, sl, sl + TILE, sl + 2 * TILE, lane, mt.n_valid, mt.beta, mt.c);
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[stage]);  // the stage may be refilled while we reduce
      warp_combine(a);
      if (lane == 0) {
        float* rec = p.part + ((long long)mt.row * p.n_chunks + mt.chunk) * 8;
        *reinterpret_cast<float4*>(rec) = make_float4(a.ref[Q_L], a.s[Q_L], a.ref[Q_P], a.s[Q_P]);
        *reinterpret_cast<float4*>(rec + 4) = make_float4(a.ref[Q_M], a.s[Q_M], a.ref[Q_R], a.s[Q_R]);
      }
    }
  }
}

// ---- launch -------------------------------------------------------------------------------------------
template <typename T, int TILE, int STAGES, int NCW, int NPW, bool BULK>
static cudaError_t launch_stream(const RoundParams& p, const LaunchInfo& li, cudaStream_t s) {
  const size_t fixed = (size_t)STAGES * 3 * TILE * sizeof(T) + 2 * STAGES * sizeof(uint64_t) +
                       STAGES * sizeof(TileMeta) + 16;
  const size_t smem = fixed + (size_t)(3 * p.B + 1) * sizeof(int);
  auto kern = verify_kernel<T, TILE, STAGES, NCW, NPW, BULK>;
  static bool attr_set_dev[64] = {};  // per instantiation and device; sized for the largest slab
  bool& attr_set = attr_set_dev[li.device & 63];
  if (!attr_set) {
    const size_t smem_max = fixed + (size_t)(3 * kMaxSlabB + 1) * sizeof(int);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  kern<<<li.sm_count, (NCW + NPW) * 32, smem, s>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_verify(const RoundParams& p, int dtype, bool aligned, const LaunchInfo& li, cudaStream_t s,
                          int* n_launches) {
  *n_launches = 2;
  cudaError_t e;
  if (dtype == SPECSTEER_F32) {
    e = aligned ? launch_stream<float, kTileF32, 16, 8, 4, true>(p, li, s)
                : launch_stream<float, kTileF32, 16, 8, 4, false>(p, li, s);
    if (e != cudaSuccess) return e;
    epilogue_kernel<float><<<p.B, kEpiWarps * 32, 0, s>>>(p);
  } else {
    e = aligned ? launch_stream<uint16_t, kTileBF16, 16, 8, 4, true>(p, li, s)
                : launch_stream<uint16_t, kTileBF16, 16, 8, 4, false>(p, li, s);
    if (e != cudaSuccess) return e;
    epilogue_kernel<uint16_t><<<p.B, kEpiWarps * 32, 0, s>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace specsteer
