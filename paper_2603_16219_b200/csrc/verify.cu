// Verification kernel: one streaming pass over the three logit tensors.
//
// Work unit: a tile = one chunk of kTile vocabulary entries of one used row, all three streams.
// A persistent CTA per SM owns a ring of shared-memory stages.  One producer thread fills stages
// with 1-D bulk (TMA) copies signalled on mbarriers; each consumer warp owns whole tiles, keeps
// four running (reference exponent, scaled sum) pairs per lane, and writes one 32-byte partial
// record per tile.  The warp that finishes a request's last tile combines the records in chunk
// order, forms the log-probabilities, alpha and the accept flags, and scans them for accept_len
// (Algorithm 1 Phase 2; Eq. 6 / Eq. 7).
#include "common.cuh"
#include "internal.h"
#include "specsteer.h"

namespace specsteer {

constexpr float kSlack = 16.f;  // a lane's reference exponent may lag its running maximum by this much

struct TileMeta {
  int b, t, chunk, n_valid;
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
template <typename T, bool MASKED> struct TilePass;

template <bool MASKED> struct TilePass<float, MASKED> {
  static __device__ __forceinline__ void run(Acc& a, const float* sl, const float* sp, const float* sm, int lane,
                                             int n_valid, float beta, float c) {
    const float4* vl = reinterpret_cast<const float4*>(sl);
    const float4* vp = reinterpret_cast<const float4*>(sp);
    const float4* vm = reinterpret_cast<const float4*>(sm);
#pragma unroll 2
    for (int it = 0; it < kTile / 256; ++it) {
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

template <bool MASKED> struct TilePass<uint16_t, MASKED> {
  static __device__ __forceinline__ void run(Acc& a, const uint16_t* sl, const uint16_t* sp, const uint16_t* sm,
                                             int lane, int n_valid, float beta, float c) {
    const uint4* vl = reinterpret_cast<const uint4*>(sl);
    const uint4* vp = reinterpret_cast<const uint4*>(sp);
    const uint4* vm = reinterpret_cast<const uint4*>(sm);
#pragma unroll 2
    for (int it = 0; it < kTile / 256; ++it) {
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

// ---- per-request epilogue (one warp): Eq. 6/7 and the accepted length ---------------------------
template <typename T>
__device__ void request_epilogue(const RoundParams& p, int b, int lane) {
  const int K = p.K, K1 = K + 1;
  const T* hl = reinterpret_cast<const T*>(p.h_llm);
  const T* hp = reinterpret_cast<const T*>(p.h_plus);
  const T* hm = reinterpret_cast<const T*>(p.h_minus);
  int status = 0;
  int len = p.draft_len[b];
  const float Tmp = p.temperature[b], lam = p.lambda[b], beta = p.beta[b];
  const bool params_ok = isfinite(Tmp) && Tmp > 0.f && isfinite(lam) && lam > 0.f && isfinite(beta);
  if (len < 0 || len > K) { status |= SPECSTEER_REQ_BAD_LEN; len = 0; }
  const bool bonus = (p.flags & SPECSTEER_FLAG_BONUS) != 0;
  const int R = len + (bonus ? 1 : 0);
  const float c = kLog2e / Tmp;
  const double cd = (double)c;
  const float qnan = __int_as_float(0x7fc00000);

  for (int t = lane; t < K; t += 32) {
    const long long i = (long long)b * K + t;
    if (p.accept_flags) p.accept_flags[i] = 0;
    if (p.alpha) p.alpha[i] = 0.f;
    if (p.logp_llm) p.logp_llm[i] = qnan;
    if (p.logp_minus) p.logp_minus[i] = qnan;
    if (p.logp_plus) p.logp_plus[i] = qnan;
    if (p.logp_star) p.logp_star[i] = qnan;
  }
  for (int t = lane; t <= K; t += 32)
    if (p.log_z) p.log_z[(long long)b * K1 + t] = qnan;
  __syncwarp();

  int n = len;
  bool decided = false;
  if (!params_ok) {
    status |= SPECSTEER_REQ_BAD_PARAM;
    n = 0;
  } else {
    for (int t = 0; t < R; ++t) {
      const long long row = (long long)b * K1 + t;
      const float* rec = p.part + row * p.n_chunks * 8;
      // pass 1: largest reference exponent per normaliser; pass 2: exact power-of-two rescale, sums in double
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
      double lse[4];
      bool fin = true;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        double s = S[q];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(kFullMask, s, o);
        lse[q] = (double)M[q] + log2(s);
        fin = fin && isfinite(lse[q]);
      }
      if (lane == 0) {
        float4 o = make_float4((float)lse[0], (float)lse[1], (float)lse[2], (float)lse[3]);
        *reinterpret_cast<float4*>(p.lse2 + row * 4) = o;
      }
      const double logz = (lse[Q_R] - lse[Q_L] - (double)beta * (lse[Q_P] - lse[Q_M])) * (double)kLn2;
      if (t >= len) {  // the bonus row
        if (fin && p.log_z && lane == 0) p.log_z[row] = (float)logz;
        if (!fin && !decided) status |= SPECSTEER_REQ_NONFINITE;
        continue;
      }
      if (!fin) {
        if (!decided) { status |= SPECSTEER_REQ_NONFINITE; n = t; decided = true; }
        continue;
      }
      const long long i = (long long)b * K + t;
      const int y = p.draft_tokens[i];
      float al = 0.f;
      double ald = 0.0;
      bool testable = true;
      double lpL = 0, lpM = 0, lpP = 0, lpS = 0;
      if (y < 0 || y >= p.V) {
        if (!decided) status |= SPECSTEER_REQ_BAD_TOKEN;
        testable = false;
      } else {
        const long long off = (long long)b * p.ld_req + (long long)t * p.ld_row + y;
        const float l = load_logit<T>(hl, off), pp = load_logit<T>(hp, off), m = load_logit<T>(hm, off);
        const double r = (double)l + (double)beta * ((double)pp - (double)m);  // Eq. 8
        const double ln2 = 0.6931471805599453;
        lpL = ((double)l * cd - lse[Q_L]) * ln2;
        lpP = ((double)pp * cd - lse[Q_P]) * ln2;
        lpM = ((double)m * cd - lse[Q_M]) * ln2;
        lpS = (r * cd - lse[Q_R]) * ln2;
        const double logrho = (p.accept_mode == SPECSTEER_ACCEPT_RATIO) ? (lpL - lpM - log((double)lam)) : (lpS - lpP);
        if (isnan(logrho)) testable = false;
        else ald = exp(fmin(0.0, logrho));
        al = (float)ald;
      }
      const bool acc = testable && ((double)p.u_accept[i] <= ald);  // "Uniform(0,1) <= alpha_t", decided in double
      if (lane == 0) {
        if (p.log_z) p.log_z[row] = (float)logz;
        if (p.alpha) p.alpha[i] = al;
        if (p.accept_flags) p.accept_flags[i] = acc ? 1 : 0;
        if (y >= 0 && y < p.V) {
          if (p.logp_llm) p.logp_llm[i] = (float)lpL;
          if (p.logp_minus) p.logp_minus[i] = (float)lpM;
          if (p.logp_plus) p.logp_plus[i] = (float)lpP;
          if (p.logp_star) p.logp_star[i] = (float)lpS;
        }
      }
      if (!decided && !acc) { n = t; decided = true; }
    }
  }
  if (lane == 0) {
    p.accept_len[b] = n;
    p.status_ws[b] = status;
    if (p.req_status) p.req_status[b] = status;
  }
}

// ---- the persistent streaming kernel --------------------------------------------------------------
template <typename T, int STAGES, int NCW, bool BULK>
__global__ void __launch_bounds__((NCW + 1) * 32, 1) verify_kernel(const RoundParams p) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  constexpr int kStageBytes = 3 * kTile * (int)sizeof(T);
  T* tiles = reinterpret_cast<T*>(smem_raw);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw + (size_t)STAGES * kStageBytes);
  uint64_t* empty = full + STAGES;
  TileMeta* meta = reinterpret_cast<TileMeta*>(empty + STAGES);
  int* abort_flag = reinterpret_cast<int*>(meta + STAGES);
  int* row_start = abort_flag + 4;  // [B + 1]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nthreads = (NCW + 1) * 32;
  const bool bonus = (p.flags & SPECSTEER_FLAG_BONUS) != 0;
  const int K = p.K;

  // ---- prologue: barriers, and the prefix of used rows per request (draft_len lives on the device)
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
  const long long total_tiles = (long long)row_start[p.B] * p.n_chunks;
  const int cta = blockIdx.x, G = gridDim.x;
  const T* hl = reinterpret_cast<const T*>(p.h_llm);
  const T* hp = reinterpret_cast<const T*>(p.h_plus);
  const T* hm = reinterpret_cast<const T*>(p.h_minus);

  if (warp == NCW) {
    // ================= producer warp =================
    long long issued = 0;
    for (long long j = 0;; ++j) {
      const long long g = (long long)cta + j * G;
      if (g >= total_tiles) break;
      const int stage = (int)(j % STAGES);
      const uint32_t phase = (uint32_t)((j / STAGES) & 1);
      bool ok = true;
      if (lane == 0) ok = mbar_wait(&empty[stage], phase ^ 1u);
      ok = __shfl_sync(kFullMask, ok ? 1 : 0, 0) != 0;
      if (!ok || *reinterpret_cast<volatile int*>(abort_flag)) {
        if (lane == 0) { *reinterpret_cast<volatile int*>(abort_flag) = 1; atomicExch(p.dev_error, 1); }
        break;
      }
      const int cr = (int)(g / p.n_chunks), chunk = (int)(g % p.n_chunks);
      int lo = 0, hi = p.B;  // largest b with row_start[b] <= cr
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (row_start[mid] <= cr) lo = mid; else hi = mid;
      }
      const int b = lo, t = cr - row_start[lo];
      const int n_valid = min(kTile, p.V - chunk * kTile);
      const long long off = (long long)b * p.ld_req + (long long)t * p.ld_row + (long long)chunk * kTile;
      T* dst = tiles + (size_t)stage * 3 * kTile;
      if (BULK) {
        if (lane == 0) {
          meta[stage] = TileMeta{b, t, chunk, n_valid};
          const int n_bulk = (int)(((size_t)n_valid * sizeof(T)) & ~(size_t)15) / (int)sizeof(T);
          for (int e = n_bulk; e < n_valid; ++e) {  // ragged end of the last chunk: < 16 bytes per stream
            dst[e] = hl[off + e]; dst[kTile + e] = hp[off + e]; dst[2 * kTile + e] = hm[off + e];
          }
          const uint32_t bytes = (uint32_t)(n_bulk * sizeof(T));
          if (bytes) {
            mbar_arrive_expect_tx(&full[stage], 3 * bytes);
            bulk_g2s(dst, hl + off, bytes, &full[stage]);
            bulk_g2s(dst + kTile, hp + off, bytes, &full[stage]);
            bulk_g2s(dst + 2 * kTile, hm + off, bytes, &full[stage]);
          } else {
            mbar_arrive(&full[stage]);
          }
        }
      } else {
        // rows that are not 16-byte aligned: the warp copies element by element
        for (int e = lane; e < n_valid; e += 32) {
          dst[e] = hl[off + e]; dst[kTile + e] = hp[off + e]; dst[2 * kTile + e] = hm[off + e];
        }
        __syncwarp();
        if (lane == 0) {
          meta[stage] = TileMeta{b, t, chunk, n_valid};
          mbar_arrive(&full[stage]);
        }
      }
      ++issued;
    }
    // On an abort, copies already issued may still be landing: wait for them (bounded) before the CTA exits.
    __syncwarp();
    if (BULK && lane == 0 && *reinterpret_cast<volatile int*>(abort_flag)) {
      const long long first = issued > STAGES ? issued - STAGES : 0;
      for (long long j = first; j < issued; ++j) mbar_wait(&full[j % STAGES], (uint32_t)((j / STAGES) & 1));
    }
  } else {
    // ================= consumer warps =================
    // requests that read no row at all still need their outputs
    for (int b = cta + warp * G; b < p.B; b += G * NCW)
      if (row_start[b + 1] == row_start[b]) request_epilogue<T>(p, b, lane);

    for (long long j = warp;; j += NCW) {
      const long long g = (long long)cta + j * G;
      if (g >= total_tiles) break;
      const int stage = (int)(j % STAGES);
      const uint32_t phase = (uint32_t)((j / STAGES) & 1);
      // every lane observes the phase itself: that is what makes the copied bytes visible to it
      bool ok = !*reinterpret_cast<volatile int*>(abort_flag) && mbar_wait(&full[stage], phase);
      ok = __all_sync(kFullMask, ok);
      if (!ok) {
        if (lane == 0) { *reinterpret_cast<volatile int*>(abort_flag) = 1; atomicExch(p.dev_error, 1); }
        break;
      }
      const TileMeta mt = meta[stage];
      const float beta = p.beta[mt.b];
      const float c = kLog2e / p.temperature[mt.b];
      const T* sl = tiles + (size_t)stage * 3 * kTile;
      Acc a;
      acc_init(a);
      if (mt.n_valid == kTile) TilePass<T, false>::run(a, sl, sl + kTile, sl + 2 * kTile, lane, kTile, beta, c);
      else TilePass<T, true>::run(a, sl, sl + kTile, sl + 2 * kTile, lane, mt.n_valid, beta, c);
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[stage]);  // the stage may be refilled while we reduce
      warp_combine(a);
      const int K1 = K + 1;
      const long long row = (long long)mt.b * K1 + mt.t;
      unsigned done = 0;
      if (lane == 0) {
        float* rec = p.part + (row * p.n_chunks + mt.chunk) * 8;
        *reinterpret_cast<float4*>(rec) = make_float4(a.ref[Q_L], a.s[Q_L], a.ref[Q_P], a.s[Q_P]);
        *reinterpret_cast<float4*>(rec + 4) = make_float4(a.ref[Q_M], a.s[Q_M], a.ref[Q_R], a.s[Q_R]);
        __threadfence();
        done = atomicAdd(p.counter + mt.b, 1u) + 1u;
      }
      done = __shfl_sync(kFullMask, done, 0);
      const unsigned need = (unsigned)(row_start[mt.b + 1] - row_start[mt.b]) * (unsigned)p.n_chunks;
      if (done == need) {
        __threadfence();
        if (lane == 0) p.counter[mt.b] = 0;  // ready for the next round
        request_epilogue<T>(p, mt.b, lane);
      }
    }
  }
}

// ---- launch -------------------------------------------------------------------------------------------
template <typename T, int STAGES, int NCW, bool BULK>
static cudaError_t launch_one(const RoundParams& p, const LaunchInfo& li, cudaStream_t s) {
  const size_t smem = (size_t)STAGES * 3 * kTile * sizeof(T) + 2 * STAGES * sizeof(uint64_t) +
                      STAGES * sizeof(TileMeta) + 16 + (size_t)(p.B + 1) * sizeof(int);
  auto kern = verify_kernel<T, STAGES, NCW, BULK>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<li.sm_count, (NCW + 1) * 32, smem, s>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_verify(const RoundParams& p, int dtype, bool aligned, const LaunchInfo& li, cudaStream_t s,
                          int* n_launches) {
  *n_launches = 1;
  if (dtype == SPECSTEER_F32)
    return aligned ? launch_one<float, 8, 8, true>(p, li, s) : launch_one<float, 8, 8, false>(p, li, s);
  return aligned ? launch_one<uint16_t, 16, 16, true>(p, li, s) : launch_one<uint16_t, 16, 16, false>(p, li, s);
}

}  // namespace specsteer
