// Verification: one streaming pass over the three logit tensors, then a small per-request epilogue.
//
// Streaming kernel.  Work unit: a tile = two chunks of vocabulary entries of one used row, all three
// streams (12 KB).  A persistent CTA per SM owns a ring of shared-memory stages.  A few producer threads
// fill stages with 1-D bulk (TMA) copies signalled on mbarriers; the consumer warps work in pairs, each
// pair owns two stages (one loads while the other is reduced) and each warp of the pair reduces one chunk:
// four (reference exponent, sum) pairs, the references uniform over the warp, and writes one 32-byte partial
// record per chunk.  A full chunk is first tried without any test inside it; an overflow sends it through
// the variant that tests every batch.
// Epilogue kernel.  One CTA per request: each warp combines the records of one row and forms the
// log-probabilities and alpha; the accept flags are then scanned for accept_len
// (Algorithm 1 Phase 2; Eq. 6 / Eq. 7).  With a sharded vocabulary the rows come from the shards' gathered
// partials instead of the records.
#include <atomic>

#include "common.cuh"
#include "internal.h"
#include "records.cuh"
#include "recover_steer.cuh"
#include "specsteer.h"

namespace specsteer {

constexpr float kSlack = 16.f;  // careful path: the reference exponent may lag the running maximum by this much

struct alignas(16) TileMeta {
  float ref[4];            // reference exponents of the row for the four normalisers (row_ref_kernel); ref[0] NaN: none.
                           // First and 16-byte aligned: they arrive with the tile, as a fourth bulk copy
  int row, tile, n_valid;  // padded row index b*(K+1)+t, tile within the row, valid entries in the tile
  float beta, c, inv_c;    // beta_b, log2(e)/T_b and its reciprocal for the owning request
  int req, pad;            // the owning request
};
static_assert(sizeof(TileMeta) == 48, "stage metadata: 16 bytes of references, then the tile's coordinates");

// Packed pairs of float32 (sm_100 f32x2 arithmetic): one instruction, two lanes of a 64-bit register.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float a, float b) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// A warp's running state for the four normalisers of a chunk (L, P, M and r of Eq. 8).  The reference
// exponents are the same in every lane; the sums are per lane.
struct Acc {
  float ref[4];    // integer-valued reference exponent (base 2), -inf while nothing finite was seen
  float thr[4];    // (ref + kSlack) / c: a logit above it raises the reference
  f32x2 nref2[4];  // (-ref, -ref), or (0, 0) while ref is -inf: the addend of the exponent FMA
  f32x2 s2[4];     // two partial sums of 2^(x*c - ref)
};

__device__ __forceinline__ void acc_set_ref(Acc& a, int q, float nr, float inv_c) {
  a.ref[q] = nr;
  const float n = (nr > kNegInf) ? -nr : 0.f;  // also 0 for a NaN reference
  a.nref2[q] = pack2(n, n);
  a.thr[q] = (nr + kSlack) * inv_c;
}

// First batch of a chunk: the references come from the warp-wide maxima of this batch, plus `bias`.
__device__ __forceinline__ void acc_start(Acc& a, const float (&bm)[4], float c, float inv_c, float bias = 0.f) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    acc_set_ref(a, q, ceilf(warp_max_redux(bm[q]) * c) + bias, inv_c);   // one warp-wide float maximum each
    a.s2[q] = 0ull;
  }
}

// A later batch holds a logit above a threshold: raise the references (rarely taken).
__device__ __forceinline__ void acc_raise(Acc& a, const float (&bm)[4], float c, float inv_c, int lane) {
  const float mine = warp_reduce4<true>(bm, lane);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float nr = fmaxf(a.ref[q], ceilf(__shfl_sync(kFullMask, mine, 8 * q) * c));
    if (nr > a.ref[q]) {
      const float f = (a.ref[q] == kNegInf || nr == -kNegInf) ? 0.f : pow2_nonpos_int(a.ref[q] - nr);
      a.s2[q] = mul2(a.s2[q], pack2(f, f));
      acc_set_ref(a, q, nr, inv_c);
    }
  }
}

__device__ __forceinline__ float max8(const f32x2 (&v)[4]) {
  float x[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) unpack2(v[i], x[2 * i], x[2 * i + 1]);
  return fmaxf(max3(max3(x[0], x[1], x[2]), max3(x[3], x[4], x[5]), x[6]), x[7]);
}

// sum += 2^(x*c - ref) over eight entries of one stream
__device__ __forceinline__ void exp_sum8(f32x2& s2, const f32x2 (&x)[4], f32x2 c2, f32x2 nref2) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float a0, a1;
    unpack2(fma2(x[i], c2, nref2), a0, a1);
    s2 = add2(s2, pack2(ex2(a0), ex2(a1)));
  }
}

// 2^a for a pair of arguments on the FMA and integer pipes instead of the special-function unit, which 16-bit
// logits saturate (half the bytes per power of two): a is clamped below at -126, n = round(a) comes from the
// 1.5 * 2^23 trick, 2^(a - n) from a cubic (relative error below 7.5e-5, 5e-6 on average), and n is added into the
// exponent field.  Used for the normaliser of h_SLM+ alone, which no decision depends on under the ratio rule
// (it feeds logp_plus and log_z).  amax collects the largest argument: the caller rejects the chunk when it is not
// below 120, since above 127 the exponent field would overflow; a NaN argument is swallowed by the clamp, which is
// why the caller also forms the normaliser of h_rec (NaN there whenever h_SLM+ is NaN) with ex2.
__device__ __forceinline__ f32x2 exp2_cubic2(f32x2 a, float& amax) {
  const float kMagic = 12582912.f;  // 1.5 * 2^23
  float a0, a1;
  unpack2(a, a0, a1);
  amax = max3(amax, a0, a1);
  const f32x2 ac = pack2(fmaxf(a0, -126.f), fmaxf(a1, -126.f));
  const f32x2 magic2 = pack2(kMagic, kMagic);
  const f32x2 y = add2(ac, magic2);
  const f32x2 f = sub2(ac, sub2(y, magic2));   // in [-0.5, 0.5]
  f32x2 q = pack2(0.05517147481441498f, 0.05517147481441498f);
  q = fma2(q, f, pack2(0.24261066317558289f, 0.24261066317558289f));
  q = fma2(q, f, pack2(0.6932609677314758f, 0.6932609677314758f));
  q = fma2(q, f, pack2(0.9999281167984009f, 0.9999281167984009f));
  float q0, q1, y0, y1;
  unpack2(q, q0, q1);
  unpack2(y, y0, y1);
  return pack2(__uint_as_float(__float_as_uint(q0) + (__float_as_uint(y0) << 23)),
               __uint_as_float(__float_as_uint(q1) + (__float_as_uint(y1) << 23)));
}

// exp_sum8 with the first NPOLY of the four pairs on the cubic
template <int NPOLY>
__device__ __forceinline__ void exp_sum8_mixed(f32x2& s2, const f32x2 (&x)[4], f32x2 c2, f32x2 nref2, float& amax) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const f32x2 arg = fma2(x[i], c2, nref2);
    if (i < NPOLY) {
      s2 = add2(s2, exp2_cubic2(arg, amax));
    } else {
      float a0, a1;
      unpack2(arg, a0, a1);
      s2 = add2(s2, pack2(ex2(a0), ex2(a1)));
    }
  }
}

// Eight vocabulary entries per lane of the three streams: r = l + beta (p - m)  (Eq. 8), then the four sums.
template <bool MASKED, bool FIRST, int SUMS>
__device__ __forceinline__ void accum8(Acc& a, f32x2 (&l)[4], f32x2 (&p)[4], f32x2 (&m)[4], f32x2 beta2, f32x2 c2,
                                       float c, float inv_c, unsigned vmask, int lane) {
  f32x2 r[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) r[i] = fma2(beta2, sub2(p[i], m[i]), l[i]);
  if (MASKED) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const bool k0 = (vmask >> (2 * i)) & 1u, k1 = (vmask >> (2 * i + 1)) & 1u;
      if (!(k0 && k1)) {
        float x0, x1;
        unpack2(l[i], x0, x1); l[i] = pack2(k0 ? x0 : kNegInf, k1 ? x1 : kNegInf);
        unpack2(p[i], x0, x1); p[i] = pack2(k0 ? x0 : kNegInf, k1 ? x1 : kNegInf);
        unpack2(m[i], x0, x1); m[i] = pack2(k0 ? x0 : kNegInf, k1 ? x1 : kNegInf);
        unpack2(r[i], x0, x1); r[i] = pack2(k0 ? x0 : kNegInf, k1 ? x1 : kNegInf);
      }
    }
  }
  // order of Q_L, Q_P, Q_M, Q_R; a normaliser that is not wanted never leaves -inf
  const float bm[4] = {(SUMS & SUM_L) ? max8(l) : kNegInf, (SUMS & SUM_P) ? max8(p) : kNegInf,
                       (SUMS & SUM_M) ? max8(m) : kNegInf, (SUMS & SUM_R) ? max8(r) : kNegInf};
  if (FIRST) {
    acc_start(a, bm, c, inv_c);
  } else {
    const bool upd = (bm[0] > a.thr[0]) | (bm[1] > a.thr[1]) | (bm[2] > a.thr[2]) | (bm[3] > a.thr[3]);
    if (__any_sync(kFullMask, upd)) acc_raise(a, bm, c, inv_c, lane);
  }
  if (SUMS & SUM_L) exp_sum8(a.s2[Q_L], l, c2, a.nref2[Q_L]);
  if (SUMS & SUM_P) exp_sum8(a.s2[Q_P], p, c2, a.nref2[Q_P]);
  if (SUMS & SUM_M) exp_sum8(a.s2[Q_M], m, c2, a.nref2[Q_M]);
  if (SUMS & SUM_R) exp_sum8(a.s2[Q_R], r, c2, a.nref2[Q_R]);
}

// ---- one chunk (half a tile) from shared memory, one warp ---------------------------------------
template <typename T> struct Batch;

template <> struct Batch<float> {
  // batch `it` of a chunk: two conflict-free 16-byte vectors per stream and lane (entries 4*i0.., 4*i1..)
  static __device__ __forceinline__ void load(const float* s, int it, int lane, f32x2 (&x)[4]) {
    const ulonglong2* v = reinterpret_cast<const ulonglong2*>(s);
    const ulonglong2 a0 = v[it * 64 + lane], a1 = v[it * 64 + 32 + lane];
    x[0] = a0.x; x[1] = a0.y; x[2] = a1.x; x[3] = a1.y;
  }
  static __device__ __forceinline__ unsigned mask(int it, int lane, int n_valid) {
    unsigned vm = 0;
    const int e0 = (it * 64 + lane) * 4, e1 = e0 + 128;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (e0 + i < n_valid) vm |= 1u << i;
      if (e1 + i < n_valid) vm |= 1u << (4 + i);
    }
    return vm;
  }
};

template <> struct Batch<uint16_t> {
  static __device__ __forceinline__ void load(const uint16_t* s, int it, int lane, f32x2 (&x)[4]) {
    const uint4 a = reinterpret_cast<const uint4*>(s)[it * 32 + lane];
    x[0] = pack2(bf16lo(a.x), bf16hi(a.x)); x[1] = pack2(bf16lo(a.y), bf16hi(a.y));
    x[2] = pack2(bf16lo(a.z), bf16hi(a.z)); x[3] = pack2(bf16lo(a.w), bf16hi(a.w));
  }
  static __device__ __forceinline__ unsigned mask(int it, int lane, int n_valid) {
    unsigned vm = 0;
    const int e0 = (it * 32 + lane) * 8;
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (e0 + i < n_valid) vm |= 1u << i;
    return vm;
  }
};

template <typename T, int CHUNK, bool MASKED, int SUMS>
__device__ __forceinline__ void chunk_pass(Acc& a, const T* sl, const T* sp, const T* sm, int lane, int n_valid,
                                           float beta, float c, float inv_c) {
  const f32x2 beta2 = pack2(beta, beta), c2 = pack2(c, c);
#pragma unroll
  for (int it = 0; it < CHUNK / 256; ++it) {
    if (MASKED && it > 0 && it * 256 >= n_valid) break;  // warp-uniform: nothing left for any lane
    f32x2 l[4], p[4], m[4];
    Batch<T>::load(sl, it, lane, l);
    if (SUMS & (SUM_P | SUM_R)) Batch<T>::load(sp, it, lane, p);   // otherwise the h_SLM+ slot was never filled
    else p[0] = p[1] = p[2] = p[3] = 0ull;
    Batch<T>::load(sm, it, lane, m);
    const unsigned vmask = MASKED ? Batch<T>::mask(it, lane, n_valid) : 0xffu;
    if (it == 0) accum8<MASKED, true, SUMS>(a, l, p, m, beta2, c2, c, inv_c, vmask, lane);
    else accum8<MASKED, false, SUMS>(a, l, p, m, beta2, c2, c, inv_c, vmask, lane);
  }
}

// The fast variant for a full chunk: nothing is tested inside it.  The reference exponents come from the row
// (row_ref_kernel: kBias binades above the row's logits at its drafted token, which was sampled from Softmax(h_SLM+)
// and so lies near the top of the row) or, when the row has none, from the maxima of the chunk's first batch plus
// kBias.  Either way later entries may exceed the value the reference was taken from by 2^(kBias + 120) before a sum
// overflows, while entries down to 2^-(126 - kBias) of it still count (what is dropped is below 2^-66 of an entry
// of the row).  At the chunk's end a sum that is not below 2^120 (or is NaN), or a cubic argument that left its
// range, makes the warp return false and the caller redoes the chunk with chunk_pass, which tests every batch.
// POLY: the first POLY of the four pairs per batch of h_SLM+ take the cubic instead of ex2.approx.
constexpr float kBias = 60.f;

template <typename T, int CHUNK, int SUMS, int POLY, bool REF>
__device__ __forceinline__ bool chunk_fast(Acc& a, const T* sl, const T* sp, const T* sm, int lane, float beta,
                                           float c, float inv_c, const float* row_ref) {
  const f32x2 beta2 = pack2(beta, beta), c2 = pack2(c, c);
  constexpr bool kPlus = (SUMS & (SUM_P | SUM_R)) != 0;   // the h_SLM+ slot is filled and read
  static_assert(POLY == 0 || (SUMS & SUM_R), "a NaN in h_SLM+ must still reach a sum formed with ex2");
  float amax = kNegInf;
  if (REF) {
#pragma unroll
    for (int q = 0; q < 4; ++q) { acc_set_ref(a, q, (SUMS & (1 << q)) ? row_ref[q] : kNegInf, inv_c); a.s2[q] = 0ull; }
  } else {   // the first batch apart: it also gives the references
    f32x2 l[4], p[4], m[4], r[4];
    Batch<T>::load(sl, 0, lane, l);
    if (kPlus) Batch<T>::load(sp, 0, lane, p);
    Batch<T>::load(sm, 0, lane, m);
    if (SUMS & SUM_R) {
#pragma unroll
      for (int i = 0; i < 4; ++i) r[i] = fma2(beta2, sub2(p[i], m[i]), l[i]);
    }
    const float bm[4] = {(SUMS & SUM_L) ? max8(l) : kNegInf, (SUMS & SUM_P) ? max8(p) : kNegInf,
                         (SUMS & SUM_M) ? max8(m) : kNegInf, (SUMS & SUM_R) ? max8(r) : kNegInf};
    acc_start(a, bm, c, inv_c, kBias);
    if (SUMS & SUM_L) exp_sum8(a.s2[Q_L], l, c2, a.nref2[Q_L]);
    if (SUMS & SUM_P) {
      if (POLY > 0) exp_sum8_mixed<POLY>(a.s2[Q_P], p, c2, a.nref2[Q_P], amax);
      else exp_sum8(a.s2[Q_P], p, c2, a.nref2[Q_P]);
    }
    if (SUMS & SUM_M) exp_sum8(a.s2[Q_M], m, c2, a.nref2[Q_M]);
    if (SUMS & SUM_R) exp_sum8(a.s2[Q_R], r, c2, a.nref2[Q_R]);
  }
#pragma unroll 1
  for (int it = REF ? 0 : 1; it < CHUNK / 256; ++it) {
    f32x2 l[4], p[4], m[4], r[4];
    Batch<T>::load(sl, it, lane, l);
    if (kPlus) Batch<T>::load(sp, it, lane, p);
    Batch<T>::load(sm, it, lane, m);
    if (SUMS & SUM_R) {
#pragma unroll
      for (int i = 0; i < 4; ++i) r[i] = fma2(beta2, sub2(p[i], m[i]), l[i]);
    }
    if (SUMS & SUM_L) exp_sum8(a.s2[Q_L], l, c2, a.nref2[Q_L]);
    if (SUMS & SUM_P) {
      if (POLY > 0) exp_sum8_mixed<POLY>(a.s2[Q_P], p, c2, a.nref2[Q_P], amax);
      else exp_sum8(a.s2[Q_P], p, c2, a.nref2[Q_P]);
    }
    if (SUMS & SUM_M) exp_sum8(a.s2[Q_M], m, c2, a.nref2[Q_M]);
    if (SUMS & SUM_R) exp_sum8(a.s2[Q_R], r, c2, a.nref2[Q_R]);
  }
  const float kBig = 1.329227995784916e36f;  // 2^120
  bool bad = false;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    float s0, s1;
    unpack2(a.s2[q], s0, s1);
    bad |= !(s0 + s1 < kBig);
  }
  if (POLY > 0) bad |= !(amax < 120.f);
  return !__any_sync(kFullMask, bad);
}

// ---- per-request epilogue: Eq. 6/7 and the accepted length ------------------------------------------
constexpr int kEpiWarps = 8;
constexpr int kEpiMaxRows = 64;  // rows of one request held in shared memory; more run in several rounds
constexpr int kFusedTailBytes = 8192;  // one-launch round: row results and sampling state at the start of the ring, chunk weights behind

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

// exp(x) in double for x <= 0 (about 1e-14 relative); 0 below the normal range.
__device__ __forceinline__ double exp_nonpos(double x) {
  const double y = x * 1.4426950408889634;
  if (!(y > -1000.0)) return (y != y) ? y : 0.0;
  const double k = rint(y), f = (y - k) * 0.6931471805599453;  // |f| <= 0.347
  double q = 1.0 / 39916800.0;
  q = fma(q, f, 1.0 / 3628800.0);
  q = fma(q, f, 1.0 / 362880.0);
  q = fma(q, f, 1.0 / 40320.0);
  q = fma(q, f, 1.0 / 5040.0);
  q = fma(q, f, 1.0 / 720.0);
  q = fma(q, f, 1.0 / 120.0);
  q = fma(q, f, 1.0 / 24.0);
  q = fma(q, f, 1.0 / 6.0);
  q = fma(q, f, 0.5);
  q = fma(q, f, 1.0);
  q = fma(q, f, 1.0);
  return __hiloint2double(__double2hiint(q) + ((int)k << 20), __double2loint(q));
}

// 2^d in double for an integer-valued d <= 0; 0 below 2^-1000.
__device__ __forceinline__ double pow2_nonpos_int_d(float d) {
  return (d < -1000.f) ? 0.0 : __hiloint2double(((int)d + 1023) << 20, 0);
}

// One warp: combine the partial records of `row` (exact power-of-two rescale, sums in double) and, for a
// drafted row, the log-probabilities, alpha and the accept decision.
template <typename T, bool PDL>
__device__ void epilogue_row(const RoundParams& p, int b, int t, int len, float beta, float lam, float c, int lane,
                             RowResult* out) {
  const int K = p.K, K1 = K + 1;
  const long long row = (long long)b * K1 + t;
  const float* rec = p.part + row * p.n_chunks * 8;
  // the drafted token's three logits: issued first so that their latency overlaps the record passes
  int y = -1;
  float gl = 0.f, gp = 0.f, gm = 0.f;
  if (t < len) {
    y = p.draft_tokens[(long long)b * K + t];
    if (p.n_shards == 0 && !p.tok_logits && y >= 0 && y < p.V) {
      const long long off = (long long)b * p.ld_req + (long long)t * p.ld_row + y;
      gl = load_logit<T>(reinterpret_cast<const T*>(p.h_llm), off);
      gm = load_logit<T>(reinterpret_cast<const T*>(p.h_minus), off);
      // Eq. 7 needs nothing of h_SLM+: when verification forms neither its normaliser nor the one of h_rec (the
      // two-phase round), that tensor is not touched on a drafted row at all
      if (p.sums & (SUM_P | SUM_R)) gp = load_logit<T>(reinterpret_cast<const T*>(p.h_plus), off);
    }
  }
  if (PDL) pdl_wait();  // everything above read inputs only; the records come from the streaming kernel
  if (p.tok_logits && y >= 0 && y < p.V) {  // fused LM-head path: the tensor-core pass left them in the workspace
    const float4 g = ld_cg_f4(p.tok_logits + row * 4);
    gl = g.x; gp = g.y; gm = g.z;
  }
  float M[4];
  double S[4];
  if (p.n_shards > 0) {
    // sharded vocabulary: lane g holds shard g's partial of this row; the token's logits come from its owner
    const bool have = lane < p.n_shards;
    ShardPartial sp;
    if (have) sp = p.shard_parts[((long long)lane * p.B + b) * K1 + t];
    float Ml[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) Ml[q] = have ? sp.m[q] : kNegInf;
    const float mine = warp_reduce4<true>(Ml, lane);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      M[q] = __shfl_sync(kFullMask, mine, 8 * q);
      double w = 0.0;
      if (have && sp.m[q] != kNegInf) w = (M[q] == -kNegInf) ? 0.0 : sp.s[q] * pow2_nonpos_int_d(sp.m[q] - M[q]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) w += __shfl_xor_sync(kFullMask, w, o);
      S[q] = w;
    }
    const unsigned owners = __ballot_sync(kFullMask, have && sp.has_token != 0);
    if (t < len && y >= 0 && y < p.vocab_total && owners) {
      const int src = __ffs(owners) - 1;
      gl = __shfl_sync(kFullMask, sp.tok_logit[0], src);
      gp = __shfl_sync(kFullMask, sp.tok_logit[1], src);
      gm = __shfl_sync(kFullMask, sp.tok_logit[2], src);
    } else if (t < len) {
      y = -1;   // outside the global vocabulary, or no shard delivered it
    }
  } else {
    row_sums_from_records(p, rec, lane, M, S);
  }
  // lanes 0..3 take the logarithm of one sum each, lane 4 that of lambda
  const double arg = lane == 0 ? S[0] : (lane == 1 ? S[1] : (lane == 2 ? S[2] : (lane == 3 ? S[3] : (double)lam)));
  const double lg = log2_pos(arg);
  RowResult r;
  bool fin = true;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    r.lse[q] = (double)M[q] + __shfl_sync(kFullMask, lg, q);
    if (p.sums & (1 << q)) fin = fin && isfinite(r.lse[q]);
  }
  const double ln2 = 0.6931471805599453;
  const double log_lam = __shfl_sync(kFullMask, lg, 4) * ln2;
  r.logz = (r.lse[Q_R] - r.lse[Q_L] - (double)beta * (r.lse[Q_P] - r.lse[Q_M])) * ln2;
  r.fin = fin; r.testable = 0; r.accept = 0; r.tok_ok = 0; r.alpha = 0.f;
  r.lp[0] = r.lp[1] = r.lp[2] = r.lp[3] = __int_as_float(0x7fc00000);
  if (lane == 0)
    *reinterpret_cast<float4*>(p.lse2 + row * 4) =
        make_float4((float)r.lse[0], (float)r.lse[1], (float)r.lse[2], (float)r.lse[3]);
  if (fin && t < len) {
    const long long i = (long long)b * K + t;
    if (y >= 0 && y < (p.n_shards > 0 ? p.vocab_total : p.V)) {
      const double cd = (double)c;
      const double l = (double)gl, pp = (double)gp, m = (double)gm;
      const double rr = l + (double)beta * (pp - m);  // Eq. 8
      const double lpL = (l * cd - r.lse[Q_L]) * ln2, lpP = (pp * cd - r.lse[Q_P]) * ln2,
                   lpM = (m * cd - r.lse[Q_M]) * ln2, lpS = (rr * cd - r.lse[Q_R]) * ln2;
      r.lp[Q_L] = (float)lpL; r.lp[Q_P] = (float)lpP; r.lp[Q_M] = (float)lpM; r.lp[Q_R] = (float)lpS;
      r.tok_ok = 1;
      const double logrho = (p.accept_mode == SPECSTEER_ACCEPT_RATIO) ? (lpL - lpM - log_lam)  // Eq. 7
                                                                      : (lpS - lpP);                    // Eq. 6
      if (!isnan(logrho)) {
        const double ald = exp_nonpos(fmin(0.0, logrho));
        r.alpha = (float)ald;
        r.testable = 1;
        r.accept = ((double)p.u_accept[i] <= ald) ? 1 : 0;  // "Uniform(0,1) <= alpha_t", decided in double
      }
    }
  }
  if (lane == 0) *out = r;
}

// The barrier of the NT threads that work on one request: the whole CTA (BAR = 0) or the named barrier BAR.
template <int BAR, int NT>
__device__ __forceinline__ void epi_sync() {
  if (BAR == 0) __syncthreads();
  else asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(NT) : "memory");
}

// One request, NT threads (tid = 0 .. NT - 1; res: kEpiMaxRows RowResults of shared memory): every warp combines
// the records of one row at a time, then the rows are scanned in order for accept_len and the status word.
template <typename T, int BAR, int NT, bool PDL>
__device__ __forceinline__ void request_epilogue(const RoundParams& p, int b, int tid, RowResult* res) {
  constexpr int NW = NT / 32;
  const int warp = tid >> 5, lane = tid & 31;
  const int K = p.K, K1 = K + 1;
  int status = 0;
  int len = p.draft_len[b];
  const float Tmp = p.temperature[b], lam = p.lambda[b], beta = p.beta[b];
  const bool params_ok = isfinite(Tmp) && Tmp > 0.f && isfinite(lam) && lam > 0.f && isfinite(beta);
  if (len < 0 || len > K) { status |= SPECSTEER_REQ_BAD_LEN; len = 0; }
  const bool bonus = (p.flags & SPECSTEER_FLAG_BONUS) != 0;
  const int R = params_ok ? len + ((bonus && p.row_mode != ROWS_DRAFTED) ? 1 : 0) : 0;  // rows with records
  const float c = kLog2e / Tmp;
  const float qnan = __int_as_float(0x7fc00000);

  for (int t = tid; t < K; t += NT) {
    const long long i = (long long)b * K + t;
    if (p.accept_flags) p.accept_flags[i] = 0;
    if (p.alpha) p.alpha[i] = 0.f;
    if (p.logp_llm) p.logp_llm[i] = qnan;
    if (p.logp_minus) p.logp_minus[i] = qnan;
    if (p.logp_plus) p.logp_plus[i] = qnan;
    if (p.logp_star) p.logp_star[i] = qnan;
  }
  for (int t = tid; t <= K; t += NT)
    if (p.log_z) p.log_z[(long long)b * K1 + t] = qnan;

  int n = len;
  bool decided = false;
  if (!params_ok) { status |= SPECSTEER_REQ_BAD_PARAM; n = 0; }
  for (int t0 = 0; t0 < R; t0 += kEpiMaxRows) {
    const int nr = min(kEpiMaxRows, R - t0);
    epi_sync<BAR, NT>();  // defaults written / previous round consumed
    for (int k = warp; k < nr; k += NW) epilogue_row<T, PDL>(p, b, t0 + k, len, beta, lam, c, lane, &res[k]);
    epi_sync<BAR, NT>();
    // outputs of these rows (any thread), then the sequential scan (every thread, same result)
    for (int k = tid; k < nr; k += NT) {
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

template <typename T>
__global__ void __launch_bounds__(kEpiWarps * 32) epilogue_kernel(const RoundParams p) {
  __shared__ RowResult res[kEpiMaxRows];
  pdl_launch_dependents();  // the recovery kernel may be set up behind this one
  request_epilogue<T, 0, kEpiWarps * 32, true>(p, blockIdx.x, threadIdx.x, res);
}

// The epilogue and the STEER recovery sample of a request in one CTA and one launch: the same device code as
// epilogue_kernel followed by recover_steer_kernel (the outputs are the same bits), without the second launch.
template <typename T, int TILE>
__global__ void __launch_bounds__(kEpiWarps * 32) epilogue_recover_kernel(const RoundParams p) {
  static_assert(kEpiWarps * 32 == kRecThreads, "one CTA shape serves both steps");
  extern __shared__ double cw[];  // [n_chunks] chunk weights of the recovery row
  __shared__ RowResult res[kEpiMaxRows];
  __shared__ PickShared sh;
  __shared__ double lse_fin[2];
  pdl_launch_dependents();
  request_epilogue<T, 0, kEpiWarps * 32, true>(p, blockIdx.x, threadIdx.x, res);
  __syncthreads();   // accept_len, the status word and the row normalisers of the request are written
  recover_steer_request<T, TILE, false, 0>(p, blockIdx.x, threadIdx.x, cw, sh, lse_fin);
}

// ---- the persistent streaming kernel --------------------------------------------------------------
// A tile is 2*CHUNK vocabulary entries of one used row, all three streams (three bulk copies, one stage).
// Warps [0, NCW) consume: warps 2k and 2k+1 share the tiles congruent to k modulo NCW/2 and each reduces
// one chunk (half) of the tile into its own partial record.  Warps [NCW, NCW+NPW) each run one elected
// producer thread that owns the stages congruent to its index modulo NPW (one thread cannot issue tiles
// fast enough for a whole SM).  Every stage is always consumed by the same pair of warps, so a waiting
// warp is never a whole barrier phase ahead of the data.
// FUSED (small rounds): the whole round in this one launch.  Every chunk that is retired is counted per request; the
// warp that retires a request's last chunk puts the request on its CTA's list, and when a CTA has streamed all its
// tiles its consumer warps run the epilogue and the recovery sample (STEER) of the requests on its list - the same
// device code the two stand-alone kernels run, so the outputs are the same bits.  Nobody waits for anybody: the
// counters are only ever incremented, and a request with no rows at all belongs to CTA (request mod grid).
template <typename T, int CHUNK, int STAGES, int NCW, int NPW, bool BULK, int SUMS, int POLY, bool FUSED>
__global__ void __launch_bounds__((NCW + NPW) * 32, 1) verify_kernel(const RoundParams p) {
  constexpr int TILE = 2 * CHUNK;
  constexpr bool kPlus = (SUMS & (SUM_P | SUM_R)) != 0;  // h_SLM+ is read at all
  constexpr int NPAIR = NCW / 2;
  static_assert(NCW % 2 == 0 && STAGES % NPAIR == 0, "each stage belongs to one fixed pair of consumer warps");
  static_assert(STAGES % NPW == 0, "each producer owns a fixed subset of the stages");
  extern __shared__ __align__(128) unsigned char smem_raw[];
  constexpr int NSLOT = kPlus ? 3 : 2;                   // streams held per stage
  constexpr int MSLOT = NSLOT - 1;                       // slot of h_SLM-
  constexpr int kStageBytes = NSLOT * TILE * (int)sizeof(T);
  T* tiles = reinterpret_cast<T*>(smem_raw);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw + (size_t)STAGES * kStageBytes);
  uint64_t* empty = full + STAGES;
  TileMeta* meta = reinterpret_cast<TileMeta*>(empty + STAGES);
  int* abort_flag = reinterpret_cast<int*>(meta + STAGES);
  int* row_start = abort_flag + 4;                                // [B + 1]
  float* beta_s = reinterpret_cast<float*>(row_start + p.B + 1);  // [B]
  float* c_s = beta_s + p.B;                                      // [B]  log2(e) / T_b
  float* ic_s = c_s + p.B;                                        // [B]  T_b / log2(e)
  int* first_s = reinterpret_cast<int*>(ic_s + p.B);              // [B]  first row of the request that is read
  int* todo = first_s + p.B;                                      // FUSED: [B] requests this CTA finishes, [B] = how many

  pdl_launch_dependents();  // the epilogue's CTAs may take over SMs as this grid's CTAs retire
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int nthreads = (NCW + NPW) * 32;
  const bool bonus = (p.flags & SPECSTEER_FLAG_BONUS) != 0;
  const int K = p.K;
  const int tiles_per_row = (p.V + TILE - 1) / TILE;

  // ---- prologue: barriers, per-request constants, and the prefix of used rows per request
  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 2); }
    *abort_flag = 0;
    row_start[0] = 0;
    if (FUSED) todo[p.B] = 0;
    fence_barrier_init();
  }
  for (int b = tid; b < p.B; b += nthreads) {
    int len = p.draft_len[b];
    if (len < 0 || len > K) len = 0;
    int cnt = len + (bonus ? 1 : 0), first = 0;
    if (p.row_mode == ROWS_DRAFTED) {
      cnt = len;
    } else if (p.row_mode == ROWS_RECOVERY) {   // the epilogue has run: one row for a request that samples
      const int n = p.accept_len[b];
      const bool bad = (p.status_ws[b] & (SPECSTEER_REQ_BAD_PARAM | SPECSTEER_REQ_NONFINITE)) != 0;
      cnt = (!bad && n >= 0 && n <= len && (n < len || bonus)) ? 1 : 0;
      first = n;
    }
    row_start[b + 1] = cnt;
    first_s[b] = first;
    beta_s[b] = p.beta[b];
    c_s[b] = kLog2e / p.temperature[b];
    ic_s[b] = p.temperature[b] * kLn2;
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
  const int total_tiles = row_start[p.B] * tiles_per_row;  // the host guarantees this fits in 31 bits
  const int cta = blockIdx.x, G = gridDim.x;
  if (FUSED) {   // a request that streams nothing still gets its epilogue (defaults, accept_len, status)
    for (int b = tid; b < p.B; b += nthreads)
      if (row_start[b + 1] == row_start[b] && b % G == cta) todo[atomicAdd(&todo[p.B], 1)] = b;
  }

  if (warp >= NCW) {
    // ================= producer warps =================
    const int pw = warp - NCW;
    const T* hl = reinterpret_cast<const T*>(p.h_llm);
    const T* hp = reinterpret_cast<const T*>(p.h_plus);
    const T* hm = reinterpret_cast<const T*>(p.h_minus);
    // tile g = cta + j*G  ->  (compact row cr, tile in row); advanced incrementally, no division in the loop
    const int g0 = cta + pw * G, gstep = NPW * G;
    const int step_rows = gstep / tiles_per_row, step_tiles = gstep % tiles_per_row;
    int cr = g0 / tiles_per_row, tr = g0 % tiles_per_row;
    int b = 0;
    const int K1 = K + 1;
    const float4 no_ref = make_float4(__int_as_float(0x7fc00000), 0.f, 0.f, 0.f);
    if (p.row_ref) pdl_wait();   // the row references come from the kernel launched just before this one
    if (BULK) {
      if (lane == 0) {  // one elected thread issues the bulk copies
        int issued = 0;
        const uint64_t stream_once = l2_policy_evict_first();   // the logits pass through L2 once and need not stay
        for (int j = pw, g = g0; g < total_tiles; j += NPW, g += gstep) {
          const int stage = j % STAGES;
          const uint32_t phase = (uint32_t)((j / STAGES) & 1);
          if (*reinterpret_cast<volatile int*>(abort_flag) || !mbar_wait(&empty[stage], phase ^ 1u, p.wait_cycles)) {
            *reinterpret_cast<volatile int*>(abort_flag) = 1;
            atomicExch(p.dev_error, 1);
            break;
          }
          while (row_start[b + 1] <= cr) ++b;  // cr < row_start[B], so b stays below B
          const int t = first_s[b] + cr - row_start[b];
          const int n_valid = min(TILE, p.V - tr * TILE);
          const long long off = (long long)b * p.ld_req + (long long)t * p.ld_row + (long long)tr * TILE;
          T* dst = tiles + (size_t)stage * NSLOT * TILE;
          TileMeta* mt = &meta[stage];
          mt->row = b * K1 + t; mt->tile = tr; mt->n_valid = n_valid;
          mt->beta = beta_s[b]; mt->c = c_s[b]; mt->inv_c = ic_s[b]; mt->req = b;
          // the row's reference exponents travel with the tile: a fourth bulk copy, 16 bytes, onto the same barrier
          const uint32_t ref_bytes = p.row_ref ? 16u : 0u;
          if (!p.row_ref) mt->ref[0] = no_ref.x;
          const int n_bulk = (int)(((size_t)n_valid * sizeof(T)) & ~(size_t)15) / (int)sizeof(T);
          for (int e = n_bulk; e < n_valid; ++e) {  // ragged end of the last tile: < 16 bytes per stream
            dst[e] = hl[off + e]; dst[MSLOT * TILE + e] = hm[off + e];
            if (kPlus) dst[TILE + e] = hp[off + e];
          }
          const uint32_t bytes = (uint32_t)(n_bulk * sizeof(T));
          if (bytes + ref_bytes) {
            mbar_arrive_expect_tx(&full[stage], (kPlus ? 3 : 2) * bytes + ref_bytes);
            if (ref_bytes) bulk_g2s(mt->ref, p.row_ref + 4ll * (b * K1 + t), 16u, &full[stage]);
          }
          if (bytes) {
            bulk_g2s(dst, hl + off, bytes, &full[stage], stream_once);
            if (kPlus) bulk_g2s(dst + TILE, hp + off, bytes, &full[stage], stream_once);
            bulk_g2s(dst + MSLOT * TILE, hm + off, bytes, &full[stage], stream_once);
          } else if (!ref_bytes) {
            mbar_arrive(&full[stage]);
          }
          ++issued;
          cr += step_rows; tr += step_tiles;
          if (tr >= tiles_per_row) { tr -= tiles_per_row; ++cr; }
        }
        // On an abort, copies already issued may still be landing: wait for them (bounded) before the CTA exits.
        if (*reinterpret_cast<volatile int*>(abort_flag)) {
          constexpr int kOwn = STAGES / NPW;
          const int first = issued > kOwn ? issued - kOwn : 0;
          for (int i = first; i < issued; ++i) {
            const int j = pw + i * NPW;
            mbar_wait(&full[j % STAGES], (uint32_t)((j / STAGES) & 1));
          }
        }
      }
    } else {
      // rows that are not 16-byte aligned: the warp copies element by element
      for (int j = pw, g = g0; g < total_tiles; j += NPW, g += gstep) {
        const int stage = j % STAGES;
        const uint32_t phase = (uint32_t)((j / STAGES) & 1);
        const bool ok = __all_sync(kFullMask, mbar_wait(&empty[stage], phase ^ 1u, p.wait_cycles));
        if (!ok || *reinterpret_cast<volatile int*>(abort_flag)) {
          if (lane == 0) { *reinterpret_cast<volatile int*>(abort_flag) = 1; atomicExch(p.dev_error, 1); }
          break;
        }
        while (row_start[b + 1] <= cr) ++b;
        const int t = first_s[b] + cr - row_start[b];
        const int n_valid = min(TILE, p.V - tr * TILE);
        const long long off = (long long)b * p.ld_req + (long long)t * p.ld_row + (long long)tr * TILE;
        T* dst = tiles + (size_t)stage * 3 * TILE;
        for (int e = lane; e < n_valid; e += 32) {
          dst[e] = hl[off + e]; dst[TILE + e] = hp[off + e]; dst[2 * TILE + e] = hm[off + e];
        }
        __syncwarp();
        if (lane == 0) {
          meta[stage] = TileMeta{{no_ref.x, 0.f, 0.f, 0.f}, b * K1 + t, tr, n_valid, beta_s[b], c_s[b], ic_s[b], b, 0};
          mbar_arrive(&full[stage]);
        }
        cr += step_rows; tr += step_tiles;
        if (tr >= tiles_per_row) { tr -= tiles_per_row; ++cr; }
      }
    }
  } else {
    // ================= consumer warps =================
    const int pair = warp >> 1, half = warp & 1;
    for (int j = pair, g = cta + pair * G; g < total_tiles; j += NPAIR, g += NPAIR * G) {
      const int stage = j % STAGES;
      const uint32_t phase = (uint32_t)((j / STAGES) & 1);
      // every lane observes the phase itself: that is what makes the copied bytes visible to it
      bool ok = !*reinterpret_cast<volatile int*>(abort_flag) && mbar_wait(&full[stage], phase, p.wait_cycles);
      ok = __all_sync(kFullMask, ok);
      if (!ok) {
        if (lane == 0) { *reinterpret_cast<volatile int*>(abort_flag) = 1; atomicExch(p.dev_error, 1); }
        break;
      }
      const TileMeta mt = meta[stage];
      const int nv = mt.n_valid - half * CHUNK;  // valid entries in this warp's chunk
      const T* sl = tiles + (size_t)stage * NSLOT * TILE + half * CHUNK;
      Acc a;
      if (nv >= CHUNK) {
        const bool fast = (mt.ref[0] == mt.ref[0])
            ? chunk_fast<T, CHUNK, SUMS, POLY, true>(a, sl, sl + TILE, sl + MSLOT * TILE, lane, mt.beta, mt.c, mt.inv_c, mt.ref)
            : chunk_fast<T, CHUNK, SUMS, POLY, false>(a, sl, sl + TILE, sl + MSLOT * TILE, lane, mt.beta, mt.c, mt.inv_c, mt.ref);
        if (!fast)
          chunk_pass<T, CHUNK, false, SUMS>(a, sl, sl + TILE, sl + MSLOT * TILE, lane, CHUNK, mt.beta, mt.c, mt.inv_c);
      } else if (nv > 0) chunk_pass<T, CHUNK, true, SUMS>(a, sl, sl + TILE, sl + MSLOT * TILE, lane, nv, mt.beta, mt.c, mt.inv_c);
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[stage]);  // the stage may be refilled while we reduce
      if (nv > 0) {
        float s4[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          float s0, s1;
          unpack2(a.s2[q], s0, s1);
          s4[q] = s0 + s1;
        }
        const float tot = warp_reduce4<false>(s4, lane);  // lanes [8q, 8q+8) hold the sum of normaliser q
        if ((lane & 7) == 0) {
          const int q = lane >> 3;
          const float rq = q == 0 ? a.ref[0] : (q == 1 ? a.ref[1] : (q == 2 ? a.ref[2] : a.ref[3]));
          // normalise to a sum in [1, 2): readers compare the exponents of different chunks and expect
          // the sums to be of order one (the fast path leaves them anywhere in the float32 range)
          float m_out = rq, s_out = tot;
          const unsigned bits = __float_as_uint(tot);
          const int ex = (int)((bits >> 23) & 0xffu);
          if (ex != 0 && ex != 255 && (bits >> 31) == 0) {
            m_out = rq + (float)(ex - 127);
            s_out = __uint_as_float((bits & 0x007fffffu) | 0x3f800000u);
          } else if (tot == 0.f) {
            m_out = kNegInf;
          }
          float* rec = p.part + ((long long)mt.row * p.n_chunks + (mt.tile * 2 + half)) * 8;
          *reinterpret_cast<float2*>(rec + 2 * q) = make_float2(m_out, s_out);
        }
        if (FUSED) {   // one more chunk of the request is in the workspace
          __threadfence();
          __syncwarp();
          if (lane == 0) {
            const int total = (row_start[mt.req + 1] - row_start[mt.req]) * p.n_chunks;
            if (atomicAdd(p.req_done + mt.req, 1) + 1 == total) {
              p.req_done[mt.req] = 0;   // nobody else touches it any more: left at zero for the next launch
              __threadfence();          // what the other CTAs wrote before they counted is visible from here on
              todo[atomicAdd(&todo[p.B], 1)] = mt.req;
            }
          }
        }
      }
    }
    if (FUSED) {
      // ---- the requests this CTA finishes: epilogue (Eq. 6 / 7, accept_len) and recovery sample (Eq. 8) ----
      constexpr int NT = NCW * 32;
      epi_sync<1, NT>();   // every consumer warp has read its last stage; the ring is free
      if (!*reinterpret_cast<volatile int*>(abort_flag)) {
        const int n_todo = *reinterpret_cast<volatile int*>(&todo[p.B]);
        RowResult* res = reinterpret_cast<RowResult*>(smem_raw);
        PickShared* psh = reinterpret_cast<PickShared*>(smem_raw + kEpiMaxRows * sizeof(RowResult));
        double* lse_fin = reinterpret_cast<double*>(smem_raw + kEpiMaxRows * sizeof(RowResult) + 256);
        double* cw = reinterpret_cast<double*>(smem_raw + kFusedTailBytes);
        for (int i = 0; i < n_todo; ++i) {
          const int b = todo[i];
          __threadfence();
          request_epilogue<T, 1, NT, false>(p, b, tid, res);
          epi_sync<1, NT>();   // accept_len, the status word and the row normalisers of the request are written
          if (tid < kRecThreads) recover_steer_request<T, CHUNK, false, 2>(p, b, tid, cw, *psh, lse_fin);
          epi_sync<1, NT>();   // the shared memory is reused by the next request
        }
      }
    }
  }
}

// ---- launch -------------------------------------------------------------------------------------------
template <typename T, int CHUNK, int STAGES, int NCW, int NPW, bool BULK, int SUMS, int POLY = 0, bool FUSED = false>
static cudaError_t launch_stream(const RoundParams& p, const LaunchInfo& li, cudaStream_t s) {
  const size_t ring = (size_t)STAGES * ((SUMS & (SUM_P | SUM_R)) ? 3 : 2) * 2 * CHUNK * sizeof(T);
  const size_t fixed = ring + 2 * STAGES * sizeof(uint64_t) + STAGES * sizeof(TileMeta) + 16;
  const size_t smem = fixed + (size_t)(6 * p.B + 2) * sizeof(int);
  if (FUSED && (size_t)kFusedTailBytes + (size_t)p.n_chunks * sizeof(double) > ring) return cudaErrorInvalidValue;
  auto kern = verify_kernel<T, CHUNK, STAGES, NCW, NPW, BULK, SUMS, POLY, FUSED>;
  // per instantiation and device; sized for the largest slab.  Contexts may be driven from different host threads:
  // the flag is atomic, and two threads that both find it clear merely set the same attribute twice.
  static std::atomic<bool> attr_set_dev[64];
  std::atomic<bool>& attr_set = attr_set_dev[li.device & 63];
  if (!attr_set.load(std::memory_order_acquire)) {
    const size_t smem_max = fixed + (size_t)(6 * kMaxSlabB + 2) * sizeof(int);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max);
    if (e != cudaSuccess) return e;
    attr_set.store(true, std::memory_order_release);
  }
  if (!p.row_ref) {
    kern<<<li.sm_count, (NCW + NPW) * 32, smem, s>>>(p);
    return cudaGetLastError();
  }
  // The row references were written by row_ref_kernel, launched just before on the same stream: this kernel may
  // start while that one drains (its producers wait for it before they read a reference).
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(li.sm_count);
  cfg.blockDim = dim3((NCW + NPW) * 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, p);
}

// ---- reference exponents per row ------------------------------------------------------------------------
// One thread per row (b, t) that will be streamed: the row's pivot is its drafted token (for the row a recovery pass
// streams: the token that was rejected there), which was drawn from Softmax(h_SLM+ / T) and therefore sits near the
// top of the row in all three tensors.  The references are kBias binades above the pivot's scaled logits, so a chunk
// overflows the fast path only if it holds an entry 2^(kBias + 120) above the pivot - with per-chunk references it
// is the first 256 entries of every chunk that have to be representative, which heavy-tailed rows at low
// temperature are not.  A row without a usable pivot (the bonus row, a bad token, non-finite logits) gets NaN and
// its chunks fall back to their own first batch.
template <typename T>
__global__ void __launch_bounds__(128) row_ref_kernel(const RoundParams p, float4* out) {
  pdl_launch_dependents();
  const int K = p.K, K1 = K + 1;
  const int row = blockIdx.x * 128 + threadIdx.x;
  if (row >= p.B * K1) return;
  const int b = row / K1, t = row - b * K1;
  float4 ref = make_float4(__int_as_float(0x7fc00000), 0.f, 0.f, 0.f);
  int len = p.draft_len[b];
  if (len < 0 || len > K) len = 0;
  const float Tmp = p.temperature[b], beta = p.beta[b];
  if (t < len && Tmp > 0.f) {
    const int y = p.draft_tokens[(long long)b * K + t];
    if (y >= 0 && y < p.V) {
      const long long off = (long long)b * p.ld_req + (long long)t * p.ld_row + y;
      const float l = load_logit<T>(reinterpret_cast<const T*>(p.h_llm), off);
      const float m = load_logit<T>(reinterpret_cast<const T*>(p.h_minus), off);
      // the two-phase verification never touches h_SLM+ on a drafted row
      const float pp = (p.sums & (SUM_P | SUM_R)) ? load_logit<T>(reinterpret_cast<const T*>(p.h_plus), off) : l;
      const float c = kLog2e / Tmp;
      const float4 cand = make_float4(ceilf(l * c) + kBias, ceilf(pp * c) + kBias, ceilf(m * c) + kBias,
                                      ceilf(fmaf(beta, pp - m, l) * c) + kBias);
      const float big = 1e30f;
      if (fabsf(cand.x) < big && fabsf(cand.y) < big && fabsf(cand.z) < big && fabsf(cand.w) < big) ref = cand;
    }
  }
  out[row] = ref;
}

cudaError_t launch_row_ref(const RoundParams& p, int dtype, cudaStream_t s) {
  const int rows = p.B * (p.K + 1);
  if (rows == 0 || !p.row_ref) return cudaSuccess;
  float4* out = reinterpret_cast<float4*>(p.row_ref);
  if (dtype == SPECSTEER_F32) row_ref_kernel<float><<<(rows + 127) / 128, 128, 0, s>>>(p, out);
  else row_ref_kernel<uint16_t><<<(rows + 127) / 128, 128, 0, s>>>(p, out);
  return cudaGetLastError();
}

// ---- vocabulary-sharded path: this shard's view of every row ---------------------------------------
template <typename T>
__global__ void __launch_bounds__(kEpiWarps * 32) shard_rows_kernel(const RoundParams p, ShardPartial* out) {
  const int b = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int K = p.K, K1 = K + 1;
  int len = p.draft_len[b];
  if (len < 0 || len > K) len = 0;
  const int R = len + ((p.flags & SPECSTEER_FLAG_BONUS) ? 1 : 0);
  pdl_wait();
  for (int t = warp; t <= K; t += kEpiWarps) {
    ShardPartial sp;
#pragma unroll
    for (int q = 0; q < 4; ++q) { sp.m[q] = kNegInf; sp.s[q] = 0.0; }
    sp.tok_logit[0] = sp.tok_logit[1] = sp.tok_logit[2] = 0.f;
    sp.has_token = 0;
    if (t < R) {
      const long long row = (long long)b * K1 + t;
      float M[4];
      double S[4];
      row_sums_from_records(p, p.part + row * p.n_chunks * 8, lane, M, S);
#pragma unroll
      for (int q = 0; q < 4; ++q) { sp.m[q] = M[q]; sp.s[q] = S[q]; }
      if (t < len) {
        const int y = p.draft_tokens[(long long)b * K + t] - p.vocab_offset;   // id within this shard
        if (p.tok_logits) {   // fused LM heads: the tensor-core pass left the token's logits, if it met the token
          const float4 g = ld_cg_f4(p.tok_logits + row * 4);
          if (y >= 0 && y < p.V && __float_as_uint(g.w) != 0u) {
            sp.tok_logit[0] = g.x; sp.tok_logit[1] = g.y; sp.tok_logit[2] = g.z;
            sp.has_token = 1;
          }
        } else if (y >= 0 && y < p.V) {
          const long long off = (long long)b * p.ld_req + (long long)t * p.ld_row + y;
          sp.tok_logit[0] = load_logit<T>(reinterpret_cast<const T*>(p.h_llm), off);
          sp.tok_logit[1] = load_logit<T>(reinterpret_cast<const T*>(p.h_plus), off);
          sp.tok_logit[2] = load_logit<T>(reinterpret_cast<const T*>(p.h_minus), off);
          sp.has_token = 1;
        }
      }
    }
    if (lane == 0) out[(long long)b * K1 + t] = sp;
  }
}

cudaError_t launch_shard_rows(const RoundParams& p, int dtype, ShardPartial* out, cudaStream_t s) {
  if (dtype == SPECSTEER_F32) shard_rows_kernel<float><<<p.B, kEpiWarps * 32, 0, s>>>(p, out);
  else shard_rows_kernel<uint16_t><<<p.B, kEpiWarps * 32, 0, s>>>(p, out);
  return cudaGetLastError();
}

cudaError_t launch_verify_stream(const RoundParams& p, int dtype, bool aligned, const LaunchInfo& li, cudaStream_t s) {
  // Ring shape per logit type, from sweeps on the two largest benchmark shapes: float32 is bound by memory and
  // runs best with 144 KB in flight (12 stages, 6 consumer pairs, 3 producers: 0.350 ms against 0.379 ms for
  // 16/16/4 on 2.33 GB); 16-bit logits need the arithmetic of 8 pairs and 4 producers (12/12/3 is 12 % slower).
  // the three sets of normalisers that occur: all four; without h_SLM+'s; h_LLM and h_SLM- alone (then the
  // h_SLM+ tensor is not read at all).  Rows that are not 16-byte aligned always take the full set.
  constexpr int kNoPlus = SUM_L | SUM_M | SUM_R, kRatio = SUM_L | SUM_M;
  const int sums = !aligned ? SUM_ALL : ((p.sums & SUM_P) ? SUM_ALL : ((p.sums & SUM_R) ? kNoPlus : kRatio));
  if (dtype == SPECSTEER_F32) {
    if (!aligned) return launch_stream<float, kChunkF32, 16, 16, 4, false, SUM_ALL>(p, li, s);
    if (sums == SUM_ALL) return launch_stream<float, kChunkF32, 12, 12, 3, true, SUM_ALL>(p, li, s);
    if (sums == kNoPlus) return launch_stream<float, kChunkF32, 12, 12, 3, true, kNoPlus>(p, li, s);
    return launch_stream<float, kChunkRatioF32, 12, 12, 3, true, kRatio>(p, li, s);
  }
  if (!aligned) return launch_stream<uint16_t, kChunkBF16, 16, 16, 4, false, SUM_ALL>(p, li, s);
  // 16-bit logits with all four normalisers are bound by the special-function unit: under the ratio rule, where the
  // normaliser of h_SLM+ decides nothing, three of its four pairs per batch take the cubic (5574 against 5274 GB/s
  // on the largest benchmark shape; one, two and four pairs gave 5363, 5512 and 5500)
  if (sums == SUM_ALL && p.accept_mode == SPECSTEER_ACCEPT_RATIO)
    return launch_stream<uint16_t, kChunkBF16, 16, 16, 4, true, SUM_ALL, 3>(p, li, s);
  if (sums == SUM_ALL) return launch_stream<uint16_t, kChunkBF16, 16, 16, 4, true, SUM_ALL>(p, li, s);
  if (sums == kNoPlus) return launch_stream<uint16_t, kChunkBF16, 16, 16, 4, true, kNoPlus>(p, li, s);
  return launch_stream<uint16_t, kChunkRatioBF16, 16, 16, 4, true, kRatio>(p, li, s);
}

// The whole round of a small batch in one launch (ROWS_ALL, STEER recovery, 16-byte aligned rows): see verify_kernel.
bool fused_round_fits(const RoundParams& p, int dtype) {
  // the chunk weights of one row share the ring with the row results (see launch_stream)
  const size_t ring = dtype == SPECSTEER_F32 ? (size_t)12 * 3 * 2 * kChunkF32 * 4 : (size_t)16 * 3 * 2 * kChunkBF16 * 2;
  return (size_t)kFusedTailBytes + (size_t)p.n_chunks * sizeof(double) <= ring;
}

cudaError_t launch_verify_fused(const RoundParams& p, int dtype, const LaunchInfo& li, cudaStream_t s) {
  constexpr int kNoPlus = SUM_L | SUM_M | SUM_R;
  const bool all = (p.sums & SUM_P) != 0;
  if (dtype == SPECSTEER_F32) {
    if (all) return launch_stream<float, kChunkF32, 12, 12, 3, true, SUM_ALL, 0, true>(p, li, s);
    return launch_stream<float, kChunkF32, 12, 12, 3, true, kNoPlus, 0, true>(p, li, s);
  }
  if (all && p.accept_mode == SPECSTEER_ACCEPT_RATIO)
    return launch_stream<uint16_t, kChunkBF16, 16, 16, 4, true, SUM_ALL, 3, true>(p, li, s);
  if (all) return launch_stream<uint16_t, kChunkBF16, 16, 16, 4, true, SUM_ALL, 0, true>(p, li, s);
  return launch_stream<uint16_t, kChunkBF16, 16, 16, 4, true, kNoPlus, 0, true>(p, li, s);
}

cudaError_t launch_epilogue(const RoundParams& p, int dtype, cudaStream_t s, bool with_recover) {
  // programmatic dependent launch: the epilogue reads its inputs while the kernel before it drains
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.B);
  cfg.blockDim = dim3(kEpiWarps * 32);
  cfg.dynamicSmemBytes = with_recover ? (size_t)p.n_chunks * sizeof(double) : 0;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (with_recover) {
    if (dtype == SPECSTEER_F32) return cudaLaunchKernelEx(&cfg, epilogue_recover_kernel<float, kChunkF32>, p);
    return cudaLaunchKernelEx(&cfg, epilogue_recover_kernel<uint16_t, kChunkBF16>, p);
  }
  if (dtype == SPECSTEER_F32) return cudaLaunchKernelEx(&cfg, epilogue_kernel<float>, p);
  return cudaLaunchKernelEx(&cfg, epilogue_kernel<uint16_t>, p);
}

cudaError_t launch_verify(const RoundParams& p, int dtype, bool aligned, const LaunchInfo& li, cudaStream_t s,
                          int* n_launches, cudaEvent_t ev_begin, cudaEvent_t ev_end, bool with_recover) {
  *n_launches = 2;
  cudaError_t e;
  if (p.row_ref) {
    if ((e = launch_row_ref(p, dtype, s)) != cudaSuccess) return e;
    *n_launches = 3;
  }
  if (ev_begin && (e = cudaEventRecord(ev_begin, s)) != cudaSuccess) return e;
  if ((e = launch_verify_stream(p, dtype, aligned, li, s)) != cudaSuccess) return e;
  if (ev_end && (e = cudaEventRecord(ev_end, s)) != cudaSuccess) return e;
  return launch_epilogue(p, dtype, s, with_recover);
}

}  // namespace specsteer
