// Partial records {exponent, sum} of a row and their combination; shared by the kernels that read them.
#pragma once
#include "common.cuh"
#include "internal.h"

namespace specsteer {

// Reduce four per-lane values over the warp at once (22 instructions instead of 40): after the first
// two exchange steps each lane carries one of the four quantities.  On return lanes [8q, 8q+8) hold the
// reduction of v[q] in the return value.
template <bool IS_MAX>
__device__ __forceinline__ float warp_reduce4(const float (&v)[4], int lane) {
  const bool hi16 = (lane & 16) != 0, hi8 = (lane & 8) != 0;
  const float keep_a = hi16 ? v[2] : v[0], keep_b = hi16 ? v[3] : v[1];
  const float send_a = hi16 ? v[0] : v[2], send_b = hi16 ? v[1] : v[3];
  const float xa = __shfl_xor_sync(kFullMask, send_a, 16), xb = __shfl_xor_sync(kFullMask, send_b, 16);
  const float ra = IS_MAX ? fmaxf(keep_a, xa) : keep_a + xa;
  const float rb = IS_MAX ? fmaxf(keep_b, xb) : keep_b + xb;
  const float keep = hi8 ? rb : ra, send = hi8 ? ra : rb;
  const float x = __shfl_xor_sync(kFullMask, send, 8);
  float r = IS_MAX ? fmaxf(keep, x) : keep + x;
#pragma unroll
  for (int o = 4; o > 0; o >>= 1) {
    const float y = __shfl_xor_sync(kFullMask, r, o);
    r = IS_MAX ? fmaxf(r, y) : r + y;
  }
  return r;
}

// 2^d for an integer-valued d <= 0 (exact); 0 below the normal range.
__device__ __forceinline__ float pow2_nonpos_int(float d) {
  return (d < -126.f) ? 0.f : __int_as_float(((int)d + 127) << 23);
}

// log2(x) in double for x > 0 (about 1e-12 absolute): exponent plus the atanh series of the mantissa
// folded into [sqrt(1/2), sqrt(2)).  Short on purpose: the library routine costs several times the
// instructions and every warp of the epilogue is latency-bound.  x = 0 gives -inf, x = +inf gives +inf,
// negative or NaN gives NaN; subnormal inputs do not occur here (sums of float32 values >= 1, or 0).
__device__ __forceinline__ double log2_pos(double x) {
  if (!(x > 0.0)) return (x == 0.0) ? -__longlong_as_double(0x7ff0000000000000ll) : __longlong_as_double(0x7ff8000000000000ll);
  const int hi = __double2hiint(x), lo = __double2loint(x);
  if (hi >= 0x7ff00000) return x;  // +inf
  int e = (hi >> 20) - 1023;
  double m = __hiloint2double((hi & 0x000fffff) | 0x3ff00000, lo);  // [1, 2)
  if (m > 1.4142135623730951) { m *= 0.5; e += 1; }
  const double z = (m - 1.0) / (m + 1.0), w = z * z;
  double q = 1.0 / 13.0;
  q = fma(q, w, 1.0 / 11.0);
  q = fma(q, w, 1.0 / 9.0);
  q = fma(q, w, 1.0 / 7.0);
  q = fma(q, w, 1.0 / 5.0);
  q = fma(q, w, 1.0 / 3.0);
  q = fma(q, w, 1.0);
  return fma(z * q, 2.8853900817779268 /* 2/ln 2 */, (double)e);
}

// One warp: the largest exponent per normaliser over the row's records and the float64 sums relative to it
// (read through L2: in the one-launch round the records come from other SMs of the same kernel); every lane gets the
// results.
__device__ __forceinline__ void row_sums_from_records(const RoundParams& p, const float* rec, int lane, float (&M)[4],
                                                      double (&S)[4]) {
  float Ml[4] = {kNegInf, kNegInf, kNegInf, kNegInf};
#pragma unroll 4
  for (int ch = lane; ch < p.n_chunks; ch += 32) {
    const float4 x = __ldcg(reinterpret_cast<const float4*>(rec + ch * 8));
    const float4 z = __ldcg(reinterpret_cast<const float4*>(rec + ch * 8 + 4));
    Ml[0] = fmaxf(Ml[0], x.x); Ml[1] = fmaxf(Ml[1], x.z); Ml[2] = fmaxf(Ml[2], z.x); Ml[3] = fmaxf(Ml[3], z.z);
  }
  const float mine = warp_reduce4<true>(Ml, lane);
#pragma unroll
  for (int q = 0; q < 4; ++q) { M[q] = __shfl_sync(kFullMask, mine, 8 * q); S[q] = 0.0; }
#pragma unroll 4
  for (int ch = lane; ch < p.n_chunks; ch += 32) {
    const float4 x = __ldcg(reinterpret_cast<const float4*>(rec + ch * 8));
    const float4 z = __ldcg(reinterpret_cast<const float4*>(rec + ch * 8 + 4));
    const float mm[4] = {x.x, x.z, z.x, z.z}, ss[4] = {x.y, x.w, z.y, z.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float w = ss[q];
      if (mm[q] != M[q]) w = (mm[q] == kNegInf || M[q] == -kNegInf) ? 0.f : w * pow2_nonpos_int(mm[q] - M[q]);
      S[q] += (double)w;
    }
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) S[q] += __shfl_xor_sync(kFullMask, S[q], o);
  }
}

}  // namespace specsteer
