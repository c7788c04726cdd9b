// Device-side helpers shared by the verify and recover kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace specsteer {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kNegInf = -__builtin_huge_valf();
constexpr unsigned kFullMask = 0xffffffffu;

// Record layout of one (row, chunk) partial: reference exponent and scaled sum for the four
// normalisers, all in the base-2 domain (value = s * 2^m).
enum { Q_L = 0, Q_P = 1, Q_M = 2, Q_R = 3 };

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ float max8(const float (&v)[8]) {
  return fmaxf(max3(max3(v[0], v[1], v[2]), max3(v[3], v[4], v[5]), v[6]), v[7]);
}

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <typename T> __device__ __forceinline__ float load_logit(const T* p, long long i);
template <> __device__ __forceinline__ float load_logit<float>(const float* p, long long i) { return __ldg(p + i); }
template <> __device__ __forceinline__ float load_logit<uint16_t>(const uint16_t* p, long long i) {
  return __uint_as_float(((uint32_t)__ldg(p + i)) << 16);
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFullMask, v, o));
  return v;
}
// The maximum over the warp in one instruction (sm_100a); NaN inputs are ignored like fmaxf ignores them.
__device__ __forceinline__ float warp_max_redux(float v) {
  float r;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
  return r;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFullMask, v, o);
  return v;
}

// ---- 64-bit selection keys: larger value first, among equal values the lower vocabulary id first ----------
typedef unsigned long long u64;
__device__ __forceinline__ uint32_t order_key(float h) {   // unsigned order = float order
  const uint32_t b = __float_as_uint(h);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float order_val(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
__device__ __forceinline__ u64 entry_key(float h, int idx) {
  return ((u64)order_key(h) << 32) | (u64)(0xffffffffu - (uint32_t)idx);
}

// ---- shared-memory barriers and bulk (TMA) copies -------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// One poll of the barrier's phase.  The thread may be suspended by the hardware for up to `hint_ns`
// nanoseconds (it is woken as soon as the phase completes), so a waiting warp issues few instructions.
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity, uint32_t hint_ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns)
      : "memory");
  return ok != 0;
}
// The phase test that never blocks.
__device__ __forceinline__ bool mbar_test_nonblocking(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up once `limit` SM clocks have passed (default: a few seconds) and returns false; the caller
// then records an error and unwinds.  The blocking form of the test may keep a thread suspended for longer than any
// hint says, so a limit of a few thousand clocks or less (the give-up path under test) polls with the form that
// never blocks: such a wait ends within its limit whatever the barrier does.
constexpr long long kWaitCycles = 1ll << 33;
constexpr uint32_t kSuspendNs = 2000;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, long long limit = kWaitCycles) {
  if (limit < 8192) {
    const long long t0 = clock64();
    for (;;) {
      if (mbar_test_nonblocking(bar, parity)) return true;
      if (clock64() - t0 > limit) return false;
    }
  }
  if (mbar_test(bar, parity, kSuspendNs)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_test(bar, parity, kSuspendNs)) return true;
    if (clock64() - t0 > limit) return false;
  }
}
// 1-D bulk copy global -> shared of this CTA alone, completion counted in bytes on `bar`.
// Both addresses must be 16-byte aligned and `bytes` a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// The same with an L2 eviction policy for the lines the copy reads (createpolicy).  The logits are read exactly once:
// marked evict-first they no longer push the partial records, the row normalisers and the next launch's small inputs
// out of L2 (measured on the two large benchmark shapes: rounds 1.1 % and 4.7 % shorter).
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar, uint64_t l2_policy) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(l2_policy)
               : "memory");
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

// Programmatic dependent launch: a kernel launched with the programmatic-serialisation attribute may start
// while the previous kernel of the stream is still running once every CTA of that kernel has called
// pdl_launch_dependents() (or exited); it must call pdl_wait() before it touches anything the previous
// kernel wrote.  Without the attribute both are no-ops.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// loads that must observe other SMs' writes (workspace written earlier in the same kernel)
__device__ __forceinline__ float4 ld_cg_f4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

}  // namespace specsteer
