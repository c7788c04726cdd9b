// The LM heads fused in front of the round (Algorithm 1: the logits h_LLM, h_SLM+, h_SLM- that the verification
// and recovery steps read are h = x W^T of the three forward passes).  The logits are formed on the tensor cores,
// tile by tile, into tensor memory, reduced there to the same per-chunk partial records the streaming kernel
// writes, and never stored: the epilogue kernel and the recovery step work from the records.
//
//   lmhead_kernel          persistent; per tile of 128 rows x 128 vocabulary entries three accumulators (h_LLM,
//                          h_SLM+, h_SLM-) of 128 columns each in tensor memory.  Warp 0 issues the TMA loads of
//                          the operand tiles (128-byte swizzle), warp 1 issues tcgen05.mma, warps 2..5 read the
//                          accumulators back (one row per thread) and write the partial record of the chunk and,
//                          where the drafted token falls into the tile, its three logits.
//   lmhead_recover_kernel  one CTA per request: places the CDF target in a chunk from the records, recomputes the
//                          128 logits of that chunk on the CUDA cores and samples within it (Eq. 8).
#include <cuda.h>

#include <atomic>

#include "common.cuh"
#include "internal.h"
#include "specsteer.h"

namespace specsteer {

namespace {

constexpr int kBM = kLmheadChunk;  // rows of hidden states per tile = lanes of tensor memory
constexpr int kBN = kLmheadChunk;  // vocabulary entries per tile = one partial record
constexpr int kBK = 64;            // hidden entries per stage: 128 bytes of bf16, one swizzle row
constexpr int kUmmaK = 16;         // hidden entries per tcgen05.mma of kind::f16
constexpr int kTileBytes = kBM * kBK * 2;   // 16 KB, one operand tile
// The operand ring is made of groups of four tiles.  A group holds either two steps of one product ({x, W} twice) or
// one step of both Specialist products when they share a head ({x+, x-, W}).  Each step has its own "full" barrier,
// the group one "empty" barrier: one tcgen05.commit per group (a commit costs about as much as an MMA).
constexpr int kGroups = 3;
constexpr int kGroupBytes = 4 * kTileBytes;
constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 512;         // 4 accumulators of 128 columns: {L even, P, M, L odd}
constexpr int kSmemBytes = kGroups * kGroupBytes + 1024 /* alignment */ + 512 /* barriers */;

struct LmKernelParams {
  int R, V, K, d_llm, d_slm, n_chunks;
  int shared_head;    // h_SLM+ and h_SLM- use the same head: its tile is loaded once for both products
  int vocab_offset;   // the heads passed are rows [vocab_offset, vocab_offset + V) of the full heads (0 if whole)
  const int* draft_tokens;
  const int* draft_len;
  const float* beta;
  const float* temperature;
  float* part;        // [R][n_chunks][8]
  float* tok_logits;  // [R][4]: the drafted token's h_LLM, h_SLM+, h_SLM- and a "token met" word
  u64* argmax_keys;   // [R][n_chunks]: per tile the key of the largest h_rec (greedy recovery), or null
  int* dev_error;
};

// ---- PTX wrappers ---------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(tm), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem] * B[smem]^T, both operands K-major bf16, float32 accumulation
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// the barrier receives one arrival once every tcgen05.mma issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// 32 consecutive columns of this warp's 32 lanes of tensor memory, one row per thread
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 operand tile laid out by TMA with the 128-byte swizzle: rows of
// 128 bytes, groups of 8 rows 1024 bytes apart (stride offset), leading offset unused (1), descriptor version 1,
// layout type 2 (128-byte swizzle).  Addresses and offsets are in units of 16 bytes.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
// Instruction descriptor of kind::f16: float32 accumulator, bf16 A and B, both K-major, N and M of the tile.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);

struct LmShared {
  uint64_t full[kGroups][2], empty[kGroups];
  uint64_t tmem_full, tmem_empty, drain;
  uint32_t tmem_slot;
  int abort_flag;
};

__device__ __forceinline__ bool aborted(const LmShared* sh) { return *reinterpret_cast<const volatile int*>(&sh->abort_flag) != 0; }
__device__ __forceinline__ void set_abort(LmShared* sh, int* dev_error) {
  *reinterpret_cast<volatile int*>(&sh->abort_flag) = 1;
  atomicExch(dev_error, 1);
}

// One slice of 32 columns of the three accumulators: running maxima of the four scaled quantities.
template <bool MASKED>
__device__ __forceinline__ void slice_max(const uint32_t (&L)[32], const uint32_t (&P)[32], const uint32_t (&M)[32], float beta,
                                          int nv, float (&mx)[4], int jbase, int& arg_r) {
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    if (MASKED && j >= nv) break;
    const float l = __uint_as_float(L[j]), p = __uint_as_float(P[j]), m = __uint_as_float(M[j]);
    const float r = fmaf(beta, p - m, l);  // Eq. 8
    mx[Q_L] = fmaxf(mx[Q_L], l); mx[Q_P] = fmaxf(mx[Q_P], p); mx[Q_M] = fmaxf(mx[Q_M], m);
    if (r > mx[Q_R]) { mx[Q_R] = r; arg_r = jbase + j; }   // ascending columns: the first maximiser stays
  }
}
template <bool MASKED>
__device__ __forceinline__ void slice_sum(const uint32_t (&L)[32], const uint32_t (&P)[32], const uint32_t (&M)[32], float beta,
                                          float c, const float (&nref)[4], int nv, float (&s)[4]) {
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    if (MASKED && j >= nv) break;
    const float l = __uint_as_float(L[j]), p = __uint_as_float(P[j]), m = __uint_as_float(M[j]);
    const float r = fmaf(beta, p - m, l);
    s[Q_L] += ex2(fmaf(l, c, nref[Q_L])); s[Q_P] += ex2(fmaf(p, c, nref[Q_P]));
    s[Q_M] += ex2(fmaf(m, c, nref[Q_M])); s[Q_R] += ex2(fmaf(r, c, nref[Q_R]));
  }
}

// A partial record {m, s} with value s * 2^m: s in [1, 2) and m integer-valued, or m = -inf for an empty sum;
// a non-finite sum is passed on as it is.
__device__ __forceinline__ float2 make_record(float ref, float tot) {
  float m_out = ref, s_out = tot;
  const unsigned bits = __float_as_uint(tot);
  const int ex = (int)((bits >> 23) & 0xffu);
  if (ex != 0 && ex != 255 && (bits >> 31) == 0) {
    m_out = ref + (float)(ex - 127);
    s_out = __uint_as_float((bits & 0x007fffffu) | 0x3f800000u);
  } else if (tot == 0.f) {
    m_out = kNegInf;
  }
  return make_float2(m_out, s_out);
}

__global__ void __launch_bounds__(kThreads, 1)
lmhead_kernel(const __grid_constant__ CUtensorMap tm_xl, const __grid_constant__ CUtensorMap tm_wl,
              const __grid_constant__ CUtensorMap tm_xp, const __grid_constant__ CUtensorMap tm_wp,
              const __grid_constant__ CUtensorMap tm_xm, const __grid_constant__ CUtensorMap tm_wm, const LmKernelParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;  // operand tiles need 1024-byte alignment
  LmShared* sh = reinterpret_cast<LmShared*>(smem_raw + (smem0 - smem_u32(smem_raw)) + kGroups * kGroupBytes);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int mb_count = (p.R + kBM - 1) / kBM, nb_count = (p.V + kBN - 1) / kBN;
  const int n_tiles = mb_count * nb_count;
  const int nkL = (p.d_llm + kBK - 1) / kBK, nkS = (p.d_slm + kBK - 1) / kBK;

  if (tid == 0) {
    for (int s = 0; s < kGroups; ++s) { mbar_init(&sh->full[s][0], 1); mbar_init(&sh->full[s][1], 1); mbar_init(&sh->empty[s], 1); }
    mbar_init(&sh->tmem_full, 1);
    mbar_init(&sh->tmem_empty, 4);
    mbar_init(&sh->drain, 1);
    sh->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(&sh->tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&sh->tmem_slot);

  if (warp == 0) {
    // ================= TMA producer =================
    if (lane == 0) {
      int grp = 0;  // groups issued so far: group i lives in slot i % kGroups
      bool ok = true;
      uint32_t base = 0;
      int gs = 0;
      auto begin_group = [&]() {
        gs = grp % kGroups;
        const uint32_t ph = (uint32_t)((grp / kGroups) & 1);
        if (aborted(sh) || !mbar_wait(&sh->empty[gs], ph ^ 1u)) { set_abort(sh, p.dev_error); ok = false; return; }
        base = smem0 + gs * kGroupBytes;
        ++grp;
      };
      // two steps of x W^T (the second one missing at an odd end): tiles {x, W, x, W}
      auto pair_steps = [&](const CUtensorMap* ta, const CUtensorMap* tb, int m0, int n0, int nk) {
        for (int kb = 0; kb < nk && ok; kb += 2) {
          begin_group();
          if (!ok) break;
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            if (kb + j < nk) {
              mbar_arrive_expect_tx(&sh->full[gs][j], 2 * kTileBytes);
              tma_load_2d(base + j * 2 * kTileBytes, ta, (kb + j) * kBK, m0, &sh->full[gs][j]);
              tma_load_2d(base + j * 2 * kTileBytes + kTileBytes, tb, (kb + j) * kBK, n0, &sh->full[gs][j]);
            } else {
              mbar_arrive(&sh->full[gs][j]);  // unused this time: keep its phase in step with the group's
            }
          }
        }
      };
      for (int g = blockIdx.x; g < n_tiles && ok; g += gridDim.x) {
        const int mb = g % mb_count, nb = g / mb_count;  // row blocks fastest: CTAs running together share W tiles in L2
        const int m0 = mb * kBM, n0 = nb * kBN;
        pair_steps(&tm_xl, &tm_wl, m0, n0, nkL);
        if (p.shared_head) {
          for (int kb = 0; kb < nkS && ok; ++kb) {   // one step of both products: tiles {x+, x-, W}
            begin_group();
            if (!ok) break;
            mbar_arrive_expect_tx(&sh->full[gs][0], 3 * kTileBytes);
            tma_load_2d(base, &tm_xp, kb * kBK, m0, &sh->full[gs][0]);
            tma_load_2d(base + kTileBytes, &tm_xm, kb * kBK, m0, &sh->full[gs][0]);
            tma_load_2d(base + 2 * kTileBytes, &tm_wp, kb * kBK, n0, &sh->full[gs][0]);
            mbar_arrive(&sh->full[gs][1]);
          }
        } else {
          pair_steps(&tm_xp, &tm_wp, m0, n0, nkS);
          pair_steps(&tm_xm, &tm_wm, m0, n0, nkS);
        }
      }
      if (!ok) {  // copies already issued may still be landing: wait for them (bounded) before the CTA exits
        for (int i = grp > kGroups ? grp - kGroups : 0; i < grp; ++i) {
          mbar_wait(&sh->full[i % kGroups][0], (uint32_t)((i / kGroups) & 1));
          mbar_wait(&sh->full[i % kGroups][1], (uint32_t)((i / kGroups) & 1));
        }
      }
    }
  } else if (warp == 1) {
    // ================= tensor-core issuer =================
    if (lane == 0) {
      int grp = 0, ti = 0;
      bool ok = true;
      // one step of 64 hidden entries: four tcgen05.mma, 32 bytes further along the swizzled row each
      auto product = [&](uint32_t col, uint32_t a, uint32_t b, int kb) {
        const uint64_t ad = smem_desc_sw128(a), bd = smem_desc_sw128(b);
#pragma unroll
        for (int k = 0; k < kBK / kUmmaK; ++k)
          umma_bf16(tmem_base + col, ad + (uint64_t)(2 * k), bd + (uint64_t)(2 * k), kIdesc, (kb | k) != 0);
      };
      auto landed = [&](int gs, int j, uint32_t ph) {
        if (aborted(sh) || !mbar_wait(&sh->full[gs][j], ph)) { set_abort(sh, p.dev_error); ok = false; return; }
        tc_fence_after();
      };
      auto pair_steps = [&](uint32_t col, int nk) {
        for (int kb = 0; kb < nk && ok; kb += 2, ++grp) {
          const int gs = grp % kGroups;
          const uint32_t ph = (uint32_t)((grp / kGroups) & 1);
          const uint32_t base = smem0 + gs * kGroupBytes;
          for (int j = 0; j < 2 && kb + j < nk && ok; ++j) {
            landed(gs, j, ph);
            if (ok) product(col, base + j * 2 * kTileBytes, base + j * 2 * kTileBytes + kTileBytes, kb + j);
          }
          if (ok) umma_commit(&sh->empty[gs]);  // the group is free once these have read it
        }
      };
      for (int g = blockIdx.x; g < n_tiles && ok; g += gridDim.x, ++ti) {
        // h_LLM alternates between two accumulators, so its long K loop of the next tile runs while the
        // epilogue drains this one; h_SLM+ and h_SLM- wait for the epilogue of the tile before
        pair_steps((ti & 1) ? 384u : 0u, nkL);
        if (ok && ti > 0) {
          if (aborted(sh) || !mbar_wait(&sh->tmem_empty, (uint32_t)((ti - 1) & 1))) { set_abort(sh, p.dev_error); ok = false; }
          tc_fence_after();
        }
        if (p.shared_head) {
          for (int kb = 0; kb < nkS && ok; ++kb, ++grp) {
            const int gs = grp % kGroups;
            const uint32_t base = smem0 + gs * kGroupBytes;
            landed(gs, 0, (uint32_t)((grp / kGroups) & 1));
            if (!ok) break;
            product(128u, base, base + 2 * kTileBytes, kb);
            product(256u, base + kTileBytes, base + 2 * kTileBytes, kb);
            umma_commit(&sh->empty[gs]);
          }
        } else {
          pair_steps(128u, nkS);
          pair_steps(256u, nkS);
        }
        if (ok) umma_commit(&sh->tmem_full);
      }
      if (!ok) {  // let everything issued finish before tensor memory is given back
        umma_commit(&sh->drain);
        mbar_wait(&sh->drain, 0);
      }
    }
  } else {
    // ================= epilogue warps: one row per thread =================
    const int quarter = warp & 3;  // the lanes of tensor memory this warp may read
    const int K1 = p.K + 1;
    int ti = 0;
    for (int g = blockIdx.x; g < n_tiles; g += gridDim.x, ++ti) {
      const int mb = g % mb_count, nb = g / mb_count;
      const int row = mb * kBM + quarter * 32 + lane, n0 = nb * kBN;
      const bool valid = row < p.R;
      float beta = 0.f, c = 1.f;
      int tok = -1;
      if (valid) {
        const int b = row / K1, t = row - b * K1;
        beta = p.beta[b];
        c = kLog2e / p.temperature[b];
        int len = p.draft_len[b];
        if (len < 0 || len > p.K) len = 0;
        if (t < len) tok = p.draft_tokens[(long long)b * p.K + t] - p.vocab_offset;   // id within the heads passed
      }
      bool ok = !aborted(sh) && mbar_wait(&sh->tmem_full, (uint32_t)(ti & 1));
      ok = __all_sync(kFullMask, ok);
      if (!ok) {
        if (lane == 0) set_abort(sh, p.dev_error);
        break;
      }
      tc_fence_after();
      const uint32_t t_l = tmem_base + ((uint32_t)(quarter * 32) << 16) + ((ti & 1) ? 384u : 0u);
      const uint32_t t_p = tmem_base + ((uint32_t)(quarter * 32) << 16) + 128u;
      const uint32_t t_m = tmem_base + ((uint32_t)(quarter * 32) << 16) + 256u;
      const int n_valid = min(kBN, p.V - n0);
      // pass 1: maxima of the four quantities, and the drafted token's logits if they are in this tile
      float mx[4] = {kNegInf, kNegInf, kNegInf, kNegInf};
      int arg_r = -1;   // column of the tile's largest h_rec (greedy recovery)
#pragma unroll 1
      for (int j0 = 0; j0 < kBN; j0 += 32) {
        uint32_t L[32], P[32], M[32];
        tmem_ld32(t_l + j0, L); tmem_ld32(t_p + j0, P); tmem_ld32(t_m + j0, M);
        tmem_ld_wait();
        const int nv = n_valid - j0;
        if (nv >= 32) slice_max<false>(L, P, M, beta, 32, mx, j0, arg_r);
        else if (nv > 0) slice_max<true>(L, P, M, beta, nv, mx, j0, arg_r);
        const int jj = tok - n0 - j0;
        if (jj >= 0 && jj < 32 && jj < nv) {
          uint32_t tl = 0, tp = 0, tm = 0;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (j == jj) { tl = L[j]; tp = P[j]; tm = M[j]; }
          *reinterpret_cast<uint4*>(p.tok_logits + (long long)row * 4) = make_uint4(tl, tp, tm, 1u)  /* fourth word: the token lies in these heads */;
        }
      }
      float ref[4], nref[4], s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        ref[q] = ceilf(mx[q] * c);
        nref[q] = (ref[q] > kNegInf && ref[q] < -kNegInf) ? -ref[q] : 0.f;
      }
      // pass 2: sums of powers of two relative to the maxima
#pragma unroll 1
      for (int j0 = 0; j0 < kBN; j0 += 32) {
        uint32_t L[32], P[32], M[32];
        tmem_ld32(t_l + j0, L); tmem_ld32(t_p + j0, P); tmem_ld32(t_m + j0, M);
        tmem_ld_wait();
        const int nv = n_valid - j0;
        if (nv >= 32) slice_sum<false>(L, P, M, beta, c, nref, 32, s);
        else if (nv > 0) slice_sum<true>(L, P, M, beta, c, nref, nv, s);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->tmem_empty);  // the accumulators may be overwritten
      if (valid && p.argmax_keys)
        p.argmax_keys[(long long)row * p.n_chunks + nb] = arg_r >= 0 ? entry_key(mx[Q_R], n0 + arg_r + p.vocab_offset) : 0ull;
      if (valid) {
        const float2 rl = make_record(ref[Q_L], s[Q_L]), rp = make_record(ref[Q_P], s[Q_P]),
                     rm = make_record(ref[Q_M], s[Q_M]), rr = make_record(ref[Q_R], s[Q_R]);
        float* rec = p.part + ((long long)row * p.n_chunks + nb) * 8;
        *reinterpret_cast<float4*>(rec) = make_float4(rl.x, rl.y, rp.x, rp.y);
        *reinterpret_cast<float4*>(rec + 4) = make_float4(rm.x, rm.y, rr.x, rr.y);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---- verification alone: h_LLM and h_SLM- (Eq. 7), tiles of 128 rows x 256 vocabulary entries -------------
// Algorithm 1's verification reads P_LLM and P_SLM- only, so when nothing of the fused target is wanted on the drafted
// rows this kernel forms just those two products.  Two accumulators of 256 columns fill tensor memory, which buys a tile
// twice as wide: every hidden-state tile is used for 256 vocabulary entries, a third fewer operand bytes per flop than
// 128 x 128 tiles with three accumulators (the 128 x 128 kernel is short of operand bytes, not of tensor throughput).
// The two normalisers are independent, so the epilogue of h_LLM runs under the product of h_SLM- and the epilogue of
// h_SLM- under the next tile's h_LLM product: no second copy of an accumulator is needed.  Records: one per row and
// tile of 256 entries, {m, s} of h_LLM and h_SLM-, the other two slots empty.
constexpr int kBN2 = 256;
constexpr int kGroups2 = 4;                       // one step of 64 hidden entries each: {x (16 KB), W (32 KB)}
constexpr int kGroupBytes2 = 3 * kTileBytes;
constexpr int kSmemBytes2 = kGroups2 * kGroupBytes2 + 1024 /* alignment */ + 512 /* barriers */;
constexpr uint32_t kIdesc2 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN2 >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);

struct LmShared2 {
  uint64_t full[kGroups2], empty[kGroups2];
  uint64_t tmem_full[2], tmem_empty[2], drain;
  uint32_t tmem_slot;
  int abort_flag;
};
__device__ __forceinline__ bool aborted2(const LmShared2* sh) { return *reinterpret_cast<const volatile int*>(&sh->abort_flag) != 0; }
__device__ __forceinline__ void set_abort2(LmShared2* sh, int* dev_error) {
  *reinterpret_cast<volatile int*>(&sh->abort_flag) = 1;
  atomicExch(dev_error, 1);
}

// One accumulator of 256 columns, one row per thread: the record {m, s} of sum_v 2^(x_v c) over the valid columns, and
// the logit in column `jtok` (if 0 <= jtok < n_valid) into *tok_out / *found.
__device__ __forceinline__ float2 reduce_acc256(uint32_t taddr, int n_valid, float c, int jtok, uint32_t* tok_out, bool* found) {
  float mx = kNegInf;
#pragma unroll 1
  for (int j0 = 0; j0 < kBN2; j0 += 32) {
    uint32_t A[32];
    tmem_ld32(taddr + j0, A);
    tmem_ld_wait();
    const int nv = n_valid - j0;
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (j < nv) mx = fmaxf(mx, __uint_as_float(A[j]));
    const int jj = jtok - j0;
    if (jj >= 0 && jj < 32 && jj < nv) {
      uint32_t t = 0;
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (j == jj) t = A[j];
      *tok_out = t;
      *found = true;
    }
  }
  const float ref = ceilf(mx * c);
  const float nref = (ref > kNegInf && ref < -kNegInf) ? -ref : 0.f;
  float s = 0.f;
#pragma unroll 1
  for (int j0 = 0; j0 < kBN2; j0 += 32) {
    uint32_t A[32];
    tmem_ld32(taddr + j0, A);
    tmem_ld_wait();
    const int nv = n_valid - j0;
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (j < nv) s += ex2(fmaf(__uint_as_float(A[j]), c, nref));
  }
  return make_record(ref, s);
}

__global__ void __launch_bounds__(kThreads, 1)
lmhead_ratio_kernel(const __grid_constant__ CUtensorMap tm_xl, const __grid_constant__ CUtensorMap tm_wl,
                    const __grid_constant__ CUtensorMap tm_xm, const __grid_constant__ CUtensorMap tm_wm,
                    const LmKernelParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;  // operand tiles need 1024-byte alignment
  LmShared2* sh = reinterpret_cast<LmShared2*>(smem_raw + (smem0 - smem_u32(smem_raw)) + kGroups2 * kGroupBytes2);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int mb_count = (p.R + kBM - 1) / kBM, nb_count = (p.V + kBN2 - 1) / kBN2;
  const int n_tiles = mb_count * nb_count;
  const int nkL = (p.d_llm + kBK - 1) / kBK, nkS = (p.d_slm + kBK - 1) / kBK;

  if (tid == 0) {
    for (int s = 0; s < kGroups2; ++s) { mbar_init(&sh->full[s], 1); mbar_init(&sh->empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&sh->tmem_full[a], 1); mbar_init(&sh->tmem_empty[a], 4); }
    mbar_init(&sh->drain, 1);
    sh->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(&sh->tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&sh->tmem_slot);

  if (warp == 0) {
    // ================= TMA producer =================
    if (lane == 0) {
      int grp = 0;
      bool ok = true;
      auto steps = [&](const CUtensorMap* ta, const CUtensorMap* tb, int m0, int n0, int nk) {
        for (int kb = 0; kb < nk && ok; ++kb, ++grp) {
          const int gs = grp % kGroups2;
          const uint32_t ph = (uint32_t)((grp / kGroups2) & 1);
          if (aborted2(sh) || !mbar_wait(&sh->empty[gs], ph ^ 1u)) { set_abort2(sh, p.dev_error); ok = false; break; }
          const uint32_t base = smem0 + gs * kGroupBytes2;
          mbar_arrive_expect_tx(&sh->full[gs], 3 * kTileBytes);
          tma_load_2d(base, ta, kb * kBK, m0, &sh->full[gs]);
          tma_load_2d(base + kTileBytes, tb, kb * kBK, n0, &sh->full[gs]);   // 256 rows of the head: 32 KB
        }
      };
      for (int g = blockIdx.x; g < n_tiles && ok; g += gridDim.x) {
        const int mb = g % mb_count, nb = g / mb_count;  // row blocks fastest: CTAs running together share W tiles in L2
        steps(&tm_xl, &tm_wl, mb * kBM, nb * kBN2, nkL);
        steps(&tm_xm, &tm_wm, mb * kBM, nb * kBN2, nkS);
      }
      if (!ok) {  // copies already issued may still be landing: wait for them (bounded) before the CTA exits
        for (int i = grp > kGroups2 ? grp - kGroups2 : 0; i < grp; ++i)
          mbar_wait(&sh->full[i % kGroups2], (uint32_t)((i / kGroups2) & 1));
      }
    }
  } else if (warp == 1) {
    // ================= tensor-core issuer =================
    if (lane == 0) {
      int grp = 0, ti = 0;
      bool ok = true;
      auto product = [&](uint32_t col, int nk) {
        for (int kb = 0; kb < nk && ok; ++kb, ++grp) {
          const int gs = grp % kGroups2;
          if (aborted2(sh) || !mbar_wait(&sh->full[gs], (uint32_t)((grp / kGroups2) & 1))) { set_abort2(sh, p.dev_error); ok = false; break; }
          tc_fence_after();
          const uint32_t base = smem0 + gs * kGroupBytes2;
          const uint64_t ad = smem_desc_sw128(base), bd = smem_desc_sw128(base + kTileBytes);
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k)
            umma_bf16(tmem_base + col, ad + (uint64_t)(2 * k), bd + (uint64_t)(2 * k), kIdesc2, (kb | k) != 0);
          umma_commit(&sh->empty[gs]);  // the group is free once these have read it
        }
      };
      for (int g = blockIdx.x; g < n_tiles && ok; g += gridDim.x, ++ti) {
        for (int a = 0; a < 2 && ok; ++a) {
          if (ti > 0) {   // the epilogue of the tile before has read this accumulator
            if (aborted2(sh) || !mbar_wait(&sh->tmem_empty[a], (uint32_t)((ti - 1) & 1))) { set_abort2(sh, p.dev_error); ok = false; break; }
            tc_fence_after();
          }
          product(a ? 256u : 0u, a ? nkS : nkL);
          if (ok) umma_commit(&sh->tmem_full[a]);
        }
      }
      if (!ok) {  // let everything issued finish before tensor memory is given back
        umma_commit(&sh->drain);
        mbar_wait(&sh->drain, 0);
      }
    }
  } else {
    // ================= epilogue warps: one row per thread =================
    const int quarter = warp & 3;  // the lanes of tensor memory this warp may read
    const int K1 = p.K + 1;
    int ti = 0;
    for (int g = blockIdx.x; g < n_tiles; g += gridDim.x, ++ti) {
      const int mb = g % mb_count, nb = g / mb_count;
      const int row = mb * kBM + quarter * 32 + lane, n0 = nb * kBN2;
      const bool valid = row < p.R;
      float c = 1.f;
      int tok = -1;
      if (valid) {
        const int b = row / K1, t = row - b * K1;
        c = kLog2e / p.temperature[b];
        int len = p.draft_len[b];
        if (len < 0 || len > p.K) len = 0;
        if (t < len) tok = p.draft_tokens[(long long)b * p.K + t] - p.vocab_offset;   // id within the heads passed
      }
      const int n_valid = min(kBN2, p.V - n0);
      float2 rec2[2];
      uint32_t tl[2] = {0u, 0u};
      bool found = false;
      bool alive = true;
      for (int a = 0; a < 2; ++a) {
        bool ok = !aborted2(sh) && mbar_wait(&sh->tmem_full[a], (uint32_t)(ti & 1));
        ok = __all_sync(kFullMask, ok);
        if (!ok) {
          if (lane == 0) set_abort2(sh, p.dev_error);
          alive = false;
          break;
        }
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (a ? 256u : 0u);
        rec2[a] = reduce_acc256(taddr, n_valid, c, tok - n0, &tl[a], &found);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh->tmem_empty[a]);  // the accumulator may be overwritten
      }
      if (!alive) break;
      if (valid) {
        if (found) *reinterpret_cast<uint4*>(p.tok_logits + (long long)row * 4) = make_uint4(tl[0], 0u, tl[1], 1u);
        float* rec = p.part + ((long long)row * p.n_chunks + nb) * 8;
        *reinterpret_cast<float4*>(rec) = make_float4(rec2[0].x, rec2[0].y, kNegInf, 0.f);
        *reinterpret_cast<float4*>(rec + 4) = make_float4(rec2[1].x, rec2[1].y, kNegInf, 0.f);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---- two-phase round on this path: the recovery rows, compacted ----------------------------------------------
// The hidden states of row accept_len of every request that takes a token, gathered into [B][d] arrays (zero rows for
// the others), so that the three-accumulator kernel can form all three logit rows of exactly those positions (Eq. 8).
__global__ void __launch_bounds__(256) lmhead_gather_rows_kernel(const RoundParams p, const LmheadOperands op, uint16_t* xl,
                                                                 uint16_t* xp, uint16_t* xm) {
  const int b = blockIdx.x, tid = threadIdx.x;
  const int K = p.K, K1 = K + 1;
  const int n = p.accept_len[b];
  int len = p.draft_len[b];
  if (len < 0 || len > K) len = 0;
  const bool bad = (p.status_ws[b] & (SPECSTEER_REQ_BAD_PARAM | SPECSTEER_REQ_NONFINITE)) != 0;
  const bool sample = !bad && n >= 0 && n <= len && (n < len || (p.flags & SPECSTEER_FLAG_BONUS));
  const long long row = (long long)b * K1 + (sample ? n : 0);
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  for (int i = tid * 8; i < op.d_llm; i += 256 * 8)
    *reinterpret_cast<uint4*>(xl + (long long)b * op.d_llm + i) =
        sample ? __ldg(reinterpret_cast<const uint4*>(op.x_llm + row * op.d_llm + i)) : zero;
  for (int i = tid * 8; i < op.d_slm; i += 256 * 8) {
    *reinterpret_cast<uint4*>(xp + (long long)b * op.d_slm + i) =
        sample ? __ldg(reinterpret_cast<const uint4*>(op.x_plus + row * op.d_slm + i)) : zero;
    *reinterpret_cast<uint4*>(xm + (long long)b * op.d_slm + i) =
        sample ? __ldg(reinterpret_cast<const uint4*>(op.x_minus + row * op.d_slm + i)) : zero;
  }
}

// Last step of the two-phase round: the compact pass sampled (or took the argmax of) one token per request into
// rec_token / rec_logprob; this puts the round's outputs together from the real accepted lengths.  c_status: the status
// words of the compact pass (a non-finite recovery row shows there).
__global__ void __launch_bounds__(128) lmhead_finish_kernel(const RoundParams p, const int* c_status, const int* c_token) {
  const int b = blockIdx.x * 128 + threadIdx.x;
  if (b >= p.B) return;
  const int K = p.K, K1 = K + 1;
  const int n = p.accept_len[b];
  int status = p.status_ws[b];
  int len = p.draft_len[b];
  if (len < 0 || len > K) len = 0;
  const bool bad = (status & (SPECSTEER_REQ_BAD_PARAM | SPECSTEER_REQ_NONFINITE)) != 0;
  bool sample = !bad && (n < len || (p.flags & SPECSTEER_FLAG_BONUS));
  if (sample && (c_status[b] & SPECSTEER_REQ_NONFINITE)) {   // the recovery row has no distribution
    status |= SPECSTEER_REQ_NONFINITE;
    p.status_ws[b] = status;
    if (p.req_status) p.req_status[b] = status;
    sample = false;
  }
  int tok = sample ? c_token[b] : -1;   // c_token may be the caller's rec_token itself
  if (!sample || tok < 0) {
    tok = -1;
    if (p.rec_logprob) p.rec_logprob[b] = __int_as_float(0x7fc00000);
  }
  if (p.rec_token) p.rec_token[b] = tok;
  if (p.out_tokens)
    for (int t = 0; t <= K; ++t)
      p.out_tokens[(long long)b * K1 + t] = (t < n) ? p.draft_tokens[(long long)b * K + t] : ((t == n && tok >= 0) ? tok : -1);
  if (p.n_out) p.n_out[b] = n + (tok >= 0 ? 1 : 0);
}

// ---- recovery ------------------------------------------------------------------------------------------
constexpr int kRecT = 1024;  // 32 warps: recomputing the chunk is a chain of dependent loads per warp, so many warps
struct LmRecShared {
  double warp_tot[kRecT / 32];
  double base, target, W;
  int jstar, jlast, tok_min, tok_last;
  int plan_owner;               // sharded heads: the shard that holds the CDF target, -1 if nothing can be sampled
  double plan_target, plan_W;   // the target within that shard, and the weight of the whole row
};

__device__ __forceinline__ double block_excl_scan_rec(double v, double* warp_tot, int tid) {
  const int lane = tid & 31, warp = tid >> 5;
  double inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double u = __shfl_up_sync(kFullMask, inc, o);
    if (lane >= o) inc += u;
  }
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  double off = 0.0;
  for (int w = 0; w < warp; ++w) off += warp_tot[w];
  __syncthreads();
  return off + inc - v;
}

// dot product of a hidden state held in shared memory with one row of the head, 8 entries per lane and step
__device__ __forceinline__ float warp_dot_bf16(const uint16_t* x_sh, const uint16_t* w_row, int d, int lane) {
  float acc = 0.f;
#pragma unroll 4
  for (int i = lane * 8; i < d; i += 256) {  // d is a multiple of 8
    const uint4 wv = __ldg(reinterpret_cast<const uint4*>(w_row + i));
    const uint4 xv = *reinterpret_cast<const uint4*>(x_sh + i);
    acc = fmaf(bf16lo(xv.x), bf16lo(wv.x), acc); acc = fmaf(bf16hi(xv.x), bf16hi(wv.x), acc);
    acc = fmaf(bf16lo(xv.y), bf16lo(wv.y), acc); acc = fmaf(bf16hi(xv.y), bf16hi(wv.y), acc);
    acc = fmaf(bf16lo(xv.z), bf16lo(wv.z), acc); acc = fmaf(bf16hi(xv.z), bf16hi(wv.z), acc);
    acc = fmaf(bf16lo(xv.w), bf16lo(wv.w), acc); acc = fmaf(bf16hi(xv.w), bf16hi(wv.w), acc);
  }
  return warp_sum(acc);
}

__global__ void __launch_bounds__(kRecT) lmhead_recover_kernel(const RoundParams p, const LmheadOperands op) {
  extern __shared__ __align__(16) unsigned char rsm[];
  double* cw = reinterpret_cast<double*>(rsm);                                          // [n_chunks]
  uint16_t* xs = reinterpret_cast<uint16_t*>(rsm + ((size_t)p.n_chunks * 8 + 15) / 16 * 16);  // x_llm | x_plus | x_minus
  __shared__ LmRecShared sh;
  __shared__ float lg[3][kBN];
  const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int K = p.K, K1 = K + 1;
  pdl_wait();
  const int n = p.accept_len[b];
  const int status = p.status_ws[b];
  int len = p.draft_len[b];
  if (len < 0 || len > K) len = 0;
  const bool bad = (status & (SPECSTEER_REQ_BAD_PARAM | SPECSTEER_REQ_NONFINITE)) != 0;
  const bool sample = !bad && (n < len || (p.flags & SPECSTEER_FLAG_BONUS));
  if (p.out_tokens)
    for (int t = tid; t <= K; t += kRecT)
      p.out_tokens[(long long)b * K1 + t] = (t < n) ? p.draft_tokens[(long long)b * K + t] : -1;
  if (!sample) {
    if (tid == 0) {
      if (p.rec_token) p.rec_token[b] = -1;
      if (p.rec_logprob) p.rec_logprob[b] = __int_as_float(0x7fc00000);
      if (p.n_out) p.n_out[b] = n;
    }
    return;
  }
  const long long row = (long long)b * K1 + n;
  const double lseR = (double)p.lse2[row * 4 + Q_R];
  const float* rec = p.part + row * p.n_chunks * 8;
  for (int j = tid; j < p.n_chunks; j += kRecT) {
    const float m = rec[j * 8 + 6], s = rec[j * 8 + 7];
    cw[j] = (m == kNegInf) ? 0.0 : (double)s * exp2((double)m - lseR);
  }
  // the three hidden states of the row
  const int dL = op.d_llm, dS = op.d_slm;
  uint16_t *xl = xs, *xp = xs + dL, *xm = xs + dL + dS;
  for (int i = tid * 8; i < dL; i += kRecT * 8)
    *reinterpret_cast<uint4*>(xl + i) = __ldg(reinterpret_cast<const uint4*>(op.x_llm + row * dL + i));
  for (int i = tid * 8; i < dS; i += kRecT * 8) {
    *reinterpret_cast<uint4*>(xp + i) = __ldg(reinterpret_cast<const uint4*>(op.x_plus + row * dS + i));
    *reinterpret_cast<uint4*>(xm + i) = __ldg(reinterpret_cast<const uint4*>(op.x_minus + row * dS + i));
  }
  if (tid == 0) { sh.jstar = 0x7fffffff; sh.jlast = -1; sh.tok_min = 0x7fffffff; sh.tok_last = -1; }
  if (p.n_shards > 0 && tid == 0) {
    // Heads split along the vocabulary: every rank holds every shard's partial of this row, so all of them place
    // the target identically: shard weights in shard order, the target u*W, the first shard whose cumulative weight
    // exceeds it (else the last shard of positive weight).
    double Wg[SPECSTEER_MAX_SHARDS], W = 0.0;
    for (int g = 0; g < p.n_shards; ++g) {
      const ShardPartial& sp = p.shard_parts[((long long)g * p.B + b) * K1 + n];
      Wg[g] = (sp.m[Q_R] == kNegInf) ? 0.0 : sp.s[Q_R] * exp2((double)sp.m[Q_R] - lseR);
      W += Wg[g];
    }
    const double tgt = (double)p.u_recover[b] * W;
    double cum = 0.0, base = 0.0, base_last = 0.0;
    int owner = -1, last = -1;
    for (int g = 0; g < p.n_shards; ++g) {
      if (Wg[g] > 0.0) { last = g; base_last = cum; }
      if (cum + Wg[g] > tgt) { owner = g; base = cum; break; }
      cum += Wg[g];
    }
    if (owner < 0) { owner = last; base = base_last; }
    sh.plan_owner = (W > 0.0 && W == W) ? owner : -1;
    sh.plan_target = fmax(tgt - base, 0.0);
    sh.plan_W = W;
  }
  __syncthreads();
  if (p.n_shards > 0 && sh.plan_owner != p.shard_rank) {   // another shard (or nobody) samples: values a MAX-reduce ignores
    if (tid == 0) {
      if (p.rec_token) p.rec_token[b] = -1;
      if (p.rec_logprob) p.rec_logprob[b] = sh.plan_owner < 0 ? __int_as_float(0x7fc00000) : kNegInf;
      if (p.n_out) p.n_out[b] = n;
    }
    return;
  }

  // ---- the chunk that holds the CDF target: first chunk whose inclusive cumulative weight exceeds u*W, else the
  // last chunk of positive weight
  const int per = (p.n_chunks + kRecT - 1) / kRecT;
  const int j0 = min(tid * per, p.n_chunks), j1 = min(j0 + per, p.n_chunks);
  double local = 0.0;
  for (int j = j0; j < j1; ++j) local += cw[j];
  const double excl = block_excl_scan_rec(local, sh.warp_tot, tid);
  if (tid == kRecT - 1) {
    sh.W = p.n_shards > 0 ? sh.plan_W : excl + local;
    sh.target = p.n_shards > 0 ? sh.plan_target : (double)p.u_recover[b] * (excl + local);
  }
  __syncthreads();
  const double target = sh.target;
  {
    double cacc = excl;
    int mine = 0x7fffffff, lastpos = -1;
    for (int j = j0; j < j1; ++j) {
      if (cw[j] > 0.0) lastpos = j;
      if (mine == 0x7fffffff && cacc + cw[j] > target) mine = j;
      cacc += cw[j];
    }
    if (mine != 0x7fffffff) atomicMin(&sh.jstar, mine);
    if (lastpos >= 0) atomicMax(&sh.jlast, lastpos);
  }
  __syncthreads();
  const int jstar = sh.jstar != 0x7fffffff ? sh.jstar : max(sh.jlast, 0);
  if (jstar >= j0 && jstar < j1) {
    double base = excl;
    for (int j = j0; j < jstar; ++j) base += cw[j];
    sh.base = base;
  }
  // ---- the logits of that chunk, recomputed: warp w takes every 8th entry
  const int v_first = jstar * kBN;
  for (int e = warp; e < kBN; e += kRecT / 32) {
    const int v = v_first + e;
    float l = 0.f, pp = 0.f, m = 0.f;
    if (v < p.V) {
      l = warp_dot_bf16(xl, op.w_llm + (long long)v * dL, dL, lane);
      pp = warp_dot_bf16(xp, op.w_plus + (long long)v * dS, dS, lane);
      m = warp_dot_bf16(xm, op.w_minus + (long long)v * dS, dS, lane);
    }
    if (lane == 0) { lg[0][e] = l; lg[1][e] = pp; lg[2][e] = m; }
  }
  __syncthreads();
  // ---- inverse CDF inside the chunk: thread e < 128 owns entry e
  const double beta = (double)p.beta[b];
  const double cd = (double)(kLog2e / p.temperature[b]);
  double w = 0.0, y2 = 0.0;
  const int v = v_first + tid;
  if (tid < kBN && v < p.V) {
    y2 = ((double)lg[0][tid] + beta * ((double)lg[1][tid] - (double)lg[2][tid])) * cd - lseR;  // log2 Softmax(h_rec)(v)
    w = exp2(y2);
  }
  const double before = block_excl_scan_rec(w, sh.warp_tot, tid);
  if (tid < kBN && w > 0.0) {
    atomicMax(&sh.tok_last, v);
    if (sh.base + before + w > sh.target) atomicMin(&sh.tok_min, v);
  }
  __syncthreads();
  const int tok = sh.tok_min != 0x7fffffff ? sh.tok_min : sh.tok_last;
  if (tid < kBN && tok == v && tok >= 0) {
    if (p.rec_token) p.rec_token[b] = tok + p.vocab_offset;
    if (p.rec_logprob) p.rec_logprob[b] = (float)(y2 * 0.6931471805599453 - log(sh.W));
    if (p.out_tokens) p.out_tokens[(long long)b * K1 + n] = tok + p.vocab_offset;
    if (p.n_out) p.n_out[b] = n + 1;
  }
  if (tok < 0 && tid == 0) {  // no positive weight anywhere in the chunk: nothing can be sampled
    if (p.rec_token) p.rec_token[b] = -1;
    if (p.rec_logprob) p.rec_logprob[b] = __int_as_float(0x7fc00000);
    if (p.n_out) p.n_out[b] = n;
  }
}

// ---- host side --------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return (EncodeTiledFn) nullptr;
    return (EncodeTiledFn)f;
  }();
  return fn;
}

// [rows][d] bf16, row-major: boxes of 64 x 128 entries (128 bytes x 128 rows), 128-byte swizzle, zero fill outside
bool encode_operand(CUtensorMap* tm, const void* base, int rows, int d, int box_rows = kBM) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)d * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_lmhead(const RoundParams& p, const LmheadOperands& op, float* tok_logits, void* argmax_keys,
                          const LaunchInfo& li, cudaStream_t s) {
  const int R = p.B * (p.K + 1);
  if (R == 0) return cudaSuccess;
  CUtensorMap tm[6];
  if (!encode_operand(&tm[0], op.x_llm, R, op.d_llm) || !encode_operand(&tm[1], op.w_llm, p.V, op.d_llm) ||
      !encode_operand(&tm[2], op.x_plus, R, op.d_slm) || !encode_operand(&tm[3], op.w_plus, p.V, op.d_slm) ||
      !encode_operand(&tm[4], op.x_minus, R, op.d_slm) || !encode_operand(&tm[5], op.w_minus, p.V, op.d_slm))
    return cudaErrorInvalidValue;
  LmKernelParams k;
  k.R = R; k.V = p.V; k.K = p.K; k.d_llm = op.d_llm; k.d_slm = op.d_slm; k.n_chunks = p.n_chunks;
  k.draft_tokens = p.draft_tokens; k.draft_len = p.draft_len; k.beta = p.beta; k.temperature = p.temperature;
  k.part = p.part; k.tok_logits = tok_logits; k.dev_error = p.dev_error;
  k.argmax_keys = reinterpret_cast<u64*>(argmax_keys);
  k.shared_head = (op.w_plus == op.w_minus) ? 1 : 0;
  k.vocab_offset = p.vocab_offset;
  static std::atomic<bool> attr_set[64];   // per device; two host threads that both find it clear set the same value
  if (!attr_set[li.device & 63].load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(lmhead_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set[li.device & 63].store(true, std::memory_order_release);
  }
  const int mb = (R + kBM - 1) / kBM, nb = (p.V + kBN - 1) / kBN;
  const long long tiles = (long long)mb * nb;
  const int grid = (int)(tiles < li.sm_count ? tiles : li.sm_count);
  lmhead_kernel<<<grid, kThreads, kSmemBytes, s>>>(tm[0], tm[1], tm[2], tm[3], tm[4], tm[5], k);
  return cudaGetLastError();
}

cudaError_t launch_lmhead_ratio(const RoundParams& p, const LmheadOperands& op, float* tok_logits, const LaunchInfo& li,
                                cudaStream_t s) {
  const int R = p.B * (p.K + 1);
  if (R == 0) return cudaSuccess;
  CUtensorMap tm[4];
  if (!encode_operand(&tm[0], op.x_llm, R, op.d_llm) || !encode_operand(&tm[1], op.w_llm, p.V, op.d_llm, kBN2) ||
      !encode_operand(&tm[2], op.x_minus, R, op.d_slm) || !encode_operand(&tm[3], op.w_minus, p.V, op.d_slm, kBN2))
    return cudaErrorInvalidValue;
  LmKernelParams k;
  k.R = R; k.V = p.V; k.K = p.K; k.d_llm = op.d_llm; k.d_slm = op.d_slm; k.n_chunks = p.n_chunks;
  k.draft_tokens = p.draft_tokens; k.draft_len = p.draft_len; k.beta = p.beta; k.temperature = p.temperature;
  k.part = p.part; k.tok_logits = tok_logits; k.dev_error = p.dev_error;
  k.argmax_keys = nullptr;
  k.shared_head = 0;
  k.vocab_offset = p.vocab_offset;
  static std::atomic<bool> attr_set[64];
  if (!attr_set[li.device & 63].load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(lmhead_ratio_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes2);
    if (e != cudaSuccess) return e;
    attr_set[li.device & 63].store(true, std::memory_order_release);
  }
  const int mb = (R + kBM - 1) / kBM, nb = (p.V + kBN2 - 1) / kBN2;
  const long long tiles = (long long)mb * nb;
  const int grid = (int)(tiles < li.sm_count ? tiles : li.sm_count);
  lmhead_ratio_kernel<<<grid, kThreads, kSmemBytes2, s>>>(tm[0], tm[1], tm[2], tm[3], k);
  return cudaGetLastError();
}

cudaError_t launch_lmhead_gather_rows(const RoundParams& p, const LmheadOperands& op, uint16_t* xl, uint16_t* xp, uint16_t* xm,
                                      cudaStream_t s) {
  if (p.B == 0) return cudaSuccess;
  lmhead_gather_rows_kernel<<<p.B, 256, 0, s>>>(p, op, xl, xp, xm);
  return cudaGetLastError();
}

cudaError_t launch_lmhead_finish(const RoundParams& p, const int* c_status, const int* c_token, cudaStream_t s) {
  if (p.B == 0) return cudaSuccess;
  lmhead_finish_kernel<<<(p.B + 127) / 128, 128, 0, s>>>(p, c_status, c_token);
  return cudaGetLastError();
}

// Greedy recovery on the fused path: the largest of the per-tile keys of row accept_len (value first, lower id among
// equal values), its log-probability from the row's normaliser.
__global__ void __launch_bounds__(256) lmhead_argmax_kernel(const RoundParams p, const u64* keys) {
  __shared__ u64 wbest[8];
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K = p.K, K1 = K + 1;
  pdl_wait();
  const int n = p.accept_len[b];
  const int status = p.status_ws[b];
  int len = p.draft_len[b];
  if (len < 0 || len > K) len = 0;
  const bool bad = (status & (SPECSTEER_REQ_BAD_PARAM | SPECSTEER_REQ_NONFINITE)) != 0;
  const bool sample = !bad && (n < len || (p.flags & SPECSTEER_FLAG_BONUS));
  if (p.out_tokens && !p.greedy_keys)
    for (int t = tid; t <= K; t += 256)
      p.out_tokens[(long long)b * K1 + t] = (t < n) ? p.draft_tokens[(long long)b * K + t] : -1;
  const long long row = (long long)b * K1 + n;
  u64 best = 0;
  if (sample)
    for (int j = tid; j < p.n_chunks; j += 256) {
      const u64 k = __ldcg(keys + row * p.n_chunks + j);
      best = k > best ? k : best;
    }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const u64 other = __shfl_xor_sync(kFullMask, best, o);
    best = other > best ? other : best;
  }
  if (lane == 0) wbest[warp] = best;
  __syncthreads();
  if (tid != 0) return;
  for (int w = 1; w < 8; ++w) best = wbest[w] > best ? wbest[w] : best;
  if (p.greedy_keys) {   // heads split along the vocabulary: the key (its id is already global) goes to the reduction over shards
    const long long id = (long long)(0xffffffffu - (uint32_t)(best & 0xffffffffu));
    p.greedy_keys[b] = (sample && best) ? (long long)(((best >> 32) << 31) | (u64)(0x7fffffffll - id)) : -1;
    return;
  }
  if (!sample || best == 0) {
    if (p.rec_token) p.rec_token[b] = -1;
    if (p.rec_logprob) p.rec_logprob[b] = __int_as_float(0x7fc00000);
    if (p.n_out) p.n_out[b] = n;
    return;
  }
  const int tok = (int)(0xffffffffu - (uint32_t)(best & 0xffffffffu));
  const double r = (double)order_val((uint32_t)(best >> 32));
  const double lseR = (double)p.lse2[row * 4 + Q_R];
  if (p.rec_token) p.rec_token[b] = tok;
  if (p.rec_logprob) p.rec_logprob[b] = (float)((r * (double)(kLog2e / p.temperature[b]) - lseR) * 0.6931471805599453);
  if (p.out_tokens) p.out_tokens[(long long)b * K1 + n] = tok;
  if (p.n_out) p.n_out[b] = n + 1;
}

cudaError_t launch_lmhead_argmax(const RoundParams& p, const void* argmax_keys, cudaStream_t s) {
  if (p.B == 0) return cudaSuccess;
  lmhead_argmax_kernel<<<p.B, 256, 0, s>>>(p, reinterpret_cast<const u64*>(argmax_keys));
  return cudaGetLastError();
}

cudaError_t launch_lmhead_recover(const RoundParams& p, const LmheadOperands& op, cudaStream_t s) {
  if (p.B == 0) return cudaSuccess;
  const size_t smem = ((size_t)p.n_chunks * 8 + 15) / 16 * 16 + (size_t)(op.d_llm + 2 * op.d_slm) * 2;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(lmhead_recover_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  lmhead_recover_kernel<<<p.B, kRecT, smem, s>>>(p, op);
  return cudaGetLastError();
}

}  // namespace specsteer
