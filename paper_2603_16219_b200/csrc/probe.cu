// Measurement aid: the rate at which one GPU evaluates ex2.approx, the instruction that bounds the streaming kernel
// on 16-bit logits together with HBM.  Not on the path of any round.
#include "common.cuh"
#include "specsteer.h"

namespace specsteer {

// Every thread runs eight independent chains of `iters` dependent ex2.approx each (arguments stay in (-1, 0], so
// nothing overflows or flushes); the results are folded into one store per thread so that nothing is optimised away.
__global__ void __launch_bounds__(1024) ex2_probe_kernel(int iters, float* sink) {
  float x[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) x[i] = -0.1f * (float)((threadIdx.x + i) & 7) - 0.05f;
#pragma unroll 1
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = ex2(x[i]) - 1.0f;   // 2^x - 1 in (-1, 0] for x in (-1, 0]
  }
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) s += x[i];
  sink[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = s;
}

}  // namespace specsteer

extern "C" specsteer_status specsteer_probe_ex2(int32_t n_ctas, int32_t iters, float* sink, void* cuda_stream) {
  if (n_ctas <= 0 || iters <= 0 || !sink) return SPECSTEER_ERR_INVALID_ARG;
  specsteer::ex2_probe_kernel<<<n_ctas, 1024, 0, (cudaStream_t)cuda_stream>>>(iters, sink);
  return cudaGetLastError() == cudaSuccess ? SPECSTEER_OK : SPECSTEER_ERR_CUDA;
}
