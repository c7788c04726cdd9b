// Verification for callers that must not allocate: the same kernels as specsteer_verify_round, with the
// workspace taken from a fixed device array that is part of the library image.
#include <mutex>

#include "internal.h"
#include "specsteer.h"

using namespace specsteer;

namespace {

// Limits of the fixed scratch (see the header): requests, rows, and per-chunk partial records.
constexpr int kStaticMaxB = 1024;
constexpr long long kStaticMaxRows = 16384;
constexpr long long kStaticMaxRecords = 229376;
constexpr size_t kPartBytes = (size_t)kStaticMaxRecords * 8 * sizeof(float);  // 7 MiB
constexpr size_t kLseBytes = (size_t)kStaticMaxRows * 4 * sizeof(float);      // 256 KiB
constexpr size_t kStatusBytes = (size_t)kStaticMaxB * sizeof(int);
constexpr size_t kStaticBytes = (size_t)8 << 20;
static_assert(kPartBytes + kLseBytes + kStatusBytes + 256 <= kStaticBytes, "scratch layout overflows the array");

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress; it is not a
// device address and must never be handed to a kernel as one.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

struct DeviceSetup {
  bool ready = false;
  unsigned char* base = nullptr;  // device address of g_static_scratch on this device
  LaunchInfo li{};
};
DeviceSetup g_setup[64];
std::mutex g_setup_mutex;

// Once per device, with that device current: resolve the array's device address and read the SM count.
specsteer_status setup_device(int dev, DeviceSetup** out) {
  if (dev < 0 || dev >= 64) return SPECSTEER_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  DeviceSetup& s = g_setup[dev];
  if (!s.ready) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
      cudaGetLastError();
      return SPECSTEER_ERR_CUDA;
    }
    s.li.device = dev;
    if (cudaDeviceGetAttribute(&s.li.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&s.li.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
      cudaGetLastError();
      return SPECSTEER_ERR_CUDA;
    }
    s.base = static_cast<unsigned char*>(ptr);
    s.ready = true;
  }
  *out = &s;
  return SPECSTEER_OK;
}

}  // namespace

extern "C" specsteer_status specsteer_verify_round_static(const specsteer_round_desc* d, void* cuda_stream) {
  // the same host-side checks as specsteer_verify_round (every recovery mode is accepted: verification does not
  // depend on it; u_recover is not needed here)
  specsteer_status chk = check_round_desc(d, false);
  if (chk != SPECSTEER_OK) return chk;
  const int tile = d->dtype == SPECSTEER_F32 ? kChunkF32 : kChunkBF16;
  const int n_chunks = (d->V + tile - 1) / tile;
  const long long rows = (long long)d->B * (d->K + 1);
  if (d->B > kStaticMaxB || rows > kStaticMaxRows || rows * n_chunks > kStaticMaxRecords)
    return SPECSTEER_ERR_STATIC_LIMIT;
  if (d->B == 0) return SPECSTEER_OK;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return SPECSTEER_ERR_CUDA;
  DeviceSetup* su = nullptr;
  specsteer_status st = setup_device(dev, &su);
  if (st != SPECSTEER_OK) return st;

  RoundParams p{};
  p.B = d->B; p.K = d->K; p.V = d->V;
  p.ld_row = d->ld_row; p.ld_req = d->ld_req;
  p.accept_mode = d->accept_mode; p.recover_mode = d->recover_mode; p.flags = d->flags;
  p.sums = sums_wanted(d);
  p.row_mode = ROWS_ALL;
  p.tile = tile; p.n_chunks = n_chunks;
  p.h_llm = d->h_llm; p.h_plus = d->h_slm_plus; p.h_minus = d->h_slm_minus;
  p.draft_tokens = d->draft_tokens; p.draft_len = d->draft_len;
  p.lambda = d->lambda; p.beta = d->beta; p.temperature = d->temperature;
  p.u_accept = d->u_accept; p.u_recover = d->u_recover;
  p.accept_len = d->accept_len; p.accept_flags = d->accept_flags; p.alpha = d->alpha;
  p.logp_llm = d->logp_llm; p.logp_minus = d->logp_minus; p.logp_plus = d->logp_plus; p.logp_star = d->logp_star;
  p.log_z = d->log_z; p.req_status = d->req_status;
  // every word of scratch a launch reads is written earlier in the same launch sequence (partial records by
  // the streaming kernel, normalisers and status by the epilogue), so nothing has to be cleared between calls;
  // the abort word is only ever set, and is not reported by this entry point
  p.part = reinterpret_cast<float*>(su->base);
  p.lse2 = reinterpret_cast<float*>(su->base + kPartBytes);
  p.status_ws = reinterpret_cast<int*>(su->base + kPartBytes + kLseBytes);
  p.dev_error = reinterpret_cast<int*>(su->base + kPartBytes + kLseBytes + kStatusBytes);
  p.wait_cycles = kDefaultWaitCycles;

  const bool aligned = rows_aligned(d);
  int nl = 0;
  if (launch_verify(p, d->dtype, aligned, su->li, (cudaStream_t)cuda_stream, &nl) != cudaSuccess) {
    cudaGetLastError();
    return SPECSTEER_ERR_CUDA;
  }
  return SPECSTEER_OK;
}
