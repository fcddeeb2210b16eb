// critiprefill_estimate_static: Algorithm 1 with the library's own, statically reserved
// scratch instead of a caller-provided workspace.
//
// Some callers cannot hand the library a workspace because they cannot allocate device
// memory at the point of the call: a serving process whose memory pool claimed the whole
// device at start-up, a latency-critical loop that must not pay cudaMalloc's implicit
// device-wide synchronisation, a plug-in that runs inside somebody else's allocator rules.
// For them the summaries (the only scratch Algorithm 1 needs) live in a fixed array in the
// library's device image.  Every GPU that loads the library carries that array until the
// process exits, so it is kept modest: kStaticScratchBytes.
#include <mutex>

#include "cp_common.cuh"

namespace {

// 8 MiB.  Enough for 128K tokens of 32 query / 8 KV heads at segment 1024 / block 128 (6 MiB of summaries) and for the
// 32 / 4-head shape (4 MiB); NOT enough for segment 512 / block 32 at 128K tokens (4 MiB of query + 16 MiB of key
// summaries), which gets CP_ERR_STATIC_LIMIT.
constexpr size_t kStaticScratchBytes = size_t(8) << 20;
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress;
// it is not a device address and must never be passed to a kernel directly.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_mutex;
void* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the array on the current device, resolved once per device and cached for the life of
// the process.  cudaDeviceReset unloads the library's device image, after which a cached address is stale:
// this entry point must not be used across a reset of a device it has already served.
int static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CP_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return CP_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return CP_OK;
}

}  // namespace

extern "C" int critiprefill_estimate_static(const cp_params* p, const void* Q, const void* K, const double* S_prev,
                                            double* S_out, void* cuda_stream) {
  using namespace cp;
  size_t need = 0;
  int rc = critiprefill_workspace_bytes(p, &need);   // validates sizes, strides and dtype
  if (rc != CP_OK) return rc;
  if (need > kStaticScratchBytes) return CP_ERR_STATIC_LIMIT;
  if (!Q || !K || !S_out) return CP_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(Q) & 15u) || (reinterpret_cast<uintptr_t>(K) & 15u) || S_out == S_prev)
    return CP_ERR_SHAPE;
  if (S_prev != nullptr && !(p->alpha >= 0.0f && p->alpha <= 1.0f)) return CP_ERR_SHAPE;
  const Dims m = make_dims(*p);
  if (m.n2 > kMaxBlocksN2) return CP_ERR_UNSUPPORTED;
  void* scratch = nullptr;
  if ((rc = static_scratch(&scratch)) != CP_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  // The array keeps whatever the previous call left.  The summaries are fully rewritten
  // before they are read; the 256-byte status head is the only part that must start at zero.
  if (cudaMemsetAsync(scratch, 0, kStatusBytes, s) != cudaSuccess) return CP_ERR_CUDA;
  if ((rc = launch_summarize(*p, m, Q, K, static_cast<char*>(scratch), s)) != CP_OK) return rc;
  return launch_score(*p, m, static_cast<char*>(scratch), S_prev, S_out, s);
}

extern "C" size_t critiprefill_static_scratch_bytes(void) { return kStaticScratchBytes; }
