// moe_router_wgrad_static: the router weight gradient dW_r = x^T dl for callers that must not allocate device
// memory.  The token-slice partial sums that the regular path keeps in the caller's workspace live here in a
// fixed array inside the library image.
#include <mutex>

#include "common.cuh"

namespace moe {

// Scratch for DWR_SPLIT token-slice partials of a [d, E] fp32 matrix.  Every GPU that loads the library holds these
// MOE_STATIC_MAX_DE * DWR_SPLIT * 4 bytes (8 MiB) until the process exits.
static __device__ __align__(256) float g_static_partials[static_cast<size_t>(DWR_SPLIT) * MOE_STATIC_MAX_DE];

// In host code the array's name is only a handle for the runtime, not a device address; the kernels need the
// address cudaGetSymbolAddress returns for the device that is current.  Looked up once per device.
constexpr int MAX_DEVICES = 64;
static float* g_partials_addr[MAX_DEVICES] = {nullptr};
static std::mutex g_partials_mutex;

static moe_status static_partials(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return MOE_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_partials_mutex);
  if (g_partials_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_partials) != cudaSuccess || p == nullptr) return MOE_ERR_CUDA;
    g_partials_addr[dev] = static_cast<float*>(p);
  }
  *out = g_partials_addr[dev];
  return MOE_OK;
}

}  // namespace moe

using namespace moe;

extern "C" moe_status moe_router_wgrad_static(int64_t T, int32_t d, int32_t E, const uint16_t* x, const float* dl,
                                              float* dW_r, void* cuda_stream) {
  if (T < 0 || d <= 0 || E < 1 || E > MAX_E || d % 64 != 0) return MOE_ERR_INVALID_ARG;
  if (!dW_r || (T > 0 && (!x || !dl))) return MOE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(x) & 3u) || (reinterpret_cast<uintptr_t>(dl) & 3u) ||
      (reinterpret_cast<uintptr_t>(dW_r) & 3u))
    return MOE_ERR_INVALID_ARG;
  if (static_cast<int64_t>(d) * E > MOE_STATIC_MAX_DE) return MOE_ERR_UNSUPPORTED;  // beyond the built-in scratch
  float* partials = nullptr;
  const moe_status rc = static_partials(&partials);
  if (rc != MOE_OK) return rc;
  const Shape s{d, E, 64, 1};
  // Every slice partial of the [d, E] region is overwritten by the first kernel (slices without tokens write
  // zeros), so nothing left behind by an earlier call is ever read and no clearing pass is needed.
  launch_dwr(s, T, x, dl, partials, dW_r, nullptr, /*partials_ready=*/false, static_cast<cudaStream_t>(cuda_stream));
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}
