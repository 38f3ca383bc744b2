// solar_lowrank_factor_static: the factorization for callers that can hand over
// input and output buffers but no scratch memory.  The partial Grams that
// solar_lowrank_factor keeps in a caller-provided workspace live here in a
// fixed array inside the library's own device image.
#include <mutex>

#include "solar_internal.cuh"

namespace {

constexpr size_t kStaticScratchBytes = (size_t)16 << 20;   // 16 MiB, held by every GPU that loads the library

// Device-resident scratch.  In host code this NAME is only a handle for the
// runtime's symbol lookup, never a device address: the address each device
// gives it is fetched once with cudaGetSymbolAddress and passed to the kernels.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};
bool g_scratch_ready[kMaxDevices] = {};

// Address of the scratch array on the CURRENT device; looked up on the first
// call per device and cached.  No allocation happens here or anywhere below.
solar_status_t scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SOLAR_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ready[dev]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || p == nullptr) return SOLAR_ERR_CUDA;
    g_scratch_addr[dev] = p;
    g_scratch_ready[dev] = true;
  }
  *out = g_scratch_addr[dev];
  return SOLAR_OK;
}

}  // namespace

extern "C" {

size_t solar_static_scratch_bytes(void) { return kStaticScratchBytes; }

solar_status_t solar_lowrank_factor_static(int B, int M, int N, int d, int r, solar_dtype_t dt,
                                           const void* H, float* S, float* V, int* info,
                                           void* stream) {
  (void)M;
  // Size screening first, on the host, so an oversized request never touches the device.
  const size_t need = solar_workspace_bytes(B, 0, N, d, r, dt);
  if (need == 0) {
    // unsupported / invalid sizes: let the regular entry point name the reason (it returns
    // before using any pointer because the sizes fail first)
    return solar_lowrank_factor(B, 0, N, d, r, dt, H, S, V, nullptr, info, nullptr, 0, stream);
  }
  if (B == 0) return SOLAR_OK;
  if (solar::factor_ws_bytes(B, N, d, dt) > kStaticScratchBytes) return SOLAR_ERR_WORKSPACE;
  void* scratch = nullptr;
  const solar_status_t st = scratch_for_current_device(&scratch);
  if (st != SOLAR_OK) return st;
  return solar_lowrank_factor(B, 0, N, d, r, dt, H, S, V, nullptr, info, scratch,
                              kStaticScratchBytes, stream);
}

}  // extern "C"
