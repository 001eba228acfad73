// moqae_decode_attn_static: decode attention for callers that cannot allocate device memory.
//
// Some hosts of this library never get to call cudaMalloc: a plug-in running inside a
// serving process whose memory pool is owned and fully reserved by the host application, a
// real-time loop that forbids allocator calls after start-up, or a thin foreign-language
// shim that can pass through the pointers it was given but has no allocator of its own.
// Such a caller still owns q, the cache and out, but has nowhere to put the split-K
// partials that moqae_decode_attn wants as `workspace`.  Here that scratch is a fixed array
// that lives in the library image itself, so every device that loads the library carries
// kStaticScratchBytes of it until the process exits.
#include <mutex>

#include "common.cuh"

namespace moqae {

namespace {

constexpr long long kStaticScratchBytes = 4ll << 20;   // 4 MiB per device
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for the runtime (not a device address): the
// address the kernels need comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_decode_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
void* g_scratch_of_device[kMaxDevices] = {};

// Device address of the scratch array on the CURRENT device, looked up once per device.
cudaError_t scratch_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_of_device[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_decode_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    g_scratch_of_device[dev] = p;
  }
  *out = g_scratch_of_device[dev];
  return cudaSuccess;
}

}  // namespace

}  // namespace moqae

#pragma GCC visibility push(default)
extern "C" {

int64_t moqae_decode_attn_static_max_bytes(void) { return moqae::kStaticScratchBytes; }

int moqae_decode_attn_static(const moqae_config* cfg, const void* q, int32_t layer, const moqae_cache* cache,
                             float* out, float scale, void* stream) {
  int64_t need = 0;
  int rc = moqae_decode_attn_workspace(cfg, &need);
  if (rc != MOQAE_OK) return rc;
  if (need > moqae::kStaticScratchBytes) return MOQAE_ERR_WORKSPACE_TOO_SMALL;
  void* scratch = nullptr;
  cudaError_t e = moqae::scratch_address(&scratch);
  if (e != cudaSuccess) {
    moqae::record_cuda_error(e);
    return MOQAE_ERR_CUDA;
  }
  // The array is shared by every configuration that is ever used on this device, so the place
  // where this one keeps its arrival counters may hold another one's partials: clear it here
  // (moqae_decode_attn itself relies on the caller having zeroed its workspace once).
  long long off = 0, len = 0;
  moqae::decode_counter_region(cfg, &off, &len);
  e = cudaMemsetAsync(static_cast<unsigned char*>(scratch) + off, 0, static_cast<size_t>(len),
                      static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) {
    moqae::record_cuda_error(e);
    return MOQAE_ERR_CUDA;
  }
  // Same kernels, same argument checks; only the home of the partials differs.
  return moqae_decode_attn(cfg, q, layer, cache, out, scale, scratch, moqae::kStaticScratchBytes, stream);
}

}  // extern "C"
#pragma GCC visibility pop
