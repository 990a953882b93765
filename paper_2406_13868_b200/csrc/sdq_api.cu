// Status plumbing of the C-ABI: sticky device flags and status strings.
#include <mutex>

#include "sdq_internal.h"

namespace sdq {

static DeviceInfo g_device_info[MAX_DEVICES];
static std::mutex g_device_mutex;

DeviceInfo* device_info_slot(int dev) { return (dev >= 0 && dev < MAX_DEVICES) ? &g_device_info[dev] : nullptr; }

DeviceInfo* device_info() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
  DeviceInfo* d = device_info_slot(dev);
  if (!d) return nullptr;
  std::lock_guard<std::mutex> lock(g_device_mutex);
  if (!d->sm_count) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return nullptr;
    d->sm_count = n;
  }
  return d;
}

__device__ uint32_t g_flags[FLAG_COUNT];

uint32_t* device_flags() {
  // resolved once per device (the symbol lives in every context that loads the library)
  static uint32_t* cache[MAX_DEVICES] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return nullptr;
  std::lock_guard<std::mutex> lock(g_device_mutex);
  if (!cache[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_flags) != cudaSuccess) return nullptr;
    cache[dev] = (uint32_t*)ptr;
  }
  return cache[dev];
}

}  // namespace sdq

extern "C" sdq_status_t sdq_device_status(void* stream)
{
  uint32_t* flags = sdq::device_flags();
  if (!flags) return SDQ_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  uint32_t h[sdq::FLAG_COUNT] = {0, 0, 0, 0};
  if (cudaMemcpyAsync(h, flags, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SDQ_ERR_CUDA;
  if (cudaMemsetAsync(flags + sdq::FLAG_TIMEOUT, 0, sizeof(uint32_t), st) != cudaSuccess) return SDQ_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return SDQ_ERR_CUDA;
  return h[sdq::FLAG_TIMEOUT] ? SDQ_ERR_TIMEOUT : SDQ_OK;
}

extern "C" const char* sdq_status_string(sdq_status_t s)
{
  switch (s) {
    case SDQ_OK: return "ok";
    case SDQ_ERR_INVALID_ARG: return "invalid argument";
    case SDQ_ERR_SHAPE: return "shape violates the preconditions";
    case SDQ_ERR_ALIGNMENT: return "pointer or leading dimension not 16-byte aligned";
    case SDQ_ERR_UNSUPPORTED: return "configuration not supported by this kernel set";
    case SDQ_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case SDQ_ERR_NONFINITE: return "non-finite weight";
    case SDQ_ERR_CUDA: return "CUDA runtime error";
    case SDQ_ERR_TIMEOUT: return "device-side bounded wait timed out";
  }
  return "unknown status";
}
