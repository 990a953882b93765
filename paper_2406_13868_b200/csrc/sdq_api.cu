// Status plumbing of the C-ABI: sticky device flags and status strings.
#include "sdq_internal.h"

namespace sdq {

__device__ uint32_t g_flags[FLAG_COUNT];

uint32_t* device_flags() {
  // resolved once per device (the symbol lives in every context that loads the library)
  static uint32_t* cache[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
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
