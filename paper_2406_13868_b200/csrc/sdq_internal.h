// Internals shared by the translation units of the library (not part of the C-ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sdq.h"

namespace sdq {

// Sticky device-side flag words (one small allocation-free __device__ array per loaded library).
enum { FLAG_NONFINITE = 0, FLAG_TIMEOUT = 1, FLAG_COUNT = 4 };

// device address of the flag words of the current device (nullptr on failure)
uint32_t* device_flags();

// Host-side facts about one device, looked up by the CURRENT device of the calling thread: they differ between the
// GPUs of one process (SM count; function attributes are per context), so nothing of this kind is a process-wide static.
struct DeviceInfo {
  int sm_count;            // 0 until queried
  uint32_t linear_attr;    // 1: the single-CTA GEMM instantiations carry their shared-memory attribute
  uint32_t pair_attr;      // bit per CTA-pair GEMM instantiation
  uint32_t diag_attr;      // the copy-rate diagnostic
  uint32_t group_attr;     // the grouped few-token GEMM
};
constexpr int MAX_DEVICES = 64;
// entry of device `dev` (0 <= dev < MAX_DEVICES) in the table; nullptr outside that range
DeviceInfo* device_info_slot(int dev);
// entry of the current device with sm_count filled in (nullptr on failure).  First use per device takes a lock.
DeviceInfo* device_info();

}  // namespace sdq
