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

}  // namespace sdq
