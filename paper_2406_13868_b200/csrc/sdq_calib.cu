// Calibration helper for the weight-activation product metric (Section 5, Stage 1: "if using calibration data is
// allowed ... weight-activation-product"): the Euclidean norm of every input channel over a set of tokens,
//   c[k] = sqrt(sum_m x[m][k]^2),
// which sdq_decompose_metric takes as its per-channel weight.  Offline; one thread per two channels walks the tokens in
// order and accumulates in fp64, so the result is reproducible and correctly rounded to fp32 for all practical sizes.
#include <cuda_bf16.h>

#include "sdq_internal.h"

namespace sdq {

constexpr int CN_THREADS = 128;

__global__ void __launch_bounds__(CN_THREADS)
channel_norm_kernel(const __nv_bfloat16* __restrict__ X, int64_t M, int64_t K, int64_t ldx, float* __restrict__ c)
{
  const int64_t k = ((int64_t)blockIdx.x * CN_THREADS + threadIdx.x) * 2;     // K is even
  if (k >= K) return;
  double s0 = 0.0, s1 = 0.0;
  const __nv_bfloat16* col = X + k;
#pragma unroll 4
  for (int64_t m = 0; m < M; ++m) {
    const uint32_t r = *reinterpret_cast<const uint32_t*>(col + m * ldx);
    const double a = (double)__uint_as_float(r << 16), b = (double)__uint_as_float(r & 0xFFFF0000u);
    s0 += a * a;
    s1 += b * b;
  }
  c[k] = (float)sqrt(s0);
  c[k + 1] = (float)sqrt(s1);
}

}  // namespace sdq

using namespace sdq;

extern "C" sdq_status_t sdq_channel_norm(const void* X, int64_t M, int64_t K, int64_t ldx, float* col_norm, void* stream)
{
  if (!X || !col_norm) return SDQ_ERR_INVALID_ARG;
  if (M <= 0 || K <= 0 || (K & 1) || ldx < K) return SDQ_ERR_SHAPE;
  if (((uintptr_t)X & 3) || (ldx & 1) || ((uintptr_t)col_norm & 3)) return SDQ_ERR_ALIGNMENT;
  const unsigned grid = (unsigned)((K / 2 + CN_THREADS - 1) / CN_THREADS);
  channel_norm_kernel<<<grid, CN_THREADS, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)X, M, K, ldx, col_norm);
  return cudaGetLastError() == cudaSuccess ? SDQ_OK : SDQ_ERR_CUDA;
}
