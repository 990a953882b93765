// Measurement and self-test aids, not part of the method (declared in include/sdq_diag.h).
// Copy rate: the rate at which all SMs together can stage bytes from L2 into shared
// memory with bulk copies.  The many-token GEMM is bound by exactly this path (a 128 x 256 tile pulls 2.09 MB of
// operands through it), so the benchmark measures its ceiling live beside the kernel.
//
// One CTA per SM keeps `nslot` bulk copies of `slot_bytes` in flight from its own region of the source (walked
// cyclically, so the source stays L2-resident after a first pass) and re-issues a slot as soon as its copy has landed;
// nothing consumes the data.  The slots are dealt out over `issuers` threads (one per warp), as the GEMM spreads its
// copies over three producer threads.  Every wait is bounded.
#include "../../include/sdq_diag.h"
#include "sdq_internal.h"
#include "sdq_ptx.cuh"

namespace sdq {

__global__ void __launch_bounds__(128, 1)
l2_copy_kernel(const uint8_t* __restrict__ src, size_t region_bytes, int iters, int nslot, int slot_bytes, int issuers, uint32_t* __restrict__ flags)
{
  extern __shared__ uint8_t dsm[];
  __shared__ __align__(8) uint64_t full[16];
  uint8_t* sm = dsm + ((128 - (ptx::smem_u32(dsm) & 127)) & 127);
  if (threadIdx.x == 0) {
    for (int s = 0; s < nslot; ++s) ptx::mbar_init(&full[s], 1);
    ptx::fence_barrier_init();
  }
  __syncthreads();
  const int me = (int)(threadIdx.x >> 5);
  if ((threadIdx.x & 31) != 0 || me >= issuers) return;
  // issuer `me` owns slots me, me + issuers, ...; copy number c (0 .. iters - 1) goes to slot c % nslot
  const uint8_t* my = src + (size_t)blockIdx.x * region_bytes;
  const size_t per_region = region_bytes / (size_t)slot_bytes;       // copies per pass over the region
  bool ok = true;
  for (int s = me; s < nslot; s += issuers) {
    // first round of this slot
    if (s < iters) {
      ptx::mbar_expect_tx(&full[s], (uint32_t)slot_bytes);
      ptx::bulk_g2s(sm + (size_t)s * slot_bytes, my + ((size_t)s % per_region) * (size_t)slot_bytes, (uint32_t)slot_bytes, &full[s]);
    }
  }
  for (int round = 1; ok; ++round) {
    bool any = false;
    for (int s = me; s < nslot && ok; s += issuers) {
      const int prev = (round - 1) * nslot + s, c = round * nslot + s;
      if (prev >= iters) continue;
      any = true;
      ok = ptx::mbar_wait(&full[s], (uint32_t)(round - 1) & 1u);       // the copy of the previous round has landed
      if (ok && c < iters) {
        ptx::mbar_expect_tx(&full[s], (uint32_t)slot_bytes);
        ptx::bulk_g2s(sm + (size_t)s * slot_bytes, my + ((size_t)c % per_region) * (size_t)slot_bytes, (uint32_t)slot_bytes, &full[s]);
      }
    }
    if (!any) break;
  }
  if (!ok) atomicOr(&flags[FLAG_TIMEOUT], 1u);
}

// a bounded wait that is made to run out: nothing ever arrives on the barrier
__global__ void wait_timeout_kernel(uint32_t polls, uint32_t* __restrict__ flags)
{
  __shared__ __align__(8) uint64_t bar;
  ptx::mbar_init(&bar, 1);
  ptx::fence_barrier_init();
  if (!ptx::mbar_wait(&bar, 0, polls)) atomicOr(&flags[FLAG_TIMEOUT], 1u);
}

}  // namespace sdq

using namespace sdq;

extern "C" sdq_status_t sdq_diag_wait_timeout(int polls, void* stream)
{
  if (polls < 1 || polls > 4096) return SDQ_ERR_SHAPE;
  uint32_t* flags = device_flags();
  if (!flags) return SDQ_ERR_CUDA;
  wait_timeout_kernel<<<1, 1, 0, (cudaStream_t)stream>>>((uint32_t)polls, flags);
  return cudaGetLastError() == cudaSuccess ? SDQ_OK : SDQ_ERR_CUDA;
}

extern "C" sdq_status_t sdq_diag_l2_copy(const void* src, size_t src_bytes, int slot_bytes, int nslot, int issuers, int iters,
                                         size_t* bytes_moved, void* stream)
{
  if (!src || !bytes_moved) return SDQ_ERR_INVALID_ARG;
  if ((uintptr_t)src & 15) return SDQ_ERR_ALIGNMENT;
  DeviceInfo* dinfo = device_info();
  if (!dinfo) return SDQ_ERR_CUDA;
  const int sm_count = dinfo->sm_count;
  const size_t region = (src_bytes / (size_t)sm_count) & ~(size_t)127;
  if (slot_bytes < 1024 || (slot_bytes & 127) || nslot < 1 || nslot > 16 || issuers < 1 || issuers > 4 || iters < 1 || (size_t)nslot * slot_bytes > 220 * 1024 ||
      region < (size_t)slot_bytes)
    return SDQ_ERR_SHAPE;
  if (!dinfo->diag_attr) {
    if (cudaFuncSetAttribute(l2_copy_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024 + 128) != cudaSuccess) return SDQ_ERR_CUDA;
    dinfo->diag_attr = 1;
  }
  uint32_t* flags = device_flags();
  if (!flags) return SDQ_ERR_CUDA;
  l2_copy_kernel<<<sm_count, 128, (size_t)nslot * slot_bytes + 128, (cudaStream_t)stream>>>((const uint8_t*)src, region, iters, nslot, slot_bytes, issuers,
                                                                                             flags);
  if (cudaGetLastError() != cudaSuccess) return SDQ_ERR_CUDA;
  *bytes_moved = (size_t)sm_count * (size_t)iters * (size_t)slot_bytes;
  return SDQ_OK;
}
