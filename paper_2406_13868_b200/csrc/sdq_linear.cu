// Fused decomposed GEMM  Y = A_i W_i^T + A_o W_o^T   (Section 5.1: O = O_i + O_o)
//
// The sparse operand of tcgen05.mma.sp is A, so the kernel computes Y^T = W X^T: the 128 weight rows
// of a tile sit on the 128 TMEM lanes, tokens on the accumulator columns.  Per 128 logical K:
//   1 x tcgen05.mma.sp kind::mxf4      (pair-wise 4:8 E2M1 inliers x E2M1 activations, E8M0 per 64 K)
//   2 x tcgen05.mma.sp kind::mxf8f6f4  (1:8 / 2:8 E4M3 outliers embedded in 2:4 x E4M3 activations;
//                                       the power-of-two row / token scales ride in as E8M0 factors)
// all into ONE fp32 TMEM accumulator.  Warp roles: warp 0 = bulk-copy (TMA) producer, warp 1 = TMEM
// owner + MMA issuer (also moves metadata / scale atoms smem -> TMEM with tcgen05.cp), warps 2..5 =
// epilogue (tcgen05.ld, convert, transposed store).  Every wait is bounded; a timeout sets a sticky flag.
#include <cuda_bf16.h>

#include "sdq_internal.h"
#include "sdq_layout.h"
#include "sdq_ptx.cuh"

namespace sdq {

constexpr int LIN_THREADS = 192;
constexpr int NSTAGE = 5;
constexpr int STAGE_BYTES = A_IN_BYTES + A_OUT_BYTES + E_OUT_BYTES + W2_BYTES + B4_BYTES + B8_BYTES + X2_BYTES;  // 41984
constexpr int SM_W1 = 0;
constexpr int SM_W2 = SM_W1 + A_IN_BYTES + A_OUT_BYTES + E_OUT_BYTES;  // 14336
constexpr int SM_B4 = SM_W2 + W2_BYTES;                                // 16896
constexpr int SM_B8 = SM_B4 + B4_BYTES;                                // 25088
constexpr int SM_X2 = SM_B8 + B8_BYTES;                                // 41472
constexpr int SM_SFOUT = NSTAGE * STAGE_BYTES;                         // two 512 B atoms
constexpr int SM_BARS = SM_SFOUT + 2 * SF_ATOM_BYTES;
constexpr int LIN_SMEM = SM_BARS + 256 + 1024;                         // + alignment slack

// TMEM columns
constexpr uint32_t TM_D = 0;         // accumulator: up to 128 columns
constexpr uint32_t TM_META = 256;    // 2 buffers x 16 columns: E_in 4 | SFA_in 4 | SFB_in 4 | E_out 4
constexpr uint32_t TM_SFA_OUT = 384;
constexpr uint32_t TM_SFB_OUT = 388;

struct LinearParams {
  const uint8_t* w;      // packed weights
  const uint8_t* x;      // quantized activations
  PackedOffsets poff;
  ActOffsets aoff;
  int64_t M, N, K;
  int out_n;
  int n_tile;            // tokens per CTA: 16..128, multiple of 16
  void* Y;
  int64_t ldy;
  uint32_t* flags;
};

template <bool F32_OUT>
__global__ void __launch_bounds__(LIN_THREADS, 1)
sdq_linear_kernel(const LinearParams p)
{
  extern __shared__ uint8_t smem_raw[];
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint8_t* sm = smem_raw + ((1024 - (ptx::smem_u32(smem_raw) & 1023)) & 1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(sm + SM_BARS);
  uint64_t* empty = full + NSTAGE;
  uint64_t* sf_full = empty + NSTAGE;
  uint64_t* acc_full = sf_full + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);

  const int64_t rt = blockIdx.x, mtile = blockIdx.y;
  const int n_tile = p.n_tile;
  const int T1 = (int)(p.K / K1), T2 = (int)(p.K / K2);
  const int W1B = w1_bytes(p.out_n);
  // token tile of this CTA inside the 128-token activation tiles
  const int64_t m0 = mtile * n_tile;
  const int64_t mt = m0 / TILE_TOK;
  const uint32_t t0 = (uint32_t)(m0 % TILE_TOK);   // multiple of n_tile (n_tile divides 128 or is 128-aligned)

  if (tid == 0) {
    for (int s = 0; s < NSTAGE; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
    ptx::mbar_init(sf_full, 1);
    ptx::mbar_init(acc_full, 1);
    ptx::fence_barrier_init();
  }
  if (warp == 1) ptx::tmem_alloc(tmem_slot, 512);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- producer: one bulk copy per operand block per stage
      const uint8_t* w1 = p.w + p.poff.w1 + (size_t)rt * T1 * W1B;
      const uint8_t* w2 = p.w + p.poff.w2 + (size_t)rt * T2 * W2_BYTES;
      const uint8_t* x1 = p.x + p.aoff.x1 + (size_t)mt * T1 * X1_BYTES;
      const uint8_t* x2 = p.x + p.aoff.x2 + (size_t)mt * T2 * X2_BYTES;
      const uint32_t b4_bytes = (uint32_t)n_tile * 64u, b8_bytes = (uint32_t)n_tile * 128u;
      if (p.out_n) {
        ptx::mbar_expect_tx(sf_full, 2 * SF_ATOM_BYTES);
        ptx::bulk_g2s(sm + SM_SFOUT, p.w + p.poff.sfa_out + (size_t)rt * SF_ATOM_BYTES, SF_ATOM_BYTES, sf_full);
        ptx::bulk_g2s(sm + SM_SFOUT + SF_ATOM_BYTES, p.x + p.aoff.sfb_out + (size_t)mt * SF_ATOM_BYTES, SF_ATOM_BYTES, sf_full);
      }
      bool ok = true;
      for (int it = 0; it < T1 && ok; ++it) {
        const int s = it % NSTAGE;
        if (it >= NSTAGE) ok = ptx::mbar_wait(&empty[s], ((it / NSTAGE) - 1) & 1);
        if (!ok) break;
        uint8_t* st = sm + (size_t)s * STAGE_BYTES;
        const uint32_t tx = (uint32_t)W1B + W2_BYTES + b4_bytes + (p.out_n ? b8_bytes : 0u) + X2_BYTES;
        ptx::mbar_expect_tx(&full[s], tx);
        ptx::bulk_g2s(st + SM_W1, w1 + (size_t)it * W1B, (uint32_t)W1B, &full[s]);
        ptx::bulk_g2s(st + SM_W2, w2 + (size_t)(it >> 1) * W2_BYTES, W2_BYTES, &full[s]);
        ptx::bulk_g2s(st + SM_B4, x1 + (size_t)it * X1_BYTES + (size_t)(t0 >> 3) * 512, b4_bytes, &full[s]);
        if (p.out_n)
          ptx::bulk_g2s(st + SM_B8, x1 + (size_t)it * X1_BYTES + B4_BYTES + (size_t)(t0 >> 3) * 1024, b8_bytes, &full[s]);
        ptx::bulk_g2s(st + SM_X2, x2 + (size_t)(it >> 1) * X2_BYTES, X2_BYTES, &full[s]);
      }
      if (!ok) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------- MMA issuer
      bool ok = true;
      const uint32_t smb = ptx::smem_u32(sm);
      if (p.out_n) {
        ok = ptx::mbar_wait(sf_full, 0);
        ptx::tc_fence_after();
        ptx::tc_cp_32x128b_warpx4(tmem + TM_SFA_OUT, ptx::smem_desc(smb + SM_SFOUT, 0, 128));
        ptx::tc_cp_32x128b_warpx4(tmem + TM_SFB_OUT, ptx::smem_desc(smb + SM_SFOUT + SF_ATOM_BYTES, 0, 128));
      }
      // SFB atoms hold 128 tokens as (t%32)*16 + (t/32)*4: a token tile starting at t0 reads column t0/32
      // and, inside the column, rows from t0%32 -- only tiles of 32+ tokens or t0%32==0 keep that simple,
      // so small tiles (n_tile < 32) always start at t0 % 32 == 0 (enforced by the host).
      const uint32_t sfb_col = t0 >> 5;
      for (int it = 0; it < T1 && ok; ++it) {
        const int s = it % NSTAGE;
        ok = ptx::mbar_wait(&full[s], (it / NSTAGE) & 1);
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t st = smb + (uint32_t)s * STAGE_BYTES;
        const uint32_t meta = tmem + TM_META + 16u * (uint32_t)(it & 1);
        const uint32_t half = (uint32_t)(it & 1);
        ptx::tc_cp_128x128b(meta + 0, ptx::smem_desc(st + SM_W2, 0, 128));
        ptx::tc_cp_32x128b_warpx4(meta + 4, ptx::smem_desc(st + SM_W2 + E_IN_BYTES, 0, 128));
        ptx::tc_cp_32x128b_warpx4(meta + 8, ptx::smem_desc(st + SM_X2, 0, 128));
        if (p.out_n) ptx::tc_cp_128x128b(meta + 12, ptx::smem_desc(st + SM_W1 + A_IN_BYTES + A_OUT_BYTES, 0, 128));
        // inliers: 128 logical K, scales 2*half and 2*half+1 of the 256-K atoms
        ptx::mma_sp_mxf4(tmem + TM_D, ptx::smem_desc(st + SM_W1, 2048, 128), ptx::smem_desc(st + SM_B4, 128, 512),
                         ptx::idesc_block_scaled(128, (uint32_t)n_tile, 1, true, 2 * half, 2 * half), meta + 0 + 2 * half,
                         meta + 4, meta + 8 + sfb_col, it > 0 ? 1u : 0u);
        if (p.out_n) {
#pragma unroll
          for (uint32_t j = 0; j < 2; ++j)
            ptx::mma_sp_mxf8(tmem + TM_D, ptx::smem_desc(st + SM_W1 + A_IN_BYTES + j * 4096, 2048, 128),
                             ptx::smem_desc(st + SM_B8 + j * 512, 128, 1024),
                             ptx::idesc_block_scaled(128, (uint32_t)n_tile, 0, true, 0, 0), meta + 12 + 2 * j, tmem + TM_SFA_OUT,
                             tmem + TM_SFB_OUT + sfb_col, 1u);
        }
        ptx::tc_commit(&empty[s]);
      }
      ptx::tc_commit(acc_full);
      if (!ok) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
    }
  } else {
    // ---------------- epilogue: warp w owns TMEM lanes 32*(w%4) .. +31 (weight rows), columns = tokens
    const bool ok = ptx::mbar_wait(acc_full, 0);
    ptx::tc_fence_after();
    if (!ok) {
      if (lane == 0) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
    } else {
      const uint32_t q = warp & 3;
      const int64_t n = rt * TILE_ROWS + q * 32 + lane;
      for (int c0 = 0; c0 < n_tile; c0 += 16) {
        uint32_t v[16];
        ptx::tmem_ld_32x32b_x16(tmem + ((q * 32u) << 16) + TM_D + (uint32_t)c0, v);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int64_t m = m0 + c0 + j;
          if (m < p.M) {
            if (F32_OUT) reinterpret_cast<float*>(p.Y)[m * p.ldy + n] = __uint_as_float(v[j]);
            else reinterpret_cast<__nv_bfloat16*>(p.Y)[m * p.ldy + n] = __float2bfloat16_rn(__uint_as_float(v[j]));
          }
        }
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) ptx::tmem_dealloc(tmem, 512);
}

}  // namespace sdq

using namespace sdq;

static sdq_status_t launch_linear(const sdq_act_t* Xq, const sdq_packed_t* P, void* Y, int64_t ldy, void* stream, bool f32)
{
  if (!Xq || !P || !Y || !Xq->dev || !P->dev) return SDQ_ERR_INVALID_ARG;
  if (Xq->K != P->K || Xq->M <= 0 || P->N <= 0 || P->N % TILE_ROWS || P->K % K2 || ldy < P->N) return SDQ_ERR_SHAPE;
  if (Xq->cfg.in_block != P->cfg.in_block || Xq->cfg.scale_rule != P->cfg.scale_rule) return SDQ_ERR_SHAPE;
  if (P->cfg.in_gran != SDQ_GRAN_PAIR || P->cfg.in_block != 64) return SDQ_ERR_UNSUPPORTED;
  if (((uintptr_t)Y & 15) || (ldy % 8)) return SDQ_ERR_ALIGNMENT;
  static bool attr_set[2] = {false, false};
  if (!attr_set[f32]) {
    cudaError_t e = f32 ? cudaFuncSetAttribute(sdq_linear_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, LIN_SMEM)
                        : cudaFuncSetAttribute(sdq_linear_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, LIN_SMEM);
    if (e != cudaSuccess) return SDQ_ERR_CUDA;
    attr_set[f32] = true;
  }
  LinearParams p;
  p.w = (const uint8_t*)P->dev;
  p.x = (const uint8_t*)Xq->dev;
  p.poff = packed_offsets(P->N, P->K, P->cfg.out_n);
  p.aoff = act_offsets(Xq->M, Xq->K);
  p.M = Xq->M; p.N = P->N; p.K = P->K;
  p.out_n = P->cfg.out_n;
  const int64_t M = Xq->M;
  p.n_tile = M >= 128 ? 128 : (M > 64 ? 128 : (M > 32 ? 64 : (M > 16 ? 32 : 16)));
  p.Y = Y; p.ldy = ldy;
  p.flags = device_flags();
  if (!p.flags) return SDQ_ERR_CUDA;
  dim3 grid((unsigned)(P->N / TILE_ROWS), (unsigned)((M + p.n_tile - 1) / p.n_tile));
  if (f32) sdq_linear_kernel<true><<<grid, LIN_THREADS, LIN_SMEM, (cudaStream_t)stream>>>(p);
  else sdq_linear_kernel<false><<<grid, LIN_THREADS, LIN_SMEM, (cudaStream_t)stream>>>(p);
  return cudaGetLastError() == cudaSuccess ? SDQ_OK : SDQ_ERR_CUDA;
}

extern "C" sdq_status_t sdq_linear(const sdq_act_t* Xq, const sdq_packed_t* P, void* Y, int64_t ldy, void* stream)
{ return launch_linear(Xq, P, Y, ldy, stream, false); }

extern "C" sdq_status_t sdq_linear_f32(const sdq_act_t* Xq, const sdq_packed_t* P, float* Y, int64_t ldy, void* stream)
{ return launch_linear(Xq, P, (void*)Y, ldy, stream, true); }
