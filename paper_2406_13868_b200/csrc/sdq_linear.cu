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
#include "sdq_linear.h"
#include "sdq_ptx.cuh"

namespace sdq {

constexpr int LIN_THREADS = 192;
constexpr int NSLOT = 5;
constexpr int SLOT_BYTES = 45056;              // one ring slot holds either an inlier or an outlier stage
constexpr int SL_A = 0;                        // WI record (A_in | E_in | SFA_in) or WO record (A_out | E_out)
constexpr int SL_B = 10752;                    // B4 (256 K) or B8 (128 K) of up to 256 tokens: 32768 B
constexpr int SL_SF = SL_B + 32768;            // inlier: SFB_in atoms (2 x 512); outlier stage 0: SFA_out | SFB_out x 2
constexpr int SM_STG = NSLOT * SLOT_BYTES;      // epilogue transpose buffer: 16 tokens x 128 features bf16
constexpr int SM_BARS = SM_STG + 4096;
constexpr int LIN_SMEM = SM_BARS + 128 + 128;  // + barriers + alignment slack

// TMEM columns
constexpr uint32_t TM_D = 0;          // accumulator: up to 256 columns (tokens)
constexpr uint32_t TM_I = 256;        // 2 buffers x 16 columns: E_in 4 | SFA_in 4 | SFB_in 8
constexpr uint32_t TM_EO = 288;       // 2 buffers x 4 columns: E_out
constexpr uint32_t TM_SFA_OUT = 296;  // 4 columns
constexpr uint32_t TM_SFB_OUT = 300;  // 8 columns



template <bool F32_OUT>
__global__ void __launch_bounds__(LIN_THREADS, 1)
sdq_linear_kernel(const LinearParams p)
{
  extern __shared__ uint8_t smem_raw[];
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint8_t* sm = smem_raw + ((128 - (ptx::smem_u32(smem_raw) & 127)) & 127);
  uint64_t* full = reinterpret_cast<uint64_t*>(sm + SM_BARS);
  uint64_t* empty = full + NSLOT;
  uint64_t* acc_full = empty + NSLOT;
  uint64_t* acc_empty = acc_full + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 1);

  const int n_tile = p.n_tile;
  const int RT = (int)(p.N / TILE_ROWS);
  const int T1 = p.out_n ? (int)(p.K / K1) : 0, T2 = (int)(p.K / K2);
  const int n_atiles = (n_tile + TILE_TOK - 1) / TILE_TOK;     // 128-token activation tiles per token tile

  if (tid == 0) {
    for (int s = 0; s < NSLOT; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
    ptx::mbar_init(acc_full, 1);
    ptx::mbar_init(acc_empty, 4);
    ptx::fence_barrier_init();
  }
  if (warp == 1) ptx::tmem_alloc(tmem_slot, 512);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    if (lane < NSLOT) {
      // ---------------- producer: bulk copies, inlier stages of the tile first, then its outlier stages.
      // Lane l owns ring slot l, so the barrier round trips of different slots overlap.
      bool ok = true;
      uint32_t it = 0;
      for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x) {
        const int rt = tile % RT, mtile = tile / RT;
        const int64_t m0 = (int64_t)mtile * n_tile;
        const int64_t mt = m0 / TILE_TOK;
        const int have = (int)min((int64_t)n_atiles, p.aoff.MT - mt);     // activation tiles that exist
        const uint32_t tok_bytes = (uint32_t)min(n_tile, TILE_TOK) * 128u;   // bytes per activation tile per stage
        const uint8_t* wi = p.w + p.poff.wi + (size_t)rt * T2 * WI_BYTES;
        const uint8_t* wo = p.w + p.poff.wo + (size_t)rt * T1 * WO_BYTES;
        const uint8_t* xi = p.x + p.aoff.xi + (size_t)mt * T2 * XI_BYTES;
        const uint8_t* xo = p.x + p.aoff.xo + (size_t)mt * T1 * XO_BYTES;
        for (int k = 0; k < T2 + T1 && ok; ++k, ++it) {
          const uint32_t s = it % NSLOT;
          if (s != lane) continue;
          if (it >= NSLOT) ok = ptx::mbar_wait(&empty[s], ((it / NSLOT) - 1) & 1);
          if (!ok) break;
          uint8_t* st = sm + (size_t)s * SLOT_BYTES;
          if (k < T2) {
            ptx::mbar_expect_tx(&full[s], WI_BYTES + (uint32_t)have * (tok_bytes + SF_ATOM_BYTES));
            ptx::bulk_g2s(st + SL_A, wi + (size_t)k * WI_BYTES, WI_BYTES, &full[s]);
            for (int a = 0; a < have; ++a) {
              const uint8_t* src = xi + ((size_t)a * T2 + k) * XI_BYTES;
              ptx::bulk_g2s(st + SL_B + a * B4_BYTES, src, tok_bytes, &full[s]);
              ptx::bulk_g2s(st + SL_SF + a * SF_ATOM_BYTES, src + B4_BYTES, SF_ATOM_BYTES, &full[s]);
            }
          } else {
            const int k1 = k - T2;
            const uint32_t sf_bytes = (k1 == 0) ? (uint32_t)(1 + have) * SF_ATOM_BYTES : 0u;
            ptx::mbar_expect_tx(&full[s], WO_BYTES + (uint32_t)have * tok_bytes + sf_bytes);
            ptx::bulk_g2s(st + SL_A, wo + (size_t)k1 * WO_BYTES, WO_BYTES, &full[s]);
            for (int a = 0; a < have; ++a)
              ptx::bulk_g2s(st + SL_B + a * B8_BYTES, xo + ((size_t)a * T1 + k1) * XO_BYTES, tok_bytes, &full[s]);
            if (k1 == 0) {
              ptx::bulk_g2s(st + SL_SF, p.w + p.poff.sfa_out + (size_t)rt * SF_ATOM_BYTES, SF_ATOM_BYTES, &full[s]);
              for (int a = 0; a < have; ++a)
                ptx::bulk_g2s(st + SL_SF + (1 + a) * SF_ATOM_BYTES, p.x + p.aoff.sfb_out + (size_t)(mt + a) * SF_ATOM_BYTES,
                              SF_ATOM_BYTES, &full[s]);
            }
          }
        }
      }
      if (!ok) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------- MMA issuer
      bool ok = true;
      const uint32_t smb = ptx::smem_u32(sm);
      uint32_t it = 0, tcount = 0;
      bool ready = false;
      const uint32_t id4[2] = {ptx::idesc_block_scaled(128, (uint32_t)n_tile, 1, true, 0, 0),
                               ptx::idesc_block_scaled(128, (uint32_t)n_tile, 1, true, 2, 2)};
      const uint32_t id8 = ptx::idesc_block_scaled(128, (uint32_t)n_tile, 0, true, 0, 0);
      for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x, ++tcount) {
        if (tcount > 0) {   // the epilogue must have drained the accumulator of the previous tile
          ok = ptx::mbar_wait(acc_empty, (tcount - 1) & 1);
          if (!ok) break;
          ptx::tc_fence_after();
        }
        for (int k = 0; k < T2 + T1 && ok; ++k, ++it) {
          const uint32_t s = it % NSLOT;
          if (!ready) ok = ptx::mbar_wait(&full[s], (it / NSLOT) & 1);
          if (!ok) break;
          ptx::tc_fence_after();
          // poll the next slot now: the answer is back by the time this stage's instructions are issued
          ready = ptx::mbar_test(&full[(it + 1) % NSLOT], ((it + 1) / NSLOT) & 1);
          const uint32_t st = smb + s * SLOT_BYTES;
          if (k < T2) {
            // inlier stage: 256 logical K = 2 sparse MXFP4 MMAs; metadata and scale atoms go to TMEM first
            const uint32_t mb = tmem + TM_I + 16u * (uint32_t)(k & 1);
            ptx::tc_cp_128x128b(mb + 0, ptx::smem_desc(st + SL_A + A_IN_BYTES, 0, 128));
            ptx::tc_cp_32x128b_warpx4(mb + 4, ptx::smem_desc(st + SL_A + A_IN_BYTES + E_IN_BYTES, 0, 128));
            ptx::tc_cp_32x128b_warpx4(mb + 8, ptx::smem_desc(st + SL_SF, 0, 128));
            if (n_atiles > 1) ptx::tc_cp_32x128b_warpx4(mb + 12, ptx::smem_desc(st + SL_SF + SF_ATOM_BYTES, 0, 128));
#pragma unroll
            for (uint32_t j = 0; j < 2; ++j)
              ptx::mma_sp_mxf4(tmem + TM_D, ptx::smem_desc(st + SL_A + j * 4096, 128, 256),
                               ptx::smem_desc(st + SL_B + j * 512, 128, 1024), id4[j], mb + 2 * j, mb + 4, mb + 8,
                               (k > 0 || j > 0) ? 1u : 0u);
          } else {
            // outlier stage: 128 logical K = 2 sparse FP8 MMAs; the row / token scales (E8M0) arrive with stage 0
            const int k1 = k - T2;
            const uint32_t eb = tmem + TM_EO + 4u * (uint32_t)(k1 & 1);
            ptx::tc_cp_128x128b(eb, ptx::smem_desc(st + SL_A + A_OUT_BYTES, 0, 128));
            if (k1 == 0) {
              ptx::tc_cp_32x128b_warpx4(tmem + TM_SFA_OUT, ptx::smem_desc(st + SL_SF, 0, 128));
              ptx::tc_cp_32x128b_warpx4(tmem + TM_SFB_OUT, ptx::smem_desc(st + SL_SF + SF_ATOM_BYTES, 0, 128));
              if (n_atiles > 1)
                ptx::tc_cp_32x128b_warpx4(tmem + TM_SFB_OUT + 4, ptx::smem_desc(st + SL_SF + 2 * SF_ATOM_BYTES, 0, 128));
            }
#pragma unroll
            for (uint32_t j = 0; j < 2; ++j)
              ptx::mma_sp_mxf8(tmem + TM_D, ptx::smem_desc(st + SL_A + j * 4096, 128, 256),
                               ptx::smem_desc(st + SL_B + j * 512, 128, 1024), id8, eb + 2 * j, tmem + TM_SFA_OUT,
                               tmem + TM_SFB_OUT, 1u);
          }
          ptx::tc_commit(&empty[s]);
        }
        ptx::tc_commit(acc_full);
      }
      if (!ok) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
    }
  } else {
    // ---------------- epilogue: warp w owns TMEM lanes 32*(w%4) .. +31 (weight rows), columns = tokens
    const uint32_t q = warp & 3;
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x, ++tcount) {
      const int rt = tile % RT, mtile = tile / RT;
      const int64_t m0 = (int64_t)mtile * n_tile;
      const int n_valid = (int)min((int64_t)n_tile, p.M - m0);
      ok = ptx::mbar_wait(acc_full, tcount & 1);
      ptx::tc_fence_after();
      if (!ok) break;
      const int64_t n0 = (int64_t)rt * TILE_ROWS;
      const uint32_t et = (warp - 2) * 32 + lane;     // 0..127 among the epilogue threads
#pragma unroll 1
      for (int c0 = 0; c0 < n_tile; c0 += 16) {
        uint32_t v[16];
        if (c0 < n_valid) {
          ptx::tmem_ld_32x32b_x16(tmem + ((q * 32u) << 16) + TM_D + (uint32_t)c0, v);
          ptx::tmem_ld_wait();
        }
        if (c0 + 16 >= n_tile) {      // accumulator fully read: hand TMEM back before the stores
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(acc_empty);
        }
        if (c0 >= n_valid) continue;  // uniform over the four epilogue warps
        if (F32_OUT) {
          float* Y = reinterpret_cast<float*>(p.Y);
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (c0 + j < n_valid) Y[(m0 + c0 + j) * p.ldy + n0 + q * 32 + lane] = __uint_as_float(v[j]);
        } else {
          // transpose through shared memory: [16 tokens][128 features] bf16, then 16-byte stores of full 256 B rows
          __nv_bfloat16* stg = reinterpret_cast<__nv_bfloat16*>(sm + SM_STG);
#pragma unroll
          for (int j = 0; j < 16; ++j) stg[j * 128 + q * 32 + lane] = __float2bfloat16_rn(__uint_as_float(v[j]));
          ptx::named_bar_sync(1, 128);
          __nv_bfloat16* Y = reinterpret_cast<__nv_bfloat16*>(p.Y);
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            const uint32_t idx = i * 128 + et, tok = idx >> 4, seg = idx & 15;
            if (c0 + (int)tok < n_valid) {
              const uint4 w = *reinterpret_cast<const uint4*>(stg + tok * 128 + seg * 8);
              *reinterpret_cast<uint4*>(Y + (m0 + c0 + tok) * p.ldy + n0 + seg * 8) = w;
            }
          }
          ptx::named_bar_sync(1, 128);   // the buffer is rewritten by the next chunk
        }
      }
    }
    if (!ok && lane == 0) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
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
  p.n_tile = M > 128 ? 256 : (M > 64 ? 128 : (M > 32 ? 64 : (M > 16 ? 32 : 16)));
  p.n_mtiles = (int)((M + p.n_tile - 1) / p.n_tile);
  p.total_tiles = (int)(P->N / TILE_ROWS) * p.n_mtiles;
  p.Y = Y; p.ldy = ldy;
  p.flags = device_flags();
  if (!p.flags) return SDQ_ERR_CUDA;
  static int sm_count = 0;
  if (!sm_count) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SDQ_ERR_CUDA;
  }
  dim3 grid((unsigned)(p.total_tiles < sm_count ? p.total_tiles : sm_count));
  if (f32) sdq_linear_kernel<true><<<grid, LIN_THREADS, LIN_SMEM, (cudaStream_t)stream>>>(p);
  else sdq_linear_kernel<false><<<grid, LIN_THREADS, LIN_SMEM, (cudaStream_t)stream>>>(p);
  return cudaGetLastError() == cudaSuccess ? SDQ_OK : SDQ_ERR_CUDA;
}

extern "C" sdq_status_t sdq_linear(const sdq_act_t* Xq, const sdq_packed_t* P, void* Y, int64_t ldy, void* stream)
{ return launch_linear(Xq, P, Y, ldy, stream, false); }

extern "C" sdq_status_t sdq_linear_f32(const sdq_act_t* Xq, const sdq_packed_t* P, float* Y, int64_t ldy, void* stream)
{ return launch_linear(Xq, P, (void*)Y, ldy, stream, true); }
