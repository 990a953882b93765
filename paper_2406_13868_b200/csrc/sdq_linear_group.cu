// Grouped decomposed GEMM for few tokens: several independent linear layers in ONE persistent launch
//   Y_i = A_i,in W_i,in^T + A_i,out W_i,out^T   (Section 5.1: O = O_i + O_o, per layer i)
//
// With a handful of tokens a layer is a stream of its packed weights through the tensor core, and one launch per
// layer costs more than the stream itself (set-up, the dependency on the previous grid, the split-K reduction).  Here
// the work items (layer, 128-row tile) of all layers of the call are dealt out round-robin over one CTA per SM; a CTA
// runs its items back to back through one shared-memory ring, so the weights of the next item are already landing
// while the current one is multiplied and stored, and no K split (hence no reduction) is needed once there are about
// as many row tiles as SMs.
//
// The outlier part is streamed in the form the method states it -- an 8-bit code and a position per S-Vector (the WC
// section, 1.5 bits per weight) -- not as the 2:4 FP8 container of the many-token kernels (5 bits per weight): four
// warps rebuild the container of each 128-K stage in shared memory (one weight row per thread, 80 bytes written)
// while the tensor core works on earlier stages.  Streamed bytes: 2.625 + 1.5 = 4.125 bits per weight against 4.0
// algorithmic.
//
// Warps: 0 bulk-copy producer (four lanes, one ring slot each per trip), 1 MMA issuer (warp-uniform loop, one elected
// lane issues; also copies metadata and scales to TMEM), 2..5 epilogue (two alternating accumulators of 32 columns:
// the next item's MMAs never wait for the stores), 6..9 outlier container builders.  A ring slot holds 256 K of one
// item: either the inlier record with the tokens' 4-bit codes and scales, or two compact outlier records with the
// tokens' 8-bit codes.  Every wait is bounded; a timeout sets the sticky flag.
#include <cuda_bf16.h>

#include "sdq_internal.h"
#include "sdq_layout.h"
#include "sdq_linear.h"
#include "sdq_ptx.cuh"

namespace sdq {

constexpr int GRP_THREADS = 320;
constexpr int GRP_NCB = 4;                       // container buffers (A_out | E_out of one 128-K stage each)
constexpr int GRP_MAX_SLOTS = 16;
constexpr uint32_t GRP_TM_ACC = 0;               // two accumulators of 32 columns
constexpr uint32_t GRP_TM_I = 64;                // 2 x 12: E_in 4 | SFA_in 4 | SFB_in 4
constexpr uint32_t GRP_TM_EO = 88;               // 2 x 4: E_out
constexpr uint32_t GRP_TM_SO = 96;               // 2 x 8: SFA_out 4 | SFB_out 4 (per item)
constexpr uint32_t GRP_TMEM_COLS = 128;

__host__ __device__ inline int group_slot_bytes(int n_tile) {
  const int xb = n_tile * 128;
  const int is = WI_BYTES + xb + SF_ATOM_BYTES, os = 2 * wc_bytes(1) + 2 * xb + 2 * SF_ATOM_BYTES;
  return is > os ? is : os;
}

// matrix of work item `item` (items are numbered matrix by matrix)
__device__ __forceinline__ int group_mat_of(const GroupParams& p, int item) {
  int i = 0;
  while (i + 1 < p.n && item >= p.m[i + 1].item0) ++i;
  return i;
}

template <bool F32_OUT>
__global__ void __launch_bounds__(GRP_THREADS, 1)
sdq_linear_group_kernel(const __grid_constant__ GroupParams p)
{
  extern __shared__ uint8_t smem_raw[];
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint8_t* sm = smem_raw + ((128 - (ptx::smem_u32(smem_raw) & 127)) & 127);
  const uint32_t nslot = (uint32_t)p.nslot, slot_bytes = (uint32_t)p.slot_bytes, xb = (uint32_t)p.n_tile * 128u;
  uint8_t* cbuf = sm + nslot * slot_bytes;                                   // GRP_NCB container buffers of WO_BYTES
  uint64_t* full = reinterpret_cast<uint64_t*>(cbuf + GRP_NCB * WO_BYTES);   // slot s has landed
  uint64_t* empty = full + GRP_MAX_SLOTS;                                    // the MMAs that read slot s have completed
  uint64_t* cb_full = empty + GRP_MAX_SLOTS;                                 // container buffer c is built
  uint64_t* cb_empty = cb_full + GRP_NCB;                                    // the MMAs that read container buffer c have completed
  uint64_t* acc_full = cb_empty + GRP_NCB;                                   // [2]
  uint64_t* acc_empty = acc_full + 2;                                        // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  if (tid == 0) ptx::griddep_launch_dependents();
  if (tid == 0) {
    for (uint32_t s = 0; s < nslot; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
    for (int c = 0; c < GRP_NCB; ++c) { ptx::mbar_init(&cb_full[c], 128); ptx::mbar_init(&cb_empty[c], 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(&acc_full[a], 1); ptx::mbar_init(&acc_empty[a], 4); }
    ptx::fence_barrier_init();
  }
  if (warp == 1) ptx::tmem_alloc(tmem_slot, GRP_TMEM_COLS);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const int first = (int)blockIdx.x, stride = (int)gridDim.x;

  if (warp == 0) {
    if (lane < 4) {
      // ---------------- producer: lane l fills the ring slots q = l, l + 4, ... of this CTA's slot sequence
      ptx::griddep_wait();                 // activations come from an earlier kernel
      bool ok = true;
      int item = first, j = (int)lane;     // this lane's position: work item and slot number inside the item
      int mat = -1, rt = 0, per_item = 0;
      for (uint32_t q = lane; ok; q += 4) {
        // advance to the item that holds slot j
        for (;;) {
          if (item >= p.total_items) break;
          if (mat < 0) {
            mat = group_mat_of(p, item);
            rt = item - p.m[mat].item0;
            per_item = p.m[mat].T2 * (p.m[mat].out_n ? 2 : 1);
          }
          if (j < per_item) break;
          j -= per_item; item += stride; mat = -1;
        }
        if (item >= p.total_items) break;
        const GroupMat& m = p.m[mat];
        const uint32_t s = q % nslot;
        if (q >= nslot && !(ok = ptx::mbar_wait(&empty[s], ((q / nslot) - 1) & 1))) break;
        uint8_t* st = sm + (size_t)s * slot_bytes;
        const int k2 = m.out_n ? (j >> 1) : j;
        if (!m.out_n || !(j & 1)) {
          // inlier slot: | WI record | 4-bit codes of the tokens | their scale atom |
          const uint8_t* xi = m.x + m.xi + (size_t)k2 * XI_BYTES;
          ptx::mbar_expect_tx(&full[s], WI_BYTES + xb + SF_ATOM_BYTES);
          ptx::bulk_g2s(st, m.w + m.wi + ((size_t)rt * m.T2 + k2) * WI_BYTES, WI_BYTES, &full[s]);
          ptx::bulk_g2s(st + WI_BYTES, xi, xb, &full[s]);
          ptx::bulk_g2s(st + WI_BYTES + xb, xi + B4_BYTES, SF_ATOM_BYTES, &full[s]);
        } else {
          // outlier slot: | two compact records (128 K each) | 8-bit codes of the tokens, 2 x 128 K | row / token scale atoms (first only) |
          const uint32_t wcb = 2u * (uint32_t)wc_bytes(1);
          const uint8_t* xo = m.x + m.xo + (size_t)(2 * k2) * XO_BYTES;
          ptx::mbar_expect_tx(&full[s], wcb + 2 * xb + (k2 == 0 ? 2u * SF_ATOM_BYTES : 0u));
          ptx::bulk_g2s(st, m.w + m.wc + ((size_t)rt * 2 * m.T2 + 2 * k2) * (size_t)wc_bytes(1), wcb, &full[s]);
          ptx::bulk_g2s(st + wcb, xo, xb, &full[s]);
          ptx::bulk_g2s(st + wcb + xb, xo + XO_BYTES, xb, &full[s]);
          if (k2 == 0) {
            ptx::bulk_g2s(st + wcb + 2 * xb, m.w + m.sfa_out + (size_t)rt * SF_ATOM_BYTES, SF_ATOM_BYTES, &full[s]);
            ptx::bulk_g2s(st + wcb + 2 * xb + SF_ATOM_BYTES, m.x + m.sfb_out, SF_ATOM_BYTES, &full[s]);
          }
        }
        j += 4;
      }
      if (!ok) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: warp-uniform loop, one elected lane issues (descriptors and TMEM addresses are
    // uniform-register operands).  tcgen05.cp and tcgen05.mma of one thread execute in issue order, so metadata and
    // scales need no barrier of their own; their TMEM buffers alternate.
    bool ok = true;
    const uint32_t smb = ptx::smem_u32(sm), cbb = ptx::smem_u32(cbuf);
    const uint32_t id4[2] = {ptx::idesc_block_scaled(128, (uint32_t)p.n_tile, 1, true, 0, 0), ptx::idesc_block_scaled(128, (uint32_t)p.n_tile, 1, true, 2, 2)};
    const uint32_t id8 = ptx::idesc_block_scaled(128, (uint32_t)p.n_tile, 0, true, 0, 0);
    const uint32_t wcb = 2u * (uint32_t)wc_bytes(1);
    uint32_t q = 0, cbq = 0, itc = 0;
    for (int item = first; item < p.total_items && ok; item += stride, ++itc) {
      const int mat = group_mat_of(p, item);
      const int T2 = p.m[mat].T2, out_n = p.m[mat].out_n;
      const uint32_t ab = itc & 1, acc_col = tmem + GRP_TM_ACC + 32u * ab, so = tmem + GRP_TM_SO + 8u * ab;
      if (itc >= 2) {    // the epilogue has read this accumulator's previous item
        ok = __all_sync(0xffffffffu, ptx::mbar_wait(&acc_empty[ab], ((itc >> 1) - 1) & 1));
        if (!ok) break;
      }
      for (int k2 = 0; k2 < T2 && ok; ++k2) {
        // one trip per 256 K: the inlier slot, the outlier slot and its two rebuilt containers.  A trip of this loop
        // (waits, vote, election) costs far more than its MMAs of 16 or 32 columns, so it takes as much as it can.
        const uint32_t s = q % nslot, s2 = (q + 1) % nslot, c0 = cbq % GRP_NCB, c1 = (cbq + 1) % GRP_NCB;
        bool rdy = ptx::mbar_wait(&full[s], (q / nslot) & 1);
        if (out_n)
          rdy = rdy && ptx::mbar_wait(&full[s2], ((q + 1) / nslot) & 1) && ptx::mbar_wait(&cb_full[c0], (cbq / GRP_NCB) & 1) &&
                ptx::mbar_wait(&cb_full[c1], ((cbq + 1) / GRP_NCB) & 1);
        ok = __all_sync(0xffffffffu, rdy);
        if (!ok) break;
        ptx::tc_fence_after();
        if (ptx::elect_one()) {
          const uint32_t sb = smb + s * slot_bytes, mb = tmem + GRP_TM_I + 12u * (uint32_t)(k2 & 1);
          ptx::tc_cp_128x128b(mb, ptx::smem_desc(sb + A_IN_BYTES, 0, 128));
          ptx::tc_cp_32x128b_warpx4(mb + 4, ptx::smem_desc(sb + A_IN_BYTES + E_IN_BYTES, 0, 128));
          ptx::tc_cp_32x128b_warpx4(mb + 8, ptx::smem_desc(sb + WI_BYTES + xb, 0, 128));
          ptx::mma_sp_mxf4(acc_col, ptx::smem_desc(sb, 128, 256), ptx::smem_desc(sb + WI_BYTES, 128, 1024), id4[0], mb, mb + 4, mb + 8,
                           k2 ? 1u : 0u);
          ptx::mma_sp_mxf4(acc_col, ptx::smem_desc(sb + 4096, 128, 256), ptx::smem_desc(sb + WI_BYTES + 512, 128, 1024), id4[1], mb + 2,
                           mb + 4, mb + 8, 1u);
          ptx::tc_commit(&empty[s]);
          if (out_n) {
            const uint32_t ob = smb + s2 * slot_bytes;
            if (k2 == 0) {
              ptx::tc_cp_32x128b_warpx4(so, ptx::smem_desc(ob + wcb + 2 * xb, 0, 128));
              ptx::tc_cp_32x128b_warpx4(so + 4, ptx::smem_desc(ob + wcb + 2 * xb + SF_ATOM_BYTES, 0, 128));
            }
#pragma unroll
            for (uint32_t h = 0; h < 2; ++h) {
              const uint32_t c = h ? c1 : c0;
              const uint32_t ca = cbb + c * WO_BYTES, eb = tmem + GRP_TM_EO + 4u * h, xa = ob + wcb + h * xb;
              ptx::tc_cp_128x128b(eb, ptx::smem_desc(ca + A_OUT_BYTES, 0, 128));
              ptx::mma_sp_mxf8(acc_col, ptx::smem_desc(ca, 128, 256), ptx::smem_desc(xa, 128, 1024), id8, eb, so, so + 4, 1u);
              ptx::mma_sp_mxf8(acc_col, ptx::smem_desc(ca + 4096, 128, 256), ptx::smem_desc(xa + 512, 128, 1024), id8, eb + 2, so, so + 4, 1u);
              ptx::tc_commit(&cb_empty[c]);
            }
            ptx::tc_commit(&empty[s2]);
          }
        }
        __syncwarp();
        q += out_n ? 2u : 1u;
        cbq += out_n ? 2u : 0u;
      }
      if (ok && ptx::elect_one()) ptx::tc_commit(&acc_full[ab]);
      __syncwarp();
    }
    if (!ok && lane == 0) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
  } else if (warp >= 2 && warp <= 5) {
    // ---------------- epilogue: warp w owns TMEM lanes 32 (w % 4) .. + 31 (weight rows), columns = tokens
    const uint32_t qd = warp & 3;
    bool ok = true;
    uint32_t itc = 0;
    ptx::griddep_wait();                   // Y may still be in use by the previous kernel
    for (int item = first; item < p.total_items && ok; item += stride, ++itc) {
      const int mat = group_mat_of(p, item);
      const GroupMat& m = p.m[mat];
      const int64_t n0 = (int64_t)(item - m.item0) * TILE_ROWS;
      const uint32_t ab = itc & 1;
      ok = ptx::mbar_wait(&acc_full[ab], (itc >> 1) & 1);
      ptx::tc_fence_after();
      if (!ok) break;
      uint32_t v[32];
      {
        uint32_t a[16], b[16];
        const uint32_t tb = tmem + ((qd * 32u) << 16) + GRP_TM_ACC + 32u * ab;
        ptx::tmem_ld_32x32b_x16(tb, a);
        if (p.n_tile > 16) ptx::tmem_ld_32x32b_x16(tb + 16, b);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i) { v[i] = a[i]; v[16 + i] = (p.n_tile > 16) ? b[i] : 0u; }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&acc_empty[ab]);
#pragma unroll
      for (int t = 0; t < 32; ++t) {
        if (t < m.M) {
          const int64_t idx = (int64_t)t * m.ldy + n0 + qd * 32 + lane;
          if (F32_OUT) reinterpret_cast<float*>(m.Y)[idx] = __uint_as_float(v[t]);
          else reinterpret_cast<__nv_bfloat16*>(m.Y)[idx] = __float2bfloat16_rn(__uint_as_float(v[t]));
        }
      }
    }
    if (!ok && lane == 0) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
  } else {
    // ---------------- outlier container builders (warps 6..9): thread r rebuilds weight row r of a 128-K stage from its
    // 16 codes + 16 positions: per S-Vector of 8 the code goes to the 2:4 slot of its group of 4 (two ascending slot
    // indices per 4: (p, 3) with the value first, or (0, 3) with the value second when p = 3; a group without outlier
    // gets (0, 1) and zeros), the form the packer writes for the many-token kernels.
    const uint32_t r = (warp - 6) * 32 + lane;
    bool ok = true;
    uint32_t q = 0, cbq = 0;
    for (int item = first; item < p.total_items && ok; item += stride) {
      const int mat = group_mat_of(p, item);
      const int T2 = p.m[mat].T2, out_n = p.m[mat].out_n;
      if (!out_n) { q += (uint32_t)T2; continue; }
      for (int k2 = 0; k2 < T2 && ok; ++k2) {
        ++q;                                               // the inlier slot
        const uint32_t s = q % nslot;
        if (!(ok = ptx::mbar_wait(&full[s], (q / nslot) & 1))) break;
        const uint8_t* st = sm + (size_t)s * slot_bytes;
        // both containers of the slot must be free again (they are released in order)
        if (cbq + 1 >= GRP_NCB && !(ok = ptx::mbar_wait(&cb_empty[(cbq + 1) % GRP_NCB], (((cbq + 1) / GRP_NCB) - 1) & 1))) break;
#pragma unroll
        for (uint32_t h = 0; h < 2; ++h, ++cbq) {
          const uint32_t c = cbq % GRP_NCB;
          const uint4 codes = *reinterpret_cast<const uint4*>(st + h * (uint32_t)wc_bytes(1) + r * 16);
          const uint2 pos = *reinterpret_cast<const uint2*>(st + h * (uint32_t)wc_bytes(1) + WC_CODE_BYTES + r * 8);
          const uint32_t cw[4] = {codes.x, codes.y, codes.z, codes.w}, pw[2] = {pos.x, pos.y};
          uint32_t stored[16], meta[4] = {0u, 0u, 0u, 0u};
#pragma unroll
          for (int g = 0; g < 16; ++g) {
            // position ps (0..7) of the outlier in its S-Vector: it sits in the group of 4 number ps >> 2 at p = ps & 3.  Stored
            // bytes of the S-Vector (two per group of 4): the code moves to byte (p == 3) + 2 (ps >> 2); metadata byte = the two
            // groups' slot-index nibbles, (p, 3) or (0, 3) for p = 3 where the outlier is, (0, 1) elsewhere -- both from
            // 8-entry byte tables held in two registers each
            const uint32_t code = __byte_perm(cw[g >> 2], 0u, 0x4440u + (uint32_t)(g & 3));
            const uint32_t ps = (pw[g >> 3] >> (4 * (g & 7))) & 7u;
            const uint32_t sh = __byte_perm(0x08000000u, 0x18101010u, ps) & 0xFFu;
            stored[g] = code << sh;
            const uint32_t mbyte = __byte_perm(0x4C4E4D4Cu, 0xC4E4D4C4u, ps) & 0xFFu;
            meta[g >> 2] |= mbyte << (8 * (g & 3));
          }
          uint8_t* cb = cbuf + (size_t)c * WO_BYTES;
          // row r: bytes 0..31 of its 64 stored bytes belong to K-block 0, 32..63 to K-block 1; 16-byte chunks 128 B apart
          uint8_t* arow = cb + (r >> 3) * 256 + (r & 7) * 16;
          *reinterpret_cast<uint4*>(arow) = make_uint4(stored[0], stored[1], stored[2], stored[3]);
          *reinterpret_cast<uint4*>(arow + 128) = make_uint4(stored[4], stored[5], stored[6], stored[7]);
          *reinterpret_cast<uint4*>(arow + 4096) = make_uint4(stored[8], stored[9], stored[10], stored[11]);
          *reinterpret_cast<uint4*>(arow + 4096 + 128) = make_uint4(stored[12], stored[13], stored[14], stored[15]);
          *reinterpret_cast<uint4*>(cb + A_OUT_BYTES + r * 16) = make_uint4(meta[0], meta[1], meta[2], meta[3]);
        }
        ptx::fence_proxy_async();                          // generic-proxy writes -> visible to the tensor core's reads
        ptx::mbar_arrive(&cb_full[(cbq - 2) % GRP_NCB]);
        ptx::mbar_arrive(&cb_full[(cbq - 1) % GRP_NCB]);
        ++q;
      }
    }
    if (!ok && lane == 0) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) ptx::tmem_dealloc(tmem, GRP_TMEM_COLS);
}

// shared memory of the launch for `n_tile` tokens per tile: as many ring slots as fit beside the container buffers
static int group_nslot(int n_tile) {
  const int avail = 232448 - 128 - GRP_NCB * WO_BYTES - (2 * GRP_MAX_SLOTS + 2 * GRP_NCB + 4 + 1) * 8;
  int n = avail / group_slot_bytes(n_tile);
  n &= ~3;                                  // the four producer lanes walk the ring in step
  return n > GRP_MAX_SLOTS ? GRP_MAX_SLOTS : n;
}

cudaError_t launch_linear_group(GroupParams p, bool f32_out, int sm_count, cudaStream_t stream, uint32_t* attr_done)
{
  p.slot_bytes = group_slot_bytes(p.n_tile);
  p.nslot = group_nslot(p.n_tile);
  const int smem = p.nslot * p.slot_bytes + GRP_NCB * WO_BYTES + (2 * GRP_MAX_SLOTS + 2 * GRP_NCB + 4 + 1) * 8 + 128;
  if (!*attr_done) {
    cudaError_t e = cudaFuncSetAttribute(sdq_linear_group_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(sdq_linear_group_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
    if (e != cudaSuccess) return e;
    *attr_done = 1;
  }
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3((unsigned)(p.total_items < sm_count ? p.total_items : sm_count));
  lc.blockDim = dim3(GRP_THREADS);
  lc.dynamicSmemBytes = (size_t)smem;
  lc.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = 1;
  return f32_out ? cudaLaunchKernelEx(&lc, sdq_linear_group_kernel<true>, p) : cudaLaunchKernelEx(&lc, sdq_linear_group_kernel<false>, p);
}

}  // namespace sdq
