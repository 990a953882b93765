// Fused decomposed GEMM  Y = A_i W_i^T + A_o W_o^T   (Section 5.1: O = O_i + O_o)
//
// The sparse operand of tcgen05.mma.sp is A, so the kernel computes Y^T = W X^T: the 128 weight rows of a
// tile sit on the 128 TMEM lanes, tokens on the accumulator columns.  A tile first runs its inlier K loop
//   2 x tcgen05.mma.sp kind::mxf4 per 256 K     (pair-wise 4:8 E2M1 inliers x E2M1 activations, E8M0 per 64 K)
// then its outlier K loop
//   2 x tcgen05.mma.sp kind::mxf8f6f4 per 128 K (1:8 / 2:8 E4M3 outliers embedded in 2:4 x E4M3 activations;
//                                                the power-of-two row / token scales ride in as E8M0 factors)
// both into ONE fp32 TMEM accumulator (dense / n:8 inliers: 4 x dense tcgen05.mma kind::mxf4 of 64 K per 256 K instead;
// one scale per 32 K: kind::mxf4nvf4 .block16).  Persistent CTAs walk tiles of 128 rows x up to 256 tokens.
// Warp roles: warps 0, 6, 7 = bulk-copy (TMA) producers for weights, activations and scale atoms (issuing a
// bulk copy costs one thread ~50 ns, so the copies of a stage are spread over three threads), warp 1 = TMEM
// owner + MMA issuer, warps 2..5 = epilogue (tcgen05.ld, convert, shared-memory transpose, 16-byte row stores),
// warp 8 = mover of metadata and scale atoms smem -> TMEM (tcgen05.cp) in the many-token instantiations; with
// runtime geometry the MMA issuer does those copies itself.  The many-token instantiations run four more warps
// (9..12), a second epilogue group: the eight epilogue warps load the accumulator into registers, hand TMEM back
// and store under the next tile's K loop.
// For few tokens the K range of a row tile is split over several CTAs: either a thread-block cluster whose members
// keep their fp32 partial tiles in shared memory and each add one slice of rows over all members in rank order
// (no global scratch), or, with a caller-provided workspace, partial tiles in global memory that the last CTA to
// arrive adds in split order.  Both orders are fixed.  Launches carry programmatic stream serialization: the
// kernel lets its successor be scheduled at once and itself waits for its predecessor only before it reads
// activations or writes Y.  Every wait is bounded; a timeout sets a sticky flag.
#include <cuda_bf16.h>
#include <stdlib.h>

#include "sdq_internal.h"
#include "sdq_layout.h"
#include "sdq_linear.h"
#include "sdq_plain.h"
#include "sdq_ptx.cuh"

namespace sdq {

constexpr int LIN_THREADS_MANY = 416;   // many-token instantiations: warps 9..12 = a second epilogue group (tokens 128..255 of the tile)
constexpr int LIN_THREADS = 288;   // warps: 0 weight producer, 1 MMA issuer, 2..5 epilogue, 6 activation producer, 7 scale-atom producer,
                                   // 8 metadata / scale mover (many-token instantiation only)
constexpr int MAX_SLOTS = 16;
constexpr int SL_A = 0;                        // WI record (A_in | E_in | SFA_in) or WO record (A_out | E_out)
constexpr int RING_BYTES = 225280;             // largest ring: nslot slots of slot_bytes each
constexpr int SM_TAIL = 4096 + 640 + 128;      // epilogue transpose buffer (16 tokens x 128 features bf16) + barriers + slack
constexpr int SM_TAIL_B32 = 640 + 128;         // many tokens, one scale per 32 K: five 46080-byte slots leave no room for the
                                               // transpose buffer; that instantiation stores from registers
constexpr int LIN_SMEM_MAX = 5 * 46080 + SM_TAIL_B32;   // the largest request

// TMEM columns: accumulator at 0 (n_tile columns, tokens), then metadata / scales.
// Runtime geometry: 84 columns at `meta_col`:
//   +0  2 buffers x 32: E_in 4 | SFA_in 4 or 8 | SFB_in up to 16     +64 2 buffers x 4: E_out     +72 SFA_out 4     +76 SFB_out 8
//   (one scale per 64 K: SFA_in 4, SFB_in 4 per token tile; per 32 K: one scale word per 128-K block, so twice as many)
// Many tokens (512 columns): 16 columns per ring slot at 256 + 16 s (E 4 | SFA 4 | SFB 8; an outlier stage uses the
// first 4; 32 per slot with one scale per 32 K: E 4 | SFA 8 | SFB 16) and, behind the slots' columns, two alternating
// 12-column buffers of outlier row / token scales.
constexpr uint32_t TM_D = 0;
constexpr uint32_t TM_META_COLS = 84;

// slot = | A record 10752 | B n_tile*128 | scale atoms 1536 |  (inlier: SFB_in x n_atiles; first outlier stage:
// SFA_out | SFB_out x n_atiles)
// (one scale per 32 K: the weight record is 512 B longer and an inlier stage carries two scale atoms per token tile)
// (dense inliers: the weight record holds twice the codes and no pattern metadata)
__host__ __device__ inline int slot_bytes_for(int n_tile, bool b32 = false, bool dense = false) {
  const int n_atiles = (n_tile + TILE_TOK - 1) / TILE_TOK, atoms = b32 ? (2 * n_atiles > 1 + n_atiles ? 2 * n_atiles : 1 + n_atiles) : 3;
  return wi_bytes(b32, dense) + n_tile * 128 + atoms * SF_ATOM_BYTES;
}

// 2^ex as a float (ex limited to the normal range), for the exact rescaling of two-level-scaled accumulators
__device__ __forceinline__ float pow2i(int ex) { return __int_as_float((min(max(ex, -126), 127) + 127) << 23); }

struct TileCoord {
  int rt, mtile, split;
  int i0, i1, o0, o1;   // inlier stages [i0, i1) of T2, outlier stages [o0, o1) of T1
};
__device__ __forceinline__ TileCoord tile_coord(int ksplit, int tile, int RT, int T1, int T2) {
  TileCoord c;
  if (ksplit == 1) {
    c.split = 0; c.rt = tile % RT; c.mtile = tile / RT;
    c.i0 = 0; c.i1 = T2; c.o0 = 0; c.o1 = T1;
    return c;
  }
  c.split = tile % ksplit;
  const int rest = tile / ksplit;
  c.rt = rest % RT;
  c.mtile = rest / RT;
  c.i0 = c.split * T2 / ksplit;           // 32-bit: split < 32, T1 <= K/128
  c.i1 = (c.split + 1) * T2 / ksplit;
  c.o0 = c.split * T1 / ksplit;
  c.o1 = (c.split + 1) * T1 / ksplit;
  return c;
}

// FLEX = false: the many-token instantiation (n_tile = 256, 5 ring slots, 512 TMEM columns, no K split) with every
// geometry constant known at compile time -- the single-thread issue loops are latency-bound, so each runtime
// parameter they touch costs time.  FLEX = true: geometry from the launch parameters (few tokens, split K).
// B32 (many-token instantiation only): one scale per 32 K, four ring slots of 45 KB.
// DENSE (many-token instantiation only): dense inliers with one scale per 32 K, four ring slots of 51 KB.
template <bool F32_OUT, bool FLEX, bool B32, bool DENSE>
__global__ void __maxnreg__(FLEX ? 96 : 128)   // runtime geometry: two 9-warp CTAs share an SM only below ~100 registers per thread;
sdq_linear_kernel(const LinearParams p)       // many tokens: 13 warps, four of them on one sub-partition of 16 K registers
{
  extern __shared__ uint8_t smem_raw[];
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint8_t* sm = smem_raw + ((128 - (ptx::smem_u32(smem_raw) & 127)) & 127);
  const int ksplit = FLEX ? p.ksplit : 1, cluster_ks = FLEX ? p.cluster_ks : 1;
  const bool release = FLEX ? (p.release != 0) : true;
  // the transpose buffer and the barriers follow the ring (many tokens: 5 x 45056, or 4 x 46080 with one scale per 32 K)
  static_assert(!(FLEX && (B32 || DENSE)) && !(B32 && DENSE), "B32 and DENSE name many-token instantiations");
  constexpr bool S32 = B32 || DENSE;                       // many tokens with one scale per 32 K
  constexpr uint32_t SLOT_FIXED = DENSE ? 52224u : (B32 ? 46080u : 45056u), NSLOT_FIXED = DENSE ? 4u : 5u;
  // the transpose buffer and then the barriers follow the ring (B32: no transpose buffer)
  const uint32_t SM_STG = FLEX ? (uint32_t)p.ring_bytes : NSLOT_FIXED * SLOT_FIXED, SM_BARS = B32 ? SM_STG : SM_STG + 4096;
  const uint32_t TM_I = FLEX ? (uint32_t)p.meta_col : 256u, TM_EO = TM_I + 64, TM_SFA_OUT = TM_I + 72, TM_SFB_OUT = TM_I + 76;
  const uint32_t tmem_cols = FLEX ? (uint32_t)p.tmem_cols : 512u;
  uint64_t* full = reinterpret_cast<uint64_t*>(sm + SM_BARS);
  uint64_t* empty = full + MAX_SLOTS;
  uint64_t* meta_full = empty + MAX_SLOTS;          // FLEX = false: metadata / scales of slot s are in TMEM
  uint64_t* full_w = meta_full + MAX_SLOTS;         // FLEX = false: weight record and scale atoms of slot s have landed
  uint64_t* acc_full = full_w + MAX_SLOTS;
  uint64_t* acc_empty = acc_full + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 1);
  uint32_t* last_flag = tmem_slot + 1;

  const int n_tile = FLEX ? p.n_tile : 256;
  const int RT = (int)(p.N / TILE_ROWS);
  const int T1 = p.out_n ? (int)(p.K / K1) : 0, T2 = (int)(p.K / K2);
  const int n_atiles = (n_tile + TILE_TOK - 1) / TILE_TOK;     // 128-token activation tiles per token tile
  const uint32_t nslot = FLEX ? (uint32_t)p.nslot : NSLOT_FIXED, slot_bytes = FLEX ? (uint32_t)p.slot_bytes : SLOT_FIXED;
  const bool b32 = FLEX ? (p.b32 != 0) : S32;              // one scale per 32 K
  const bool dense = FLEX ? (p.dense != 0) : DENSE;        // dense inliers (always with one scale per 32 K)
  constexpr uint32_t MS = S32 ? 32u : 16u;                 // many tokens: metadata / scale columns per ring slot
  const uint32_t wib = (uint32_t)wi_bytes(b32, dense), xib = (uint32_t)xi_bytes(b32), na = b32 ? 2u : 1u;
  const uint32_t sl_b = wib;                               // B4 / B8 follow the (longest) weight record
  const uint32_t sl_sf = sl_b + (uint32_t)n_tile * 128u;

  // the coordinates of the first tile are worked out by every thread while the barriers and TMEM are being set up
  // (a lone thread needs ~0.5 us for the integer divisions, which would otherwise delay the first copies)
  const TileCoord first_tc = tile_coord(ksplit, (int)blockIdx.x, RT, T1, T2);
  if (tid == 0) ptx::griddep_launch_dependents();   // the next launch may be scheduled as soon as every CTA got here
  if (tid == 0) {
    // FLEX = false: the weight and scale-atom producers arrive on full_w[s] (the mover starts from it while the
    // larger activation copies are still landing), the activation producer on full[s]
    for (uint32_t s = 0; s < nslot; ++s) {
      ptx::mbar_init(&full[s], FLEX ? 3 : 1);
      ptx::mbar_init(&empty[s], 1);
      ptx::mbar_init(&meta_full[s], 1);
      ptx::mbar_init(&full_w[s], 2);
    }
    ptx::mbar_init(acc_full, 1);
    ptx::mbar_init(acc_empty, FLEX ? 4 : 8);
    ptx::fence_barrier_init();
  }
  if (warp == 1) ptx::tmem_alloc(tmem_slot, tmem_cols);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0 || warp == 6 || warp == 7) {
    if (lane == 0) {
      // ---------------- producers: role 0 = weight records, role 1 = activation codes, role 2 = scale atoms.
      // Each arrives once per stage on full[s] with the bytes it is about to copy.
      const int role = warp == 0 ? 0 : (int)warp - 5;
      if (role != 0) ptx::griddep_wait();    // activations and their scales come from an earlier kernel; weights do not
      bool ok = true;
      uint32_t s = 0, wrapped = 0, ph = 0;   // ring slot, whether the ring has wrapped, phase parity of `empty`
      for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x) {
        const TileCoord tc = (tile == (int)blockIdx.x) ? first_tc : tile_coord(ksplit, tile, RT, T1, T2);
        const int mt = tc.mtile * n_tile / TILE_TOK;
        const int have = min(n_atiles, (int)p.aoff.MT - mt);                 // activation tiles that exist
        const uint32_t tok_bytes = (uint32_t)min(n_tile, TILE_TOK) * 128u;   // bytes per activation tile per stage
        const uint8_t* wi = p.w + p.poff.wi + ((size_t)tc.rt * T2 + tc.i0) * wib;
        const uint8_t* wo = p.w + p.poff.wo + ((size_t)tc.rt * T1 + tc.o0) * WO_BYTES;
        const uint8_t* xi = p.x + p.aoff.xi + ((size_t)mt * T2 + tc.i0) * xib;
        const uint8_t* xo = p.x + p.aoff.xo + ((size_t)mt * T1 + tc.o0) * XO_BYTES;
        const size_t xi_tile = (size_t)T2 * xib, xo_tile = (size_t)T1 * XO_BYTES;
        const int ni = tc.i1 - tc.i0, no = tc.o1 - tc.o0;
        for (int k = 0; k < ni + no; ++k) {
          if (wrapped && release && !(ok = ptx::mbar_wait(&empty[s], ph ^ 1))) break;
          uint8_t* st = sm + (size_t)s * slot_bytes;
          const bool first_o = (k == ni);
          uint64_t* bw = FLEX ? &full[s] : &full_w[s];
          if (role == 0) {
            if (k < ni) {
              ptx::mbar_expect_tx(bw, wib);
              ptx::bulk_g2s(st + SL_A, wi, wib, bw);
              wi += wib;
            } else {
              ptx::mbar_expect_tx(bw, WO_BYTES + (first_o ? SF_ATOM_BYTES : 0u));
              ptx::bulk_g2s(st + SL_A, wo, WO_BYTES, bw);
              if (first_o) ptx::bulk_g2s(st + sl_sf, p.w + p.poff.sfa_out + (size_t)tc.rt * SF_ATOM_BYTES, SF_ATOM_BYTES, bw);
              wo += WO_BYTES;
            }
          } else if (role == 1) {
            ptx::mbar_expect_tx(&full[s], (uint32_t)have * tok_bytes);
            if (k < ni) {
              for (int a = 0; a < have; ++a) ptx::bulk_g2s(st + sl_b + a * B4_BYTES, xi + a * xi_tile, tok_bytes, &full[s]);
              xi += xib;
            } else {
              for (int a = 0; a < have; ++a) ptx::bulk_g2s(st + sl_b + a * B8_BYTES, xo + a * xo_tile, tok_bytes, &full[s]);
              xo += XO_BYTES;
            }
          } else {
            if (k < ni) {
              ptx::mbar_expect_tx(bw, (uint32_t)have * na * SF_ATOM_BYTES);
              for (int a = 0; a < have; ++a)
                ptx::bulk_g2s(st + sl_sf + a * na * SF_ATOM_BYTES, xi + a * xi_tile + B4_BYTES, na * SF_ATOM_BYTES, bw);
              xi += xib;
            } else if (first_o) {
              ptx::mbar_expect_tx(bw, (uint32_t)have * SF_ATOM_BYTES);
              for (int a = 0; a < have; ++a)
                ptx::bulk_g2s(st + sl_sf + (1 + a) * SF_ATOM_BYTES, p.x + p.aoff.sfb_out + (size_t)(mt + a) * SF_ATOM_BYTES, SF_ATOM_BYTES,
                              bw);
            } else {
              ptx::mbar_arrive(bw);
            }
          }
          if (++s == nslot) { s = 0; wrapped = 1; ph ^= 1; }
        }
      }
      if (!ok) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------- MMA issuer
      bool ok = true;
      const uint32_t smb = ptx::smem_u32(sm);
      uint32_t s = 0, ph = 0, tcount = 0;
      bool ready = false;
      // (two-level scaling: the .block16 kind reads its scale codes as unsigned E4M3 when bit 23 is clear)
      const uint32_t id4[2] = {ptx::idesc_block_scaled(128, (uint32_t)n_tile, 1, true, 0, 0) ^ (p.tw ? (1u << 23) : 0u),
                               ptx::idesc_block_scaled(128, (uint32_t)n_tile, 1, true, 2, 2)};
      const uint32_t id8 = ptx::idesc_block_scaled(128, (uint32_t)n_tile, 0, true, 0, 0);
      const uint32_t idd[2] = {ptx::idesc_block_scaled(128, (uint32_t)n_tile, 1, false, 0, 0),      // dense inliers
                               ptx::idesc_block_scaled(128, (uint32_t)n_tile, 1, false, 2, 2)};
      // descriptors of slot 0; slot s adds s * slot_bytes / 16 to the start-address field
      const uint64_t d_a = ptx::smem_desc(smb + SL_A, 128, 256), d_b = ptx::smem_desc(smb + sl_b, 128, 1024);
      const uint64_t d_e_in = ptx::smem_desc(smb + SL_A + A_IN_BYTES, 0, 128);
      const uint64_t d_sfa_in = ptx::smem_desc(smb + SL_A + (uint32_t)(a_in_bytes(dense) + e_in_bytes(dense)), 0, 128);
      const uint64_t d_e_out = ptx::smem_desc(smb + SL_A + A_OUT_BYTES, 0, 128);
      const uint64_t d_sf0 = ptx::smem_desc(smb + sl_sf, 0, 128), d_sf1 = ptx::smem_desc(smb + sl_sf + SF_ATOM_BYTES, 0, 128);
      const uint64_t d_sf2 = ptx::smem_desc(smb + sl_sf + 2 * SF_ATOM_BYTES, 0, 128);
      const uint32_t slot16 = slot_bytes >> 4;
      for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x, ++tcount) {
        const TileCoord tc = (tcount == 0) ? first_tc : tile_coord(ksplit, tile, RT, T1, T2);
        const int ni = tc.i1 - tc.i0, no = tc.o1 - tc.o0;
        if (tcount > 0) {   // the epilogue must have drained the accumulator of the previous tile
          ok = ptx::mbar_wait(acc_empty, (tcount - 1) & 1);
          if (!ok) break;
          ptx::tc_fence_after();
        }
        uint32_t acc = 0;   // the first MMA of the tile overwrites the accumulator
        if constexpr (!FLEX) {
          // many tokens: warp 8 has already moved the metadata and scales of slot s to TMEM (16 columns per slot, the
          // outlier scales in one of two per-tile buffers); this thread only issues the MMAs
          const uint32_t sfo = tmem + 256u + MS * nslot + 12u * (tcount & 1);
          for (int k = 0; k < ni + no; ++k) {
            if (!ready) ok = ptx::mbar_wait(&meta_full[s], ph);
            if (ok) ok = ptx::mbar_wait(&full[s], ph);          // the activation codes of the slot
            if (!ok) break;
            ptx::tc_fence_after();
            const uint32_t sn = (s + 1 == nslot) ? 0 : s + 1;
            ready = ptx::mbar_test(&meta_full[sn], sn ? ph : ph ^ 1);
            const uint64_t so = (uint64_t)(s * slot16);
            const uint32_t mb = tmem + 256u + MS * s;
            if (k < ni) {
              if constexpr (DENSE) {
#pragma unroll
                for (uint32_t j = 0; j < 4; ++j)
                  ptx::mma_mxf4(tmem + TM_D, d_a + so + ((4096 * j) >> 4), d_b + so + ((256 * j) >> 4), idd[j & 1], mb + 4 + 4 * (j >> 1),
                                mb + 12 + 8 * (j >> 1), j ? 1u : acc);
              } else if constexpr (B32) {
                ptx::mma_sp_nvf4(tmem + TM_D, d_a + so, d_b + so, id4[0], mb, mb + 4, mb + 12, acc);
                ptx::mma_sp_nvf4(tmem + TM_D, d_a + so + (4096 >> 4), d_b + so + (512 >> 4), id4[0], mb + 2, mb + 8, mb + 20, 1u);
              } else {
                ptx::mma_sp_mxf4(tmem + TM_D, d_a + so, d_b + so, id4[0], mb, mb + 4, mb + 8, acc);
                ptx::mma_sp_mxf4(tmem + TM_D, d_a + so + (4096 >> 4), d_b + so + (512 >> 4), id4[1], mb + 2, mb + 4, mb + 8, 1u);
              }
            } else {
              ptx::mma_sp_mxf8(tmem + TM_D, d_a + so, d_b + so, id8, mb, sfo, sfo + 4, acc);
              ptx::mma_sp_mxf8(tmem + TM_D, d_a + so + (4096 >> 4), d_b + so + (512 >> 4), id8, mb + 2, sfo, sfo + 4, 1u);
            }
            acc = 1;
            ptx::tc_commit(&empty[s]);
            s = sn;
            if (sn == 0) ph ^= 1;
          }
          ptx::tc_commit(acc_full);
        } else {
        for (int k = 0; k < ni + no; ++k) {
          if (!ready) ok = ptx::mbar_wait(&full[s], ph);
          if (!ok) break;
          ptx::tc_fence_after();
          const uint32_t sn = (s + 1 == nslot) ? 0 : s + 1;
          // poll the next slot now: the answer is back by the time this stage's instructions are issued
          ready = ptx::mbar_test(&full[sn], sn ? ph : ph ^ 1);
          const uint64_t so = (uint64_t)(s * slot16);
          if (k < ni) {
            // inlier stage: 256 logical K = 2 sparse MXFP4 MMAs; metadata and scale atoms go to TMEM first
            const uint32_t mb = tmem + TM_I + 32u * (uint32_t)(k & 1);
            if (!dense) ptx::tc_cp_128x128b(mb + 0, d_e_in + so);
            ptx::tc_cp_32x128b_warpx4(mb + 4, d_sfa_in + so);
            if (!b32) {
              ptx::tc_cp_32x128b_warpx4(mb + 8, d_sf0 + so);
              if (n_atiles > 1) ptx::tc_cp_32x128b_warpx4(mb + 12, d_sf1 + so);
              ptx::mma_sp_mxf4(tmem + TM_D, d_a + so, d_b + so, id4[0], mb, mb + 4, mb + 8, acc);
              ptx::mma_sp_mxf4(tmem + TM_D, d_a + so + (4096 >> 4), d_b + so + (512 >> 4), id4[1], mb + 2, mb + 4, mb + 8, 1u);
            } else {
              // one scale per 32 K: scale word of K-block kb for the weights at mb + 4 + 4 kb, for the tokens at
              // mb + 12 + 4 n_atiles kb (+ 4 per token tile); the staged atoms are ordered [token tile][K-block]
              ptx::tc_cp_32x128b_warpx4(mb + 8, d_sfa_in + so + (SF_ATOM_BYTES >> 4));
              for (uint32_t a = 0; a < (uint32_t)n_atiles; ++a)
                for (uint32_t kb = 0; kb < 2; ++kb)
                  ptx::tc_cp_32x128b_warpx4(mb + 12 + 4 * (kb * (uint32_t)n_atiles + a), d_sf0 + so + (((2 * a + kb) * SF_ATOM_BYTES) >> 4));
              if (!dense) {
                ptx::mma_sp_nvf4(tmem + TM_D, d_a + so, d_b + so, id4[0], mb, mb + 4, mb + 12, acc);
                ptx::mma_sp_nvf4(tmem + TM_D, d_a + so + (4096 >> 4), d_b + so + (512 >> 4), id4[0], mb + 2, mb + 8,
                                 mb + 12 + 4 * (uint32_t)n_atiles, 1u);
              } else {
                // dense inliers: four MMAs of 64 K; MMA j reads K-block j of the weights (4096 B apart), bytes 32 j .. 32 j + 31
                // of every token (two 16-byte chunks, 256 B apart per j) and scales 2 (j & 1), 2 (j & 1) + 1 of the scale
                // word of 128-K block j / 2
#pragma unroll
                for (uint32_t j = 0; j < 4; ++j)
                  ptx::mma_mxf4(tmem + TM_D, d_a + so + ((4096 * j) >> 4), d_b + so + ((256 * j) >> 4), idd[j & 1], mb + 4 + 4 * (j >> 1),
                                mb + 12 + 4 * (uint32_t)n_atiles * (j >> 1), j ? 1u : acc);
              }
            }
          } else {
            // outlier stage: 128 logical K = 2 sparse FP8 MMAs; the row / token scales (E8M0) arrive with the first one
            const uint32_t eb = tmem + TM_EO + 4u * (uint32_t)(k & 1);
            ptx::tc_cp_128x128b(eb, d_e_out + so);
            if (k == ni) {
              ptx::tc_cp_32x128b_warpx4(tmem + TM_SFA_OUT, d_sf0 + so);
              ptx::tc_cp_32x128b_warpx4(tmem + TM_SFB_OUT, d_sf1 + so);
              if (n_atiles > 1) ptx::tc_cp_32x128b_warpx4(tmem + TM_SFB_OUT + 4, d_sf2 + so);
            }
            ptx::mma_sp_mxf8(tmem + TM_D, d_a + so, d_b + so, id8, eb, tmem + TM_SFA_OUT, tmem + TM_SFB_OUT, acc);
            ptx::mma_sp_mxf8(tmem + TM_D, d_a + so + (4096 >> 4), d_b + so + (512 >> 4), id8, eb + 2, tmem + TM_SFA_OUT,
                             tmem + TM_SFB_OUT, 1u);
          }
          acc = 1;
          if (release) ptx::tc_commit(&empty[s]);   // ring slots are reused only when a CTA runs more stages than slots
          s = sn;
          if (sn == 0) ph ^= 1;
        }
        ptx::tc_commit(acc_full);
        }
      }
      if (!ok) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
    }
  } else if (warp == 8) {
    if (!FLEX && lane == 0) {
      // ---------------- metadata / scale mover: smem -> TMEM (tcgen05.cp) for every slot as soon as it has landed, so
      // that the MMA issuer's instruction stream holds nothing but MMAs.  TMEM buffer s belongs to ring slot s: it is
      // free again exactly when the slot is (the producers refill a slot only after its MMAs have completed).
      bool ok = true;
      const uint32_t smb = ptx::smem_u32(sm);
      uint32_t s = 0, ph = 0, tcount = 0;
      const uint64_t d_e_in = ptx::smem_desc(smb + SL_A + A_IN_BYTES, 0, 128);
      const uint64_t d_sfa_in = ptx::smem_desc(smb + SL_A + (DENSE ? 2 * A_IN_BYTES : A_IN_BYTES + E_IN_BYTES), 0, 128);
      const uint64_t d_e_out = ptx::smem_desc(smb + SL_A + A_OUT_BYTES, 0, 128);
      const uint64_t d_sf0 = ptx::smem_desc(smb + sl_sf, 0, 128), d_sf1 = ptx::smem_desc(smb + sl_sf + SF_ATOM_BYTES, 0, 128);
      const uint64_t d_sf2 = ptx::smem_desc(smb + sl_sf + 2 * SF_ATOM_BYTES, 0, 128);
      const uint32_t slot16 = slot_bytes >> 4;
      for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x, ++tcount) {
        const uint32_t sfo = tmem + 256u + MS * nslot + 12u * (tcount & 1);
        for (int k = 0; k < T2 + T1; ++k) {
          if (!(ok = ptx::mbar_wait(&full_w[s], ph))) break;
          ptx::tc_fence_after();
          const uint64_t so = (uint64_t)(s * slot16);
          const uint32_t mb = tmem + 256u + MS * s;
          if (k < T2) {
            if constexpr (!DENSE) ptx::tc_cp_128x128b(mb + 0, d_e_in + so);
            ptx::tc_cp_32x128b_warpx4(mb + 4, d_sfa_in + so);
            if constexpr (S32) {
              // scale words: weights K-block 0 / 1 at +4 / +8; tokens K-block kb, token tile a at +12 + 4 (2 kb + a), staged
              // as [token tile][K-block]
              ptx::tc_cp_32x128b_warpx4(mb + 8, d_sfa_in + so + (SF_ATOM_BYTES >> 4));
              ptx::tc_cp_32x128b_warpx4(mb + 12, d_sf0 + so);
              ptx::tc_cp_32x128b_warpx4(mb + 20, d_sf1 + so);
              ptx::tc_cp_32x128b_warpx4(mb + 16, d_sf2 + so);
              ptx::tc_cp_32x128b_warpx4(mb + 24, d_sf2 + so + (SF_ATOM_BYTES >> 4));
            } else {
              ptx::tc_cp_32x128b_warpx4(mb + 8, d_sf0 + so);
              ptx::tc_cp_32x128b_warpx4(mb + 12, d_sf1 + so);
            }
          } else {
            ptx::tc_cp_128x128b(mb + 0, d_e_out + so);
            if (k == T2) {
              ptx::tc_cp_32x128b_warpx4(sfo, d_sf0 + so);
              ptx::tc_cp_32x128b_warpx4(sfo + 4, d_sf1 + so);
              ptx::tc_cp_32x128b_warpx4(sfo + 8, d_sf2 + so);
            }
          }
          ptx::tc_commit(&meta_full[s]);
          if (++s == nslot) { s = 0; ph ^= 1; }
        }
      }
      if (!ok) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
    }
  } else if ((warp >= 2 && warp <= 5) || warp >= 9) {
    // ---------------- epilogue: warp w owns TMEM lanes 32*(w%4) .. +31 (weight rows), columns = tokens; many tokens: a
    // second group of four warps (9..12) takes tokens 128..255 of the tile
    const uint32_t q = warp & 3;
    const uint32_t grp = warp >= 9 ? 1u : 0u;
    const uint32_t et = (warp - (grp ? 9u : 2u)) * 32 + lane;     // 0..127 among the epilogue threads of the group
    uint32_t tcount = 0;
    bool ok = true;
    ptx::griddep_wait();                            // Y and the workspace may still be in use by the previous kernel
    for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x, ++tcount) {
      const TileCoord tc = (tcount == 0) ? first_tc : tile_coord(ksplit, tile, RT, T1, T2);
      const int64_t m0 = (int64_t)tc.mtile * n_tile;
      const int n_valid = (int)min((int64_t)n_tile, p.M - m0);
      ok = ptx::mbar_wait(acc_full, tcount & 1);
      ptx::tc_fence_after();
      if (!ok) break;
      const int64_t n0 = (int64_t)tc.rt * TILE_ROWS;
      const int twr = p.tw ? __ldg(p.tw + n0 + q * 32 + lane) : 0;     // two-level scaling: this thread's row factor
      auto rescale = [&](uint32_t (&v)[16], int c0) {                  // columns c0 .. c0 + 15 of the tile, by 2^(tw + tx)
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (c0 + j < n_valid) v[j] = __float_as_uint(__uint_as_float(v[j]) * pow2i(twr + __ldg(p.tx + m0 + c0 + j)));
      };
      // split-K: this CTA's fp32 partial tile [token][128 rows] in the workspace
      float* part = nullptr;
      if (cluster_ks > 1) part = reinterpret_cast<float*>(sm);   // the ring is idle once the accumulator is complete
      else if (ksplit > 1)
        part = p.ws_partial + ((size_t)(tc.rt * p.n_mtiles + tc.mtile) * ksplit + tc.split) * (size_t)n_tile * TILE_ROWS;
      if constexpr (!FLEX && F32_OUT) {
        if (grp) {                                  // fp32 output (tests): the first group stores everything
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(acc_empty);
          continue;
        }
      }
      if constexpr (!FLEX && !F32_OUT) {
        // many tokens, bf16 output: the accumulator cannot be double-buffered (TMEM is full), so the epilogue first
        // drains it into registers -- one weight row x 128 tokens per thread as 64 packed bf16 pairs -- hands TMEM back,
        // and only then transposes and stores: the stores run under the next tile's K loop
        uint32_t pk[64];
        {
          uint32_t va[16], vb[16];
          const uint32_t tbase = tmem + ((q * 32u) << 16) + TM_D + 128u * grp;
          ptx::tmem_ld_32x32b_x16(tbase, va);
#pragma unroll
          for (int c = 0; c < 128; c += 32) {
            ptx::tmem_ld_wait();
            ptx::tmem_ld_32x32b_x16(tbase + (uint32_t)(c + 16), vb);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(va[2 * j]), __uint_as_float(va[2 * j + 1]));
              pk[c / 2 + j] = *reinterpret_cast<const uint32_t*>(&h);
            }
            ptx::tmem_ld_wait();
            if (c + 32 < 128) ptx::tmem_ld_32x32b_x16(tbase + (uint32_t)(c + 32), va);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(vb[2 * j]), __uint_as_float(vb[2 * j + 1]));
              pk[c / 2 + 8 + j] = *reinterpret_cast<const uint32_t*>(&h);
            }
          }
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(acc_empty);
        const int g0 = 128 * (int)grp;
        if constexpr (B32) {
          // no room for a transpose buffer beside five slots: every thread stores its row's 128 tokens itself (for one
          // token the 32 lanes of a warp write 64 contiguous bytes); measured 2-4 % slower than the transposed stores
          // below, which the fifth slot more than pays for
          uint16_t* Y = reinterpret_cast<uint16_t*>(p.Y) + n0 + q * 32 + lane;
#pragma unroll
          for (int j = 0; j < 64; ++j) {
            const int t = g0 + 2 * j;
            if (t >= n_valid) break;                  // uniform over the warp
            uint32_t lo = pk[j] << 16, hi = pk[j] & 0xFFFF0000u;
            if (p.tw) {
              // two-level scaling: multiplying the rounded value by the power of two is the rounding of the multiplied
              // value, so the factors go in here, after TMEM has been handed back
              lo = __float_as_uint(__uint_as_float(lo) * pow2i(twr + __ldg(p.tx + m0 + t)));
              if (t + 1 < n_valid) hi = __float_as_uint(__uint_as_float(hi) * pow2i(twr + __ldg(p.tx + m0 + t + 1)));
            }
            Y[(m0 + t) * p.ldy] = (uint16_t)(lo >> 16);
            if (t + 1 < n_valid) Y[(m0 + t + 1) * p.ldy] = (uint16_t)(hi >> 16);
          }
        } else {
          // transpose through shared memory, 8 tokens at a time per group: [8 tokens][128 features] bf16, then one
          // 16-byte store per thread (full 256 B rows)
          uint16_t* stg = reinterpret_cast<uint16_t*>(sm + SM_STG) + grp * 1024u;
          __nv_bfloat16* Y = reinterpret_cast<__nv_bfloat16*>(p.Y);
#pragma unroll
          for (int c0 = 0; c0 < 128; c0 += 8) {
            if (g0 + c0 < n_valid) {                  // uniform over the four warps of the group
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                stg[(2 * j) * 128 + q * 32 + lane] = (uint16_t)(pk[c0 / 2 + j] & 0xFFFFu);
                stg[(2 * j + 1) * 128 + q * 32 + lane] = (uint16_t)(pk[c0 / 2 + j] >> 16);
              }
              ptx::named_bar_sync(1 + grp, 128);
              const uint32_t tok = et >> 4, seg = et & 15;
              if (g0 + c0 + (int)tok < n_valid) {
                const uint4 w = *reinterpret_cast<const uint4*>(stg + tok * 128 + seg * 8);
                *reinterpret_cast<uint4*>(Y + (m0 + g0 + c0 + tok) * p.ldy + n0 + seg * 8) = w;
              }
              ptx::named_bar_sync(1 + grp, 128);       // the buffer is rewritten by the next chunk
            }
          }
        }
        continue;
      }
      if (part) {
        // split K: all n_tile token columns of the partial tile go out (the reduction reads only the valid ones); the
        // TMEM load of the next 16 columns is in flight while the current 16 are stored
        uint32_t va[16], vb[16];
        const uint32_t tbase = tmem + ((q * 32u) << 16) + TM_D;
        float* dst = part + q * 32 + lane;
        ptx::tmem_ld_32x32b_x16(tbase, va);
#pragma unroll 1
        for (int c0 = 0; c0 < n_tile; c0 += 32) {
          ptx::tmem_ld_wait();
          if (c0 + 16 < n_tile) ptx::tmem_ld_32x32b_x16(tbase + (uint32_t)(c0 + 16), vb);
#pragma unroll
          for (int j = 0; j < 16; ++j) dst[(size_t)(c0 + j) * TILE_ROWS] = __uint_as_float(va[j]);
          if (c0 + 16 < n_tile) {
            ptx::tmem_ld_wait();
            if (c0 + 32 < n_tile) ptx::tmem_ld_32x32b_x16(tbase + (uint32_t)(c0 + 32), va);
#pragma unroll
            for (int j = 0; j < 16; ++j) dst[(size_t)(c0 + 16 + j) * TILE_ROWS] = __uint_as_float(vb[j]);
          }
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(acc_empty);   // accumulator fully read
      }
#pragma unroll 1
      for (int c0 = 0; c0 < (part ? 0 : n_tile); c0 += 16) {
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
        if (p.tw) rescale(v, c0);
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
      if (part && cluster_ks <= 1) {
        // the last CTA of this (row tile, token tile) to finish adds the partial tiles in split order
        __threadfence();
        ptx::named_bar_sync(1, 128);
        uint32_t* counter = p.ws_counter + tc.rt * p.n_mtiles + tc.mtile;
        if (et == 0) {
          const uint32_t old = atomicAdd(counter, 1u);
          *last_flag = (old == (uint32_t)ksplit - 1) ? 1u : 0u;
        }
        ptx::named_bar_sync(1, 128);
        if (*last_flag) {
          __threadfence();
          const float* base = p.ws_partial + (size_t)(tc.rt * p.n_mtiles + tc.mtile) * ksplit * (size_t)n_tile * TILE_ROWS;
          // 8 tokens at a time: the loads of one split are independent, only the adds follow split order
          for (int t0 = 0; t0 < n_valid; t0 += 8) {
            float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 2
            for (int sp = 0; sp < ksplit; ++sp) {
              const float* src = base + ((size_t)sp * n_tile + t0) * TILE_ROWS + et;
              float v[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) v[j] = (t0 + j < n_valid) ? __ldcg(src + (size_t)j * TILE_ROWS) : 0.0f;
#pragma unroll
              for (int j = 0; j < 8; ++j) acc[j] += v[j];
            }
            if (p.tw) {
              const int twe = __ldg(p.tw + n0 + et);
#pragma unroll
              for (int j = 0; j < 8; ++j)
                if (t0 + j < n_valid) acc[j] *= pow2i(twe + __ldg(p.tx + m0 + t0 + j));
            }
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (t0 + j < n_valid) {
                if (F32_OUT) reinterpret_cast<float*>(p.Y)[(m0 + t0 + j) * p.ldy + n0 + et] = acc[j];
                else reinterpret_cast<__nv_bfloat16*>(p.Y)[(m0 + t0 + j) * p.ldy + n0 + et] = __float2bfloat16_rn(acc[j]);
              }
          }
          if (et == 0) *counter = 0u;     // ready for the next call
        }
        ptx::named_bar_sync(1, 128);       // last_flag is rewritten by the next tile
      }
    }
    if (!ok && lane == 0) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
  }
  if (cluster_ks > 1) {
    // ---------------- cluster split-K: one tile per CTA; CTA r adds its share of the tile's rows over all members
    ptx::cluster_sync();                         // every member's partial tile is in its shared memory
    if (warp >= 2 && warp <= 5) {
      const uint32_t et = (warp - 2) * 32 + lane;
      const uint32_t ks = (uint32_t)cluster_ks, rank = ptx::cluster_ctarank();
      const int n_valid = (int)min((int64_t)n_tile, p.M - (int64_t)first_tc.mtile * n_tile);
      const int64_t m0 = (int64_t)first_tc.mtile * n_tile, n0 = (int64_t)first_tc.rt * TILE_ROWS;
      const uint32_t local = ptx::smem_u32(sm);
      // four rows x one token per item: one 16-byte load per member, added in rank order.  The 32 quads of rows are
      // dealt out evenly over the members (ks need not divide 32: 3 members take 10, 11 and 11 quads)
      uint32_t peer[8];
#pragma unroll
      for (uint32_t sp = 0; sp < 8; ++sp) peer[sp] = ptx::mapa_u32(local, sp < ks ? sp : 0u);
      const uint32_t q_begin = rank * 32u / ks, q_per = (rank + 1) * 32u / ks - q_begin;
      const uint32_t n_items = q_per * (uint32_t)n_valid;
      auto item_row = [&](uint32_t idx, uint32_t& tok) { tok = idx / q_per; return (q_begin + (idx - tok * q_per)) << 2; };
      auto out4 = [&](uint32_t idx, float4 acc) {
        uint32_t tok;
        const uint32_t row = item_row(idx, tok);
        if (p.tw) {
          const int4 t4 = __ldg(reinterpret_cast<const int4*>(p.tw + n0 + row));
          const int txe = __ldg(p.tx + m0 + tok);
          acc.x *= pow2i(t4.x + txe); acc.y *= pow2i(t4.y + txe); acc.z *= pow2i(t4.z + txe); acc.w *= pow2i(t4.w + txe);
        }
        if (F32_OUT) {
          *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.Y) + (m0 + tok) * p.ldy + n0 + row) = acc;
        } else {
          const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
          uint2 w;
          w.x = *reinterpret_cast<const uint32_t*>(&lo);
          w.y = *reinterpret_cast<const uint32_t*>(&hi);
          *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.Y) + (m0 + tok) * p.ldy + n0 + row) = w;
        }
      };
      auto item_off = [&](uint32_t idx) { uint32_t tok; const uint32_t row = item_row(idx, tok); return (tok * TILE_ROWS + row) * 4; };
      // two items per round: up to 16 loads of 16 bytes in flight per thread
      for (uint32_t idx = et; idx < n_items; idx += 256) {
        const uint32_t idx2 = idx + 128;
        const bool two = idx2 < n_items;
        const uint32_t off = item_off(idx), off2 = item_off(two ? idx2 : idx);
        float4 v[8], w[8];
#pragma unroll
        for (uint32_t sp = 0; sp < 8; ++sp) {
          v[sp] = sp < ks ? ptx::ld_cluster_f32x4(peer[sp] + off) : make_float4(0.f, 0.f, 0.f, 0.f);
          w[sp] = (sp < ks && two) ? ptx::ld_cluster_f32x4(peer[sp] + off2) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f), acc2 = acc;
#pragma unroll
        for (uint32_t sp = 0; sp < 8; ++sp) {   // rank order; absent members add +0
          acc.x += v[sp].x; acc.y += v[sp].y; acc.z += v[sp].z; acc.w += v[sp].w;
          acc2.x += w[sp].x; acc2.y += w[sp].y; acc2.z += w[sp].z; acc2.w += w[sp].w;
        }
        out4(idx, acc);
        if (two) out4(idx2, acc2);
      }
    }
    ptx::cluster_sync();                         // nobody leaves while its shared memory may still be read
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) ptx::tmem_dealloc(tmem, tmem_cols);
}

}  // namespace sdq

using namespace sdq;

// SM count of the current device (0 on failure)
static int sm_count_current() {
  const DeviceInfo* d = device_info();
  return d ? d->sm_count : 0;
}

// number of K splits for a call: only for M <= 128 (one token tile), as many as keep one CTA per SM,
// never more than the inlier stages so that every split owns at least one
static int choose_ksplit(int64_t M, int64_t N, int64_t K, int sm_count) {
  if (M > 128 || sm_count <= 0) return 1;
  const int RT = (int)(N / TILE_ROWS), T2 = (int)(K / K2);
  // few tokens: short K chains and two small CTAs per SM hide the per-CTA latencies best
  int ks = (M <= 32 ? 2 * sm_count : sm_count) / RT;
  if (ks > T2) ks = T2;
  if (ks > 32) ks = 32;
  return ks < 1 ? 1 : ks;
}
// CTAs a few-token grid may have per SM, in tenths (two small CTAs fit an SM; a little more runs a short second wave)
#ifndef SDQ_FEW_TOKEN_CTA_BUDGET_TENTHS
#define SDQ_FEW_TOKEN_CTA_BUDGET_TENTHS 20
#endif
static int n_tile_for(int64_t M) { return M > 128 ? 256 : (M > 64 ? 128 : (M > 32 ? 64 : (M > 16 ? 32 : 16))); }

extern "C" sdq_status_t sdq_workspace_size(int64_t M, int64_t N, int64_t K, const sdq_config_t* cfg, size_t* bytes)
{
  if (!cfg || !bytes) return SDQ_ERR_INVALID_ARG;
  if (M <= 0 || N <= 0 || K <= 0 || N % TILE_ROWS || K % K2) return SDQ_ERR_SHAPE;
  const int ks = choose_ksplit(M, N, K, sm_count_current());
  const size_t RT = (size_t)(N / TILE_ROWS);
  // counters first (one per row tile, 256 B aligned), then ks fp32 partial tiles per row tile
  *bytes = ks > 1 ? ((RT * 4 + 255) & ~(size_t)255) + RT * (size_t)ks * (size_t)n_tile_for(M) * TILE_ROWS * 4 : 0;
  return SDQ_OK;
}

static sdq_status_t launch_linear(const sdq_act_t* Xq, const sdq_packed_t* P, void* Y, int64_t ldy, void* ws, size_t ws_bytes,
                                  void* stream, bool f32)
{
  if (!Xq || !P || !Y || !Xq->dev || !P->dev) return SDQ_ERR_INVALID_ARG;
  if (Xq->K != P->K || Xq->M <= 0 || P->N <= 0 || P->N % TILE_ROWS || P->K % K2 || ldy < P->N) return SDQ_ERR_SHAPE;
  if (Xq->cfg.in_block != P->cfg.in_block || Xq->cfg.scale_rule != P->cfg.scale_rule) return SDQ_ERR_SHAPE;
  if (!is_tensor_core_reading(P->cfg)) return SDQ_ERR_UNSUPPORTED;
  if (P->cfg.out_n > 0 && Xq->cfg.out_fmt != P->cfg.out_fmt) return SDQ_ERR_SHAPE;
  if (P->cfg.out_n > 0 && P->cfg.out_fmt == SDQ_OUT_INT8) return SDQ_ERR_UNSUPPORTED;   // int8 outliers: the grouped few-token kernel only
  if (is_compact(*P)) return SDQ_ERR_UNSUPPORTED;                                       // no 2:4 containers in the buffer: likewise
  if (P->cfg.scale_rule == SDQ_SCALE_UE4M3 && !(P->cfg.in_gran == SDQ_GRAN_PAIR && P->cfg.in_block == 32)) return SDQ_ERR_UNSUPPORTED;
  if (((uintptr_t)Y & 15) || (ldy % 8) || ((uintptr_t)ws & 15)) return SDQ_ERR_ALIGNMENT;
  DeviceInfo* dinfo = device_info();
  if (!dinfo) return SDQ_ERR_CUDA;
  if (!dinfo->linear_attr) {     // function attributes belong to the device's context: once per device
    const cudaFuncAttribute a = cudaFuncAttributeMaxDynamicSharedMemorySize;
    if (cudaFuncSetAttribute(sdq_linear_kernel<true, true, false, false>, a, LIN_SMEM_MAX) != cudaSuccess ||
        cudaFuncSetAttribute(sdq_linear_kernel<false, true, false, false>, a, LIN_SMEM_MAX) != cudaSuccess ||
        cudaFuncSetAttribute(sdq_linear_kernel<true, false, false, false>, a, LIN_SMEM_MAX) != cudaSuccess ||
        cudaFuncSetAttribute(sdq_linear_kernel<false, false, false, false>, a, LIN_SMEM_MAX) != cudaSuccess ||
        cudaFuncSetAttribute(sdq_linear_kernel<true, false, true, false>, a, LIN_SMEM_MAX) != cudaSuccess ||
        cudaFuncSetAttribute(sdq_linear_kernel<false, false, true, false>, a, LIN_SMEM_MAX) != cudaSuccess ||
        cudaFuncSetAttribute(sdq_linear_kernel<true, false, false, true>, a, LIN_SMEM_MAX) != cudaSuccess ||
        cudaFuncSetAttribute(sdq_linear_kernel<false, false, false, true>, a, LIN_SMEM_MAX) != cudaSuccess)
      return SDQ_ERR_CUDA;
    dinfo->linear_attr = 1;
  }
  const int sm_count = dinfo->sm_count;
  LinearParams p;
  p.w = (const uint8_t*)P->dev;
  p.x = (const uint8_t*)Xq->dev;
  p.b32 = P->cfg.in_block == 32 ? 1 : 0;
  const bool ue = P->cfg.scale_rule == SDQ_SCALE_UE4M3;
  p.dense = is_dense_layout(P->cfg) ? 1 : 0;   // the n:8, 3:4 and element-wise 2:4 patterns are stored and run like the dense one
  p.poff = tiled_offsets(P->N, P->K, P->cfg);
  p.aoff = act_offsets(Xq->M, Xq->K, p.b32 != 0);
  p.tw = ue ? reinterpret_cast<const int32_t*>(p.w + p.poff.wtexp) : nullptr;
  p.tx = reinterpret_cast<const int32_t*>(p.x + p.aoff.sexp);
  p.M = Xq->M; p.N = P->N; p.K = P->K;
  p.out_n = P->cfg.out_n;
  const int64_t M = Xq->M;
  p.n_tile = n_tile_for(M);
  p.n_mtiles = (int)((M + p.n_tile - 1) / p.n_tile);
  p.slot_bytes = slot_bytes_for(p.n_tile, p.b32 != 0, p.dense != 0);
  p.ksplit = 1;
  p.cluster_ks = 1;
  p.ws_counter = nullptr;
  p.ws_partial = nullptr;
  if (!ws) {
    // cluster split-K: a cluster of up to 8 CTAs per (row tile, token tile), one tile per CTA
    const int tiles = (int)(P->N / TILE_ROWS) * p.n_mtiles, T2c = (int)(P->K / K2);
    // as many members (1..8) as the budget and the inlier stages allow.  Clusters are placed inside one GPC, whose SM count
    // varies: sizes 3, 5, 6, 7 pack worse than powers of two, and a grid that needs every slot then runs a second wave
    // (96 clusters of 3 took 21 us, 96 of 2 take 14), so odd sizes only get 88 % of the budget
    auto split_for = [&](int cta_budget) {
      for (int k = 8; k > 1; --k) {
        const bool pow2 = (k & (k - 1)) == 0;
        if (k <= T2c && (int64_t)k * tiles <= (pow2 ? cta_budget : cta_budget * 22 / 25)) return k;
      }
      return 1;
    };
    int ks = 1;
    if (M <= 128) {
      // CTAs the grid may have: up to 64 tokens the CTAs are small enough for two per SM; from 65 to 128 tokens two
      // per SM leave only three ring slots, which pays only when one per SM would leave many SMs idle
      ks = split_for((M <= 64 ? SDQ_FEW_TOKEN_CTA_BUDGET_TENTHS * sm_count / 10 : sm_count));
      if (M > 64 && ks * tiles * 5 <= sm_count * 3) ks = split_for(2 * sm_count);
      // more row tiles than SMs: one CTA per SM walking whole-K tiles streams a tile in ~19 us however few tiles its
      // last round holds (149 tiles took 38 us, 148 took 16), while two half-K CTAs per SM keep more bytes in flight;
      // split in two and let the grid run in waves of two CTAs per SM (K >= 2048: below that the halves are too short)
      if (ks == 1 && tiles > sm_count && T2c >= 8) ks = 2;
    } else if (tiles * 2 <= sm_count) {
      // a few hundred tokens against a narrow weight matrix: fewer 256-token tiles than half the SMs
      ks = split_for(sm_count);
    }
    if (ks > 1) { p.ksplit = ks; p.cluster_ks = ks; }
  }
  if (ws) {
    const int ks = choose_ksplit(M, P->N, P->K, sm_count);
    size_t need = 0;
    sdq_workspace_size(M, P->N, P->K, &P->cfg, &need);
    if (ks > 1) {
      if (ws_bytes < need) return SDQ_ERR_BUFFER_TOO_SMALL;
      p.ksplit = ks;
      p.ws_counter = (uint32_t*)ws;
      p.ws_partial = (float*)((uint8_t*)ws + (((size_t)(P->N / TILE_ROWS) * 4 + 255) & ~(size_t)255));
    }
  }
  p.total_tiles = (int)(P->N / TILE_ROWS) * p.n_mtiles * p.ksplit;
  p.Y = Y; p.ldy = ldy;
  p.flags = device_flags();
  if (!p.flags) return SDQ_ERR_CUDA;
  // ring geometry: a CTA that runs a single tile with no more stages than fit never reuses a slot, needs only as
  // much shared memory as its stages take (so that small CTAs share an SM) and skips the slot-release traffic
  const int T1 = p.out_n ? (int)(P->K / K1) : 0, T2 = (int)(P->K / K2);
  const int stages_per_tile = (T2 + p.ksplit - 1) / p.ksplit + (T1 + p.ksplit - 1) / p.ksplit;
  // many tokens without K split: the instantiations with compile-time geometry (five ring slots; four with dense inliers)
  const bool many = p.n_tile == 256 && p.ksplit == 1;
  // ... as CTA pairs on tiles of 256 rows x 256 tokens wherever the shape allows (fewer L2 bytes per output)
  if (many && pair_kernel_applies(M, P->N, P->K, p.out_n)) {
    const cudaError_t pe = launch_linear_pair(p, f32, sm_count, (cudaStream_t)stream, &dinfo->pair_attr);
    return pe == cudaSuccess && cudaGetLastError() == cudaSuccess ? SDQ_OK : SDQ_ERR_CUDA;
  }
  int max_slots = many ? (p.dense ? 4 : 5) : RING_BYTES / p.slot_bytes;
  if (p.cluster_ks > 1 && p.total_tiles > sm_count) {
    // cluster split K with more CTAs than SMs (few tokens, one tile per CTA): the grid is one wave only if two CTAs
    // share an SM, so a ring gets half of an SM's shared memory (228 KB, 1 KB of it reserved per CTA)
    const int half = (233472 / 2 - 1024 - SM_TAIL) / p.slot_bytes;
    if (half < max_slots) max_slots = half;
  }
  if (max_slots > MAX_SLOTS) max_slots = MAX_SLOTS;
  int grid_x;
  if (p.total_tiles <= 2 * sm_count && stages_per_tile <= max_slots && p.n_tile <= 32) {
    grid_x = p.total_tiles;
    p.nslot = stages_per_tile;
    p.release = 0;
  } else if (p.cluster_ks > 1) {
    grid_x = p.total_tiles;          // one tile per CTA (the cluster reduction relies on it); total_tiles <= SM count
    p.nslot = max_slots;
    p.release = 1;
  } else {
    grid_x = p.total_tiles < sm_count ? p.total_tiles : sm_count;
    p.nslot = max_slots;
    p.release = 1;
  }
  p.ring_bytes = p.nslot * p.slot_bytes;
  p.meta_col = p.n_tile < 32 ? 32 : p.n_tile;
  int cols = p.meta_col + (int)TM_META_COLS;
  p.tmem_cols = cols <= 128 ? 128 : (cols <= 256 ? 256 : 512);
  const int smem = p.ring_bytes + (many && p.b32 && !p.dense ? SM_TAIL_B32 : SM_TAIL);
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3((unsigned)grid_x);
  lc.blockDim = dim3(LIN_THREADS);   // the many-token instantiations get LIN_THREADS_MANY below
  lc.dynamicSmemBytes = (size_t)smem;
  lc.stream = (cudaStream_t)stream;
  // the kernel may be scheduled while the previous one in the stream drains: set-up and weight copies overlap its tail
  cudaLaunchAttribute attr[2];
  int na = 0;
  attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[na].val.programmaticStreamSerializationAllowed = 1;
  ++na;
  if (p.cluster_ks > 1) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = (unsigned)p.cluster_ks;
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  lc.attrs = attr;
  lc.numAttrs = na;
  const bool flex = !many;
  if (!flex) lc.blockDim = dim3(LIN_THREADS_MANY);
  cudaError_t le;
  if (flex) le = f32 ? cudaLaunchKernelEx(&lc, sdq_linear_kernel<true, true, false, false>, p) : cudaLaunchKernelEx(&lc, sdq_linear_kernel<false, true, false, false>, p);
  else if (p.dense) le = f32 ? cudaLaunchKernelEx(&lc, sdq_linear_kernel<true, false, false, true>, p) : cudaLaunchKernelEx(&lc, sdq_linear_kernel<false, false, false, true>, p);
  else if (p.b32) le = f32 ? cudaLaunchKernelEx(&lc, sdq_linear_kernel<true, false, true, false>, p) : cudaLaunchKernelEx(&lc, sdq_linear_kernel<false, false, true, false>, p);
  else le = f32 ? cudaLaunchKernelEx(&lc, sdq_linear_kernel<true, false, false, false>, p) : cudaLaunchKernelEx(&lc, sdq_linear_kernel<false, false, false, false>, p);
  return le == cudaSuccess && cudaGetLastError() == cudaSuccess ? SDQ_OK : SDQ_ERR_CUDA;
}

extern "C" sdq_status_t sdq_linear(const sdq_act_t* Xq, const sdq_packed_t* P, void* Y, int64_t ldy, void* stream)
{ return launch_linear(Xq, P, Y, ldy, nullptr, 0, stream, false); }

extern "C" sdq_status_t sdq_linear_f32(const sdq_act_t* Xq, const sdq_packed_t* P, float* Y, int64_t ldy, void* stream)
{ return launch_linear(Xq, P, (void*)Y, ldy, nullptr, 0, stream, true); }

extern "C" sdq_status_t sdq_workspace_init(void* ws, size_t ws_bytes, void* stream)
{
  if (!ws) return SDQ_ERR_INVALID_ARG;
  if ((uintptr_t)ws & 15) return SDQ_ERR_ALIGNMENT;
  return cudaMemsetAsync(ws, 0, ws_bytes, (cudaStream_t)stream) == cudaSuccess ? SDQ_OK : SDQ_ERR_CUDA;
}

extern "C" sdq_status_t sdq_linear_ws(const sdq_act_t* Xq, const sdq_packed_t* P, void* Y, int64_t ldy, void* ws, size_t ws_bytes,
                                      void* stream)
{ return launch_linear(Xq, P, Y, ldy, ws, ws_bytes, stream, false); }

extern "C" sdq_status_t sdq_linear_f32_ws(const sdq_act_t* Xq, const sdq_packed_t* P, float* Y, int64_t ldy, void* ws, size_t ws_bytes,
                                          void* stream)
{ return launch_linear(Xq, P, (void*)Y, ldy, ws, ws_bytes, stream, true); }

// ---------------------------------------------------------------------------------------------------------
// Several independent layers in one call (see include/sdq.h).  Few tokens everywhere and enough row tiles to occupy
// the GPU: one persistent launch of the grouped kernel; otherwise the layers are enqueued one after the other.
static sdq_status_t launch_group(int n, const sdq_act_t* const* Xq, const sdq_packed_t* const* P, void* const* Y, const int64_t* ldy,
                                 void* stream, bool f32)
{
  if (n <= 0 || !Xq || !P || !Y || !ldy) return SDQ_ERR_INVALID_ARG;
  DeviceInfo* dinfo = device_info();
  if (!dinfo) return SDQ_ERR_CUDA;
  bool fused = n <= GROUP_MAX;
  int64_t items = 0, max_m = 0;
  for (int i = 0; i < n; ++i) {
    const sdq_act_t* x = Xq[i];
    const sdq_packed_t* w = P[i];
    if (!x || !w || !Y[i] || !x->dev || !w->dev) return SDQ_ERR_INVALID_ARG;
    if (x->K != w->K || x->M <= 0 || w->N <= 0 || w->N % TILE_ROWS || w->K % K2 || ldy[i] < w->N) return SDQ_ERR_SHAPE;
    if (x->cfg.in_block != w->cfg.in_block || x->cfg.scale_rule != w->cfg.scale_rule) return SDQ_ERR_SHAPE;
    if (!is_tensor_core_reading(w->cfg)) return SDQ_ERR_UNSUPPORTED;
    if (w->cfg.out_n > 0 && x->cfg.out_fmt != w->cfg.out_fmt) return SDQ_ERR_SHAPE;
    if (((uintptr_t)Y[i] & 15) || (ldy[i] % 8)) return SDQ_ERR_ALIGNMENT;
    // the grouped kernel carries the primary format: pair-wise 4:8 inliers, one E8M0 scale per 64 K, at most one outlier per S-Vector
    fused = fused && x->M <= 32 && w->cfg.in_gran == SDQ_GRAN_PAIR && w->cfg.in_block == 64 && w->cfg.scale_rule != SDQ_SCALE_UE4M3 &&
            w->cfg.out_n <= 1 && w->cfg.out_n == P[0]->cfg.out_n && w->cfg.out_fmt == P[0]->cfg.out_fmt &&
            w->K >= 4 * K2;   // an item spans at least half the ring: the kernel's per-item barriers then never run two phases apart
    items += w->N / TILE_ROWS;
    if (x->M > max_m) max_m = x->M;
  }
  fused = fused && items * 2 >= dinfo->sm_count && items < (1 << 30);
  if (!fused) {
    for (int i = 0; i < n; ++i) {
      const sdq_status_t st = launch_linear(Xq[i], P[i], Y[i], ldy[i], nullptr, 0, stream, f32);
      if (st != SDQ_OK) return st;
    }
    return SDQ_OK;
  }
  GroupParams g;
  g.n = n;
  g.n_tile = max_m <= 16 ? 16 : 32;
  g.out_n = P[0]->cfg.out_n;
  g.out_i8 = g.out_n > 0 && P[0]->cfg.out_fmt == SDQ_OUT_INT8;
  g.x_bf16 = nullptr; g.x_ld = 0; g.x_M = 0; g.scale_rule = P[0]->cfg.scale_rule;
  g.total_items = (int)items;
  g.flags = device_flags();
  if (!g.flags) return SDQ_ERR_CUDA;
  int item0 = 0;
  for (int i = 0; i < n; ++i) {
    const PackedOffsets po = tiled_offsets(*P[i]);
    const ActOffsets ao = act_offsets(Xq[i]->M, Xq[i]->K, false);
    GroupMat& m = g.m[i];
    m.w = (const uint8_t*)P[i]->dev; m.x = (const uint8_t*)Xq[i]->dev; m.Y = Y[i]; m.ldy = ldy[i];
    m.wi = po.wi; m.wc = po.wc; m.sfa_out = po.sfa_out;
    m.xi = ao.xi; m.xo = ao.xo; m.sfb_out = ao.sfb_out;
    m.wsc = po.osexp; m.xsc = ao.sexp;
    m.M = (int)Xq[i]->M; m.T2 = (int)(P[i]->K / K2);
    m.item0 = item0;
    item0 += (int)(P[i]->N / TILE_ROWS);
  }
  const cudaError_t e = launch_linear_group(g, f32, dinfo->sm_count, (cudaStream_t)stream, &dinfo->group_attr);
  return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? SDQ_OK : SDQ_ERR_CUDA;
}

// The same with the activation quantizer inside the kernel: all layers read one bf16 X (see include/sdq.h).
static sdq_status_t launch_group_x(int n, const void* X, int64_t M, int64_t K, int64_t ldx, const sdq_packed_t* const* P, void* const* Y,
                                   const int64_t* ldy, void* stream, bool f32)
{
  if (n <= 0 || !X || !P || !Y || !ldy) return SDQ_ERR_INVALID_ARG;
  if (M <= 0 || K <= 0 || K % K2 || ldx < K) return SDQ_ERR_SHAPE;
  if (((uintptr_t)X & 15) || (ldx % 8)) return SDQ_ERR_ALIGNMENT;
  DeviceInfo* dinfo = device_info();
  if (!dinfo) return SDQ_ERR_CUDA;
  int64_t items = 0;
  for (int i = 0; i < n; ++i) {
    const sdq_packed_t* w = P[i];
    if (!w || !Y[i] || !w->dev) return SDQ_ERR_INVALID_ARG;
    if (w->K != K || w->N <= 0 || w->N % TILE_ROWS || ldy[i] < w->N) return SDQ_ERR_SHAPE;
    if (!is_tensor_core_reading(w->cfg)) return SDQ_ERR_UNSUPPORTED;
    if (((uintptr_t)Y[i] & 15) || (ldy[i] % 8)) return SDQ_ERR_ALIGNMENT;
    const sdq_config_t& c = w->cfg, &c0 = P[0]->cfg;
    if (c.in_gran != SDQ_GRAN_PAIR || c.in_block != 64 || c.scale_rule == SDQ_SCALE_UE4M3 || c.out_n > 1 || c.out_n != c0.out_n ||
        c.out_fmt != c0.out_fmt || c.scale_rule != c0.scale_rule)
      return SDQ_ERR_UNSUPPORTED;
    items += w->N / TILE_ROWS;
  }
  // (the in-kernel quantizer keeps a token's K <= 4096 elements in the registers of its 11 x 4 lanes)
  if (n > GROUP_MAX || M > 16 || K < 4 * K2 || K > 16 * K2 || !group_xres_fits((int)(K / K2), P[0]->cfg.out_n) || items * 2 < dinfo->sm_count || items >= (1 << 30))
    return SDQ_ERR_UNSUPPORTED;
  GroupParams g;
  g.n = n;
  g.n_tile = 16;
  g.out_n = P[0]->cfg.out_n;
  g.out_i8 = g.out_n > 0 && P[0]->cfg.out_fmt == SDQ_OUT_INT8;
  g.x_bf16 = X; g.x_ld = ldx; g.x_M = (int)M; g.scale_rule = P[0]->cfg.scale_rule;
  g.total_items = (int)items;
  g.flags = device_flags();
  if (!g.flags) return SDQ_ERR_CUDA;
  int item0 = 0;
  for (int i = 0; i < n; ++i) {
    const PackedOffsets po = tiled_offsets(*P[i]);
    GroupMat& m = g.m[i];
    m.w = (const uint8_t*)P[i]->dev; m.x = nullptr; m.Y = Y[i]; m.ldy = ldy[i];
    m.wi = po.wi; m.wc = po.wc; m.sfa_out = po.sfa_out;
    m.xi = m.xo = m.sfb_out = m.xsc = 0;
    m.wsc = po.osexp;
    m.M = (int)M; m.T2 = (int)(K / K2);
    m.item0 = item0;
    item0 += (int)(P[i]->N / TILE_ROWS);
  }
  const cudaError_t e = launch_linear_group(g, f32, dinfo->sm_count, (cudaStream_t)stream, &dinfo->group_attr);
  return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? SDQ_OK : SDQ_ERR_CUDA;
}

extern "C" sdq_status_t sdq_linear_group_x(int n, const void* X_bf16, int64_t M, int64_t K, int64_t ldx, const sdq_packed_t* const* P,
                                           void* const* Y, const int64_t* ldy, void* stream)
{ return launch_group_x(n, X_bf16, M, K, ldx, P, Y, ldy, stream, false); }

extern "C" sdq_status_t sdq_linear_group_x_f32(int n, const void* X_bf16, int64_t M, int64_t K, int64_t ldx, const sdq_packed_t* const* P,
                                               float* const* Y, const int64_t* ldy, void* stream)
{ return launch_group_x(n, X_bf16, M, K, ldx, P, (void* const*)Y, ldy, stream, true); }

extern "C" sdq_status_t sdq_linear_group(int n, const sdq_act_t* const* Xq, const sdq_packed_t* const* P, void* const* Y,
                                         const int64_t* ldy, void* stream)
{ return launch_group(n, Xq, P, Y, ldy, stream, false); }

extern "C" sdq_status_t sdq_linear_group_f32(int n, const sdq_act_t* const* Xq, const sdq_packed_t* const* P, float* const* Y,
                                             const int64_t* ldy, void* stream)
{ return launch_group(n, Xq, P, (void* const*)Y, ldy, stream, true); }

// ---------------------------------------------------------------------------------------------------------
// Allocation-free variant of sdq_linear_ws (see include/sdq.h).  The split-K scratch lives in this library's
// own device image instead of a caller buffer.
namespace sdq {
static __device__ __align__(256) unsigned char g_static_ws[SDQ_STATIC_WS_BYTES];
}

// Device address of the built-in scratch for the current device.  `g_static_ws` in host code is only a handle
// for the symbol, not an address a kernel could use, so the address is asked from the runtime, once per
// device and with that device current.
static void* static_ws_address() {
  static void* cache[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!cache[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, sdq::g_static_ws) != cudaSuccess) return nullptr;
    cache[dev] = ptr;
  }
  return cache[dev];
}

extern "C" sdq_status_t sdq_linear_noalloc(const sdq_act_t* Xq, const sdq_packed_t* P, void* Y, int64_t ldy, void* stream)
{
  if (!Xq || !P) return SDQ_ERR_INVALID_ARG;
  size_t need = 0;
  const sdq_status_t st = sdq_workspace_size(Xq->M, P->N, P->K, &P->cfg, &need);
  if (st != SDQ_OK) return st;
  if (need == 0) return launch_linear(Xq, P, Y, ldy, nullptr, 0, stream, false);   // this shape uses no scratch
  if (need > (size_t)SDQ_STATIC_WS_BYTES) return SDQ_ERR_BUFFER_TOO_SMALL;
  void* ws = static_ws_address();
  if (!ws) return SDQ_ERR_CUDA;
  // the array keeps whatever the previous call left: the arrival counters must start at zero
  const size_t counter_bytes = ((size_t)(P->N / TILE_ROWS) * 4 + 255) & ~(size_t)255;
  if (cudaMemsetAsync(ws, 0, counter_bytes, (cudaStream_t)stream) != cudaSuccess) return SDQ_ERR_CUDA;
  return launch_linear(Xq, P, Y, ldy, ws, need, stream, false);
}
