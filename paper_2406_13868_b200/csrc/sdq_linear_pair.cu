// Fused decomposed GEMM for many tokens, CTA-pair form  Y = A_i W_i^T + A_o W_o^T   (Section 5.1: O = O_i + O_o)
//
// The many-token layer is bound by the bytes a tile pulls from L2 into shared memory, and three quarters of those are
// activation codes that every row tile fetches again.  Here the two CTAs of a cluster work as one tensor-core unit
// (tcgen05 cta_group::2) on a tile of 256 weight rows x 256 tokens: CTA r stages weight rows 128 r .. 128 r + 127 and
// the codes of tokens 128 r .. 128 r + 127 only, and the pair-wide MMA takes half of its B operand from each CTA's
// shared memory -- 27 KB per CTA and stage instead of 43 KB for the same MMA time.  The stage sequence of a tile is
// that of the single-CTA kernel (all inlier stages of 256 K, then all outlier stages of 128 K, one fp32 accumulator).
//
// Per CTA: warps 0 / 6 / 7 bulk-copy producers (own weight records / own activation codes / scale atoms of both token
// halves; two lanes each, see there), warps 2..5 and 9..12 epilogue (own 128 rows x 256 tokens: TMEM -> registers as
// packed bf16, TMEM handed back, transposed stores under the next tile's K loop).  Even CTA (leader): warp 1 copies
// metadata and scales of both CTAs to TMEM (pair-wide tcgen05.cp) and issues the pair-wide MMAs; its tcgen05.commit
// signals "slots consumed" / "accumulator complete" to the barriers of both CTAs.  Odd CTA: two lanes of warp 1
// forward "my part of the slot has landed" to the leader's barriers.  Every wait is bounded.
//
// What was measured on the way (B200, 2048 tokens, 4096 -> 11008, 1:8 outliers; the single-CTA kernel takes 84 us):
// a first version with one release per slot, a separate TMEM-mover thread and cluster-scope release / acquire on the
// forwarding hop took 213 us -- a remote mbarrier arrive with .release.cluster costs ~0.8 us under load (the default
// semantics suffice: the data was written by the bulk-copy engine and is read by the tensor core, both outside the
// forwarding thread's view of memory) -> 94 us; warp-uniform issue loops, the copies to TMEM folded into the MMA issuer,
// one barrier per slot and batches of landed slots -> 78 us; two lanes per producer -> 67 us (2.75 PFLOP/s).
#include <cuda_bf16.h>

#include "sdq_internal.h"
#include "sdq_layout.h"
#include "sdq_linear.h"
#include "sdq_ptx.cuh"

namespace sdq {

constexpr int PAIR_THREADS = 416;            // 13 warps
constexpr int PAIR_MAX_SLOTS = 8;
constexpr int PAIR_TAIL = 2048 + 384 + 128;  // transpose buffer (2 groups x 4 tokens x 128 features bf16) + barriers + alignment slack

template <bool B32, bool DENSE>
struct PairGeom {
  static constexpr bool S32 = B32 || DENSE;                       // one scale per 32 K
  static constexpr uint32_t WIB = DENSE ? 17408u : (B32 ? 11264u : 10752u);   // inlier weight record (>= the outlier record)
  static constexpr uint32_t NA = S32 ? 2u : 1u;                   // scale atoms per token tile and inlier stage
  static constexpr uint32_t ATOMS = S32 ? 4u : 3u;                // inlier: NA per token half; first outlier stage: SFA_out + 2 SFB_out
  static constexpr uint32_t SL_B = WIB;                           // own 128 tokens: B4 (256 K) or B8 (128 K)
  static constexpr uint32_t SL_SF = WIB + 16384u;
  static constexpr uint32_t SLOT = SL_SF + ATOMS * SF_ATOM_BYTES; // 28672 / 29696 / 35840
  static constexpr uint32_t NSLOT = S32 ? 6u : 8u;                // ring slots, released two at a time (see the MMA issuer)
  static constexpr uint32_t MS = S32 ? 32u : 16u;                 // TMEM columns of metadata / scales per ring slot
  static constexpr uint32_t SM_STG = NSLOT * SLOT;                // transpose buffer, then the barriers
  static constexpr uint32_t SM_BARS = SM_STG + 2048u;
  static constexpr uint32_t SMEM = SM_STG + PAIR_TAIL;
  static_assert(256u + MS * NSLOT + 24u <= 512u, "TMEM columns");
  static_assert(SMEM <= 232448u, "shared memory");
};

template <bool F32_OUT, bool B32, bool DENSE>
__global__ void __cluster_dims__(2, 1, 1) __maxnreg__(128)
sdq_linear_pair_kernel(const LinearParams p)
{
  using G = PairGeom<B32, DENSE>;
  constexpr bool S32 = G::S32;
  constexpr uint32_t NSLOT = G::NSLOT, SLOT = G::SLOT, MS = G::MS, NA = G::NA;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint8_t* sm = smem_raw + ((128 - (ptx::smem_u32(smem_raw) & 127)) & 127);
  uint64_t* full = reinterpret_cast<uint64_t*>(sm + G::SM_BARS);   // the three producers' parts of slot s have landed (leader: + the peer's)
  uint64_t* empty = full + PAIR_MAX_SLOTS;                         // [s / 2]: the MMAs that read slots s and s ^ 1 have completed
  uint64_t* acc_full = empty + PAIR_MAX_SLOTS;
  uint64_t* acc_empty = acc_full + 1;                              // leader: all 16 epilogue warps of the pair have drained TMEM
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 1);
  volatile uint32_t* timed_out = tmem_slot + 1;                    // an epilogue group's wait gave up

  const uint32_t rank = ptx::cluster_ctarank();                    // 0 = leader
  const int pair = (int)(blockIdx.x >> 1), n_pairs = (int)(gridDim.x >> 1);
  const int RTP = (int)(p.N / (2 * TILE_ROWS));                    // row-pair tiles
  const int T1 = p.out_n ? (int)(p.K / K1) : 0, T2 = (int)(p.K / K2);
  const uint32_t xib = (uint32_t)xi_bytes(S32);

  if (tid == 0) ptx::griddep_launch_dependents();
  if (tid == 0) {
    *timed_out = 0u;
    for (uint32_t s = 0; s < NSLOT; ++s) {
      ptx::mbar_init(&full[s], rank == 0 ? 4 : 3);
      if (!(s & 1)) ptx::mbar_init(&empty[s >> 1], 1);
    }
    ptx::mbar_init(acc_full, 1);
    ptx::mbar_init(acc_empty, 16);
    ptx::fence_barrier_init();
  }
  if (warp == 1) ptx::tmem_alloc_pair(tmem_slot, 512);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync();                                             // both CTAs' barriers exist before any remote arrival
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0 || warp == 6 || warp == 7) {
    if (lane < 2) {
      // ---------------- producers (both CTAs): role 0 = own weight records, 1 = own activation codes, 2 = scale atoms.
      // One trip of a producer's loop (barrier wait, address arithmetic, expect-tx, copy) takes ~0.3 us, which one thread
      // per role cannot hide at two MMAs per stage; ring slots are released in pairs, so lanes 0 and 1 of the warp run the
      // loop in lockstep, lane l filling the slots of parity l: two stages per trip.
      const int role = warp == 0 ? 0 : (int)warp - 5;
      if (role != 0) ptx::griddep_wait();    // activations come from an earlier kernel; weights do not
      const int S = T2 + T1;
      const int my_tiles = p.total_tiles > pair ? (p.total_tiles - pair + n_pairs - 1) / n_pairs : 0;
      const int total = my_tiles * S;                                        // stages of this CTA, numbered through its tiles
      const size_t xi_tile = (size_t)T2 * xib, xo_tile = (size_t)T1 * XO_BYTES;
      bool ok = true;
      uint32_t s = lane, wrapped = 0, ph = 0;
      int tseq = 0, k = (int)lane;                                           // this lane's stage: tile number in the CTA's sequence, stage in the tile
      if (k >= S) { k -= S; ++tseq; }                                        // (S >= 2)
      int cur = -1, rt = 0, mt0 = 0, have = 0;
      bool own = false;
      for (int i = (int)lane; i < total && ok; i += 2) {
        if (tseq != cur) {
          cur = tseq;
          const int tile = pair + tseq * n_pairs;
          rt = 2 * (tile % RTP) + (int)rank;
          mt0 = 2 * (tile / RTP);                                            // first activation tile of the token tile
          have = min(2, (int)p.aoff.MT - mt0);                               // activation tiles that exist (1 or 2)
          own = (int)rank < have;                                            // this CTA's 128 tokens exist
        }
        if (wrapped && !(ok = ptx::mbar_wait(&empty[s >> 1], ph ^ 1))) break;
        uint8_t* st = sm + (size_t)s * SLOT;
        const bool inl = k < T2, first_o = (k == T2);
        const int ko = k - T2;                                               // outlier stage number
        if (role == 0) {
          if (inl) {
            ptx::mbar_expect_tx(&full[s], G::WIB);
            ptx::bulk_g2s(st, p.w + p.poff.wi + ((size_t)rt * T2 + k) * G::WIB, G::WIB, &full[s]);
          } else {
            ptx::mbar_expect_tx(&full[s], WO_BYTES + (first_o ? SF_ATOM_BYTES : 0u));
            ptx::bulk_g2s(st, p.w + p.poff.wo + ((size_t)rt * T1 + ko) * WO_BYTES, WO_BYTES, &full[s]);
            if (first_o) ptx::bulk_g2s(st + G::SL_SF, p.w + p.poff.sfa_out + (size_t)rt * SF_ATOM_BYTES, SF_ATOM_BYTES, &full[s]);
          }
        } else if (role == 1) {
          if (!own) {
            ptx::mbar_arrive(&full[s]);
          } else if (inl) {
            ptx::mbar_expect_tx(&full[s], B4_BYTES);
            ptx::bulk_g2s(st + G::SL_B, p.x + p.aoff.xi + (size_t)(mt0 + (int)rank) * xi_tile + (size_t)k * xib, B4_BYTES, &full[s]);
          } else {
            ptx::mbar_expect_tx(&full[s], B8_BYTES);
            ptx::bulk_g2s(st + G::SL_B, p.x + p.aoff.xo + (size_t)(mt0 + (int)rank) * xo_tile + (size_t)ko * XO_BYTES, B8_BYTES, &full[s]);
          }
        } else {
          if (inl) {
            ptx::mbar_expect_tx(&full[s], (uint32_t)have * NA * SF_ATOM_BYTES);
            for (int a = 0; a < have; ++a)
              ptx::bulk_g2s(st + G::SL_SF + a * NA * SF_ATOM_BYTES, p.x + p.aoff.xi + (size_t)(mt0 + a) * xi_tile + (size_t)k * xib + B4_BYTES,
                            NA * SF_ATOM_BYTES, &full[s]);
          } else if (first_o) {
            ptx::mbar_expect_tx(&full[s], (uint32_t)have * SF_ATOM_BYTES);
            for (int a = 0; a < have; ++a)
              ptx::bulk_g2s(st + G::SL_SF + (1 + a) * SF_ATOM_BYTES, p.x + p.aoff.sfb_out + (size_t)(mt0 + a) * SF_ATOM_BYTES, SF_ATOM_BYTES,
                            &full[s]);
          } else {
            ptx::mbar_arrive(&full[s]);
          }
        }
        s += 2;
        if (s >= NSLOT) { s -= NSLOT; wrapped = 1; ph ^= 1; }
        k += 2;
        if (k >= S) { k -= S; ++tseq; }
      }
      if (!ok) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
    }
  } else if (warp == 1 && rank == 1) {
    if (lane < 2) {
      // ---------------- odd CTA: forward "my part of the slot has landed" to the leader's barrier (lane l: slots of parity l)
      const int S = T2 + T1;
      const int my_tiles = p.total_tiles > pair ? (p.total_tiles - pair + n_pairs - 1) / n_pairs : 0;
      const int total = my_tiles * S;
      bool ok = true;
      uint32_t s = lane, ph = 0;
      for (int i = (int)lane; i < total; i += 2) {
        if (!(ok = ptx::mbar_wait(&full[s], ph))) break;
        ptx::mbar_arrive_remote(&full[s], 0);
        s += 2;
        if (s >= NSLOT) { s -= NSLOT; ph ^= 1; }
      }
      if (!ok) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
    }
  } else if (warp == 1) {
    {
      // ---------------- MMA issuer (leader): per slot the copies of metadata and scales to TMEM (both CTAs), then the
      // pair-wide MMAs; tcgen05.cp and tcgen05.mma of one thread execute in issue order, so nothing waits in between, and
      // TMEM buffer s (metadata, scales) simply belongs to ring slot s.
      // The whole warp runs the loop and one elected lane issues: descriptors and TMEM addresses of tcgen05 instructions
      // are uniform-register operands, and only warp-uniform control flow keeps the loop's arithmetic on the uniform
      // datapath.  Even so one trip of the loop (barrier test, vote, election) costs more than the tensor pipe needs for
      // the two MMAs of a slot, so a trip takes every slot that has landed: lane i tests slot s + i, one ballot gives the
      // run of ready slots, and their instructions go out back to back.  When the pipe is the bottleneck the batches grow
      // and the loop cost is spread; when the copies are, a batch is one slot and the loop is idle anyway.
      // A pair-wide commit costs the pipe a bubble of ~80 ns (measured), hence one release per two slots.
      bool ok = true;
      const uint32_t smb = ptx::smem_u32(sm);
      uint32_t s = 0, ph = 0, tcount = 0;
      // (two-level scaling: the .block16 kind reads its scale codes as unsigned E4M3 when bit 23 is clear)
      const uint32_t id4[2] = {ptx::idesc_block_scaled(256, 256, 1, true, 0, 0) ^ (p.tw ? (1u << 23) : 0u),
                               ptx::idesc_block_scaled(256, 256, 1, true, 2, 2)};
      const uint32_t id8 = ptx::idesc_block_scaled(256, 256, 0, true, 0, 0);
      const uint32_t idd[2] = {ptx::idesc_block_scaled(256, 256, 1, false, 0, 0), ptx::idesc_block_scaled(256, 256, 1, false, 2, 2)};
      const uint64_t d_a = ptx::smem_desc(smb, 128, 256), d_b = ptx::smem_desc(smb + G::SL_B, 128, 1024);
      const uint64_t d_e_in = ptx::smem_desc(smb + A_IN_BYTES, 0, 128);
      const uint64_t d_sfa_in = ptx::smem_desc(smb + (DENSE ? 2 * A_IN_BYTES : A_IN_BYTES + E_IN_BYTES), 0, 128);
      const uint64_t d_e_out = ptx::smem_desc(smb + A_OUT_BYTES, 0, 128);
      const uint64_t d_sf0 = ptx::smem_desc(smb + G::SL_SF, 0, 128), d_sf1 = ptx::smem_desc(smb + G::SL_SF + SF_ATOM_BYTES, 0, 128);
      const uint64_t d_sf2 = ptx::smem_desc(smb + G::SL_SF + 2 * SF_ATOM_BYTES, 0, 128);
      constexpr uint32_t slot16 = SLOT >> 4;
      const int S = T2 + T1;
      for (int tile = pair; tile < p.total_tiles && ok; tile += n_pairs, ++tcount) {
        const uint32_t sfo = tmem + 256u + MS * NSLOT + 12u * (tcount & 1);   // outlier row / token scales: two alternating buffers
        int k = 0;
        while (k < S) {
          // lane i: has slot s + i (the i-th next stage of this tile) landed in both CTAs?
          const uint32_t idx = s + lane, sl = idx >= NSLOT ? idx - NSLOT : idx;
          // (four slots ahead at most: testing all eight costs more per trip than the longer runs save, measured 1 %)
          const bool r = (int)lane < min(4, S - k) && ptx::mbar_test(&full[sl], idx >= NSLOT ? ph ^ 1 : ph);
          int n = __ffs(~__ballot_sync(0xffffffffu, r)) - 1;     // length of the run of ready slots
          if (n == 0) {   // nothing yet: wait for the next slot, then look again (its neighbours tend to land with it)
            ok = __all_sync(0xffffffffu, ptx::mbar_wait(&full[s], ph));
            if (!ok) break;
            continue;
          }
          if (k == 0 && tcount > 0) {   // the epilogues of both CTAs must have drained the accumulator of the previous tile
            ok = __all_sync(0xffffffffu, ptx::mbar_wait(acc_empty, (tcount - 1) & 1));
            if (!ok) break;
          }
          ptx::tc_fence_after();
          if (ptx::elect_one()) {
            uint32_t ss = s;
            for (int kk = k; kk < k + n; ++kk) {
              const uint64_t so = (uint64_t)(ss * slot16);
              const uint32_t mb = tmem + 256u + MS * ss;
              const uint32_t acc = kk ? 1u : 0u;   // the first MMA of the tile overwrites the accumulator
              if (kk < T2) {
                if constexpr (!DENSE) ptx::tc2_cp_128x128b(mb + 0, d_e_in + so);
                ptx::tc2_cp_32x128b_warpx4(mb + 4, d_sfa_in + so);
                if constexpr (S32) {
                  // scale words: weights K-block 0 / 1 at +4 / +8; tokens K-block kb, token tile a at +12 + 4 (2 kb + a), staged
                  // as [token tile][K-block]
                  ptx::tc2_cp_32x128b_warpx4(mb + 8, d_sfa_in + so + (SF_ATOM_BYTES >> 4));
                  ptx::tc2_cp_32x128b_warpx4(mb + 12, d_sf0 + so);
                  ptx::tc2_cp_32x128b_warpx4(mb + 20, d_sf1 + so);
                  ptx::tc2_cp_32x128b_warpx4(mb + 16, d_sf2 + so);
                  ptx::tc2_cp_32x128b_warpx4(mb + 24, d_sf2 + so + (SF_ATOM_BYTES >> 4));
                } else {
                  ptx::tc2_cp_32x128b_warpx4(mb + 8, d_sf0 + so);
                  ptx::tc2_cp_32x128b_warpx4(mb + 12, d_sf1 + so);
                }
                if constexpr (DENSE) {
#pragma unroll
                  for (uint32_t j = 0; j < 4; ++j)
                    ptx::mma2_mxf4(tmem, d_a + so + ((4096 * j) >> 4), d_b + so + ((256 * j) >> 4), idd[j & 1], mb + 4 + 4 * (j >> 1),
                                   mb + 12 + 8 * (j >> 1), j ? 1u : acc);
                } else if constexpr (B32) {
                  ptx::mma2_sp_nvf4(tmem, d_a + so, d_b + so, id4[0], mb, mb + 4, mb + 12, acc);
                  ptx::mma2_sp_nvf4(tmem, d_a + so + (4096 >> 4), d_b + so + (512 >> 4), id4[0], mb + 2, mb + 8, mb + 20, 1u);
                } else {
                  ptx::mma2_sp_mxf4(tmem, d_a + so, d_b + so, id4[0], mb, mb + 4, mb + 8, acc);
                  ptx::mma2_sp_mxf4(tmem, d_a + so + (4096 >> 4), d_b + so + (512 >> 4), id4[1], mb + 2, mb + 4, mb + 8, 1u);
                }
              } else {
                ptx::tc2_cp_128x128b(mb + 0, d_e_out + so);
                if (kk == T2) {
                  ptx::tc2_cp_32x128b_warpx4(sfo, d_sf0 + so);
                  ptx::tc2_cp_32x128b_warpx4(sfo + 4, d_sf1 + so);
                  ptx::tc2_cp_32x128b_warpx4(sfo + 8, d_sf2 + so);
                }
                ptx::mma2_sp_mxf8(tmem, d_a + so, d_b + so, id8, mb, sfo, sfo + 4, acc);
                ptx::mma2_sp_mxf8(tmem, d_a + so + (4096 >> 4), d_b + so + (512 >> 4), id8, mb + 2, sfo, sfo + 4, 1u);
              }
              if (ss & 1) ptx::tc2_commit_both(&empty[ss >> 1]);     // slots ss - 1 and ss may be refilled (both CTAs)
              if (kk == S - 1) ptx::tc2_commit_both(acc_full);       // the tile's accumulator is complete (both CTAs)
              if (++ss == NSLOT) ss = 0;
            }
          }
          __syncwarp();
          k += n;
          s += (uint32_t)n;
          if (s >= NSLOT) { s -= NSLOT; ph ^= 1; }
        }
      }
      // (a kernel whose stage count is odd leaves its last slot unreleased: nobody waits for it)
      if (!ok && lane == 0) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
    }
  } else if ((warp >= 2 && warp <= 5) || warp >= 9) {
    // ---------------- epilogue (both CTAs): warp w owns TMEM lanes 32 (w % 4) .. + 31 (own weight rows); group 0 (warps 2..5)
    // takes tokens 0..127 of the tile, group 1 (warps 9..12) tokens 128..255
    const uint32_t q = warp & 3;
    const uint32_t grp = warp >= 9 ? 1u : 0u;
    const uint32_t et = (warp - (grp ? 9u : 2u)) * 32 + lane;
    uint32_t tcount = 0;
    bool ok = true;
    auto hand_back = [&]() {      // this warp has read its part of the accumulator
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) { if (rank == 0) ptx::mbar_arrive(acc_empty); else ptx::mbar_arrive_remote(acc_empty, 0); }
    };
    ptx::griddep_wait();                            // Y may still be in use by the previous kernel
    for (int tile = pair; tile < p.total_tiles && ok; tile += n_pairs, ++tcount) {
      const int rt = 2 * (tile % RTP) + (int)rank, mtile = tile / RTP;
      const int64_t m0 = (int64_t)mtile * 256;
      const int n_valid = (int)min((int64_t)256, p.M - m0);
      // one thread per group polls the barrier and releases the other 127 through a hardware barrier: hundreds of threads
      // polling one mbarrier notice its completion late and slow the CTA's other barrier traffic down
      if (et == 0 && !ptx::mbar_wait(acc_full, tcount & 1)) *timed_out = 1u;
      ptx::named_bar_sync(3 + grp, 128);
      if (*timed_out) { ok = false; break; }
      ptx::tc_fence_after();
      const int64_t n0 = (int64_t)rt * TILE_ROWS;
      const int twr = p.tw ? __ldg(p.tw + n0 + q * 32 + lane) : 0;     // two-level scaling: this thread's row factor
      if constexpr (F32_OUT) {
        // fp32 output (tests): the first group stores everything, straight from TMEM
        if (grp) { hand_back(); continue; }
        float* Y = reinterpret_cast<float*>(p.Y);
#pragma unroll 1
        for (int c0 = 0; c0 < 256; c0 += 16) {
          uint32_t v[16];
          if (c0 < n_valid) {
            ptx::tmem_ld_32x32b_x16(tmem + ((q * 32u) << 16) + (uint32_t)c0, v);
            ptx::tmem_ld_wait();
          }
          if (c0 + 16 >= 256) hand_back();
          if (c0 >= n_valid) continue;
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (c0 + j < n_valid) {
              float f = __uint_as_float(v[j]);
              if (p.tw) f *= __int_as_float((min(max(twr + __ldg(p.tx + m0 + c0 + j), -126), 127) + 127) << 23);
              Y[(m0 + c0 + j) * p.ldy + n0 + q * 32 + lane] = f;
            }
        }
      } else {
        // bf16 output: drain the accumulator into registers (one weight row x 128 tokens per thread as 64 packed bf16
        // pairs), hand TMEM back, then transpose and store under the next tile's K loop
        uint32_t pk[64];
        {
          uint32_t va[16], vb[16];
          const uint32_t tbase = tmem + ((q * 32u) << 16) + 128u * grp;
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
        hand_back();
        const int g0 = 128 * (int)grp;
        // transpose through shared memory, 4 tokens at a time per group: [4 tokens][128 features] bf16, then one 8-byte
        // store per thread (a warp writes one token's 256 B).  Two-level scaling: multiplying the rounded value by the power
        // of two is the rounding of the multiplied value, so the factors go in here, after TMEM has been handed back.
        uint16_t* stg = reinterpret_cast<uint16_t*>(sm + G::SM_STG) + grp * 512u;
        __nv_bfloat16* Y = reinterpret_cast<__nv_bfloat16*>(p.Y);
#pragma unroll
        for (int c0 = 0; c0 < 128; c0 += 4) {
          if (g0 + c0 < n_valid) {                  // uniform over the four warps of the group
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              uint32_t lo = pk[c0 / 2 + j] << 16, hi = pk[c0 / 2 + j] & 0xFFFF0000u;
              if (p.tw) {
                const int t = g0 + c0 + 2 * j;
                if (t < n_valid) lo = __float_as_uint(__uint_as_float(lo) * __int_as_float((min(max(twr + __ldg(p.tx + m0 + t), -126), 127) + 127) << 23));
                if (t + 1 < n_valid) hi = __float_as_uint(__uint_as_float(hi) * __int_as_float((min(max(twr + __ldg(p.tx + m0 + t + 1), -126), 127) + 127) << 23));
              }
              stg[(2 * j) * 128 + q * 32 + lane] = (uint16_t)(lo >> 16);
              stg[(2 * j + 1) * 128 + q * 32 + lane] = (uint16_t)(hi >> 16);
            }
            ptx::named_bar_sync(1 + grp, 128);
            const uint32_t tok = et >> 5, seg = et & 31;
            if (g0 + c0 + (int)tok < n_valid) {
              const uint2 w = *reinterpret_cast<const uint2*>(stg + tok * 128 + seg * 4);
              *reinterpret_cast<uint2*>(Y + (m0 + g0 + c0 + tok) * p.ldy + n0 + seg * 4) = w;
            }
            ptx::named_bar_sync(1 + grp, 128);       // the buffer is rewritten by the next chunk
          }
        }
      }
    }
    if (!ok && lane == 0) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync();     // neither CTA leaves (or frees TMEM) while the other may still read its shared memory
  if (warp == 1) ptx::tmem_dealloc_pair(tmem, 512);
}

template <bool F32_OUT, bool B32, bool DENSE>
static cudaError_t launch_one(const LinearParams& p, int pairs, cudaStream_t stream, uint32_t* attr_mask, uint32_t bit)
{
  using G = PairGeom<B32, DENSE>;
  auto kern = sdq_linear_pair_kernel<F32_OUT, B32, DENSE>;
  if (!(*attr_mask & bit)) {     // once per device and instantiation
    const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)G::SMEM);
    if (e != cudaSuccess) return e;
    *attr_mask |= bit;
  }
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3((unsigned)(2 * pairs));
  lc.blockDim = dim3(PAIR_THREADS);
  lc.dynamicSmemBytes = G::SMEM;
  lc.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = 1;
  return cudaLaunchKernelEx(&lc, kern, p);
}

bool pair_kernel_applies(int64_t M, int64_t N, int64_t K, int out_n)
{
  // The accumulator is not double-buffered, so every tile pays for the epilogue's drain of TMEM (~1 us); tiles of fewer
  // than 32 stages (no outlier part and K <= 7936, or K < 2816 with one) run faster on the single-CTA kernel's smaller
  // tiles (measured: 4096 -> 11008 without outliers 40 against 36 us; 11008 -> 4096 without outliers 30 against 34 us).
  const int64_t stages = K / K2 + (out_n ? K / K1 : 0);
  return M > 128 && N % (2 * TILE_ROWS) == 0 && stages >= 32;
}

cudaError_t launch_linear_pair(LinearParams p, bool f32_out, int sm_count, cudaStream_t stream, uint32_t* attr_mask)
{
  const int n_mtiles = (int)((p.M + 255) / 256);
  p.total_tiles = (int)(p.N / (2 * TILE_ROWS)) * n_mtiles;
  int pairs = sm_count / 2;
  if (p.total_tiles < pairs) pairs = p.total_tiles;
  const int v = (f32_out ? 4 : 0) | (p.dense ? 2 : (p.b32 ? 1 : 0));
  switch (v) {
    case 0: return launch_one<false, false, false>(p, pairs, stream, attr_mask, 1u << 0);
    case 1: return launch_one<false, true, false>(p, pairs, stream, attr_mask, 1u << 1);
    case 2: return launch_one<false, false, true>(p, pairs, stream, attr_mask, 1u << 2);
    case 4: return launch_one<true, false, false>(p, pairs, stream, attr_mask, 1u << 4);
    case 5: return launch_one<true, true, false>(p, pairs, stream, attr_mask, 1u << 5);
    default: return launch_one<true, false, true>(p, pairs, stream, attr_mask, 1u << 6);
  }
}

}  // namespace sdq

