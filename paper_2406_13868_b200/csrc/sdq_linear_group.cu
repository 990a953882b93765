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
// section, 1.5 bits per weight) -- not as the 2:4 FP8 container of the many-token kernels (5 bits per weight): sixteen
// warps in groups of four rebuild the containers of each 256-K unit (one weight row per thread) and write them with
// tcgen05.st into tensor memory, from where the outlier MMAs take their A operand and their metadata, while the tensor
// core works on earlier units.  Shared memory carries every streamed byte once in (bulk copy) and once out (operand
// read); an earlier version that rebuilt the containers in shared memory moved 86 KB per unit through it, two thirds of
// its bandwidth at the rate aimed for, and had room for two container pairs only, whose build -> multiply -> release
// cycle set the pace.  Streamed bytes: 2.625 + 1.5 = 4.125 bits per weight against 4.0 algorithmic.
//
// The ring is organised in units of 256 K of one item: an inlier slot (the WI record with the tokens' 4-bit codes and
// scale atom) and an outlier slot (two compact records with the tokens' 8-bit codes); tensor memory holds one container
// set per ring position.  All of a unit is released by ONE tcgen05.commit per issuer.  An mbarrier test costs 15..50 cycles
// when the phase has completed, a tcgen05 instruction ~40 to issue, but a hand-over between roles (complete -> noticed)
// several hundred, so every role keeps its trips few and its waits parallel: where a role waits for several barriers,
// different lanes wait for them at the same time.
//
// Warps: 0 and 10 bulk-copy producers (inlier / outlier slots, six lanes each), 1 and 23 MMA issuers (inlier / outlier
// product, each into its own accumulator; warp-uniform loops, one elected lane issues; they also copy the inlier metadata
// and the scales to TMEM), 2..5 epilogue (adds the two accumulators; accumulator pairs alternate per item, so the next
// item's MMAs never wait for the stores), 6..9, 11..14, 15..18 and 19..22 container builders (up to four groups).
// Every wait is bounded; a timeout sets the sticky flag.
//
// Variants.  Outlier operands in int8 (SDQ_OUT_INT8): the same containers and token codes read as integers by a sparse
// kind::i8 MMA into an int32 accumulator; the epilogue converts the exact sums and applies the fp32 row and token scales.
// Activation-resident (template XRES, sdq_linear_group_x): all layers read one bf16 X of up to 16 tokens, which every CTA
// quantizes into its own shared memory (22 warps; the codes, scales and layouts of sdq_quantize_act) while its producers
// already stream weights; the ring slots then hold the weight records only.
//
// What bounds it (measured): the SM's instruction issue is half used, more than half of it by the builders' byte
// arithmetic; a CTA runs a unit in ~0.45-0.5 us against 0.38 us at the HBM peak.
#include <cuda_bf16.h>

#include "sdq_codec.cuh"
#include "sdq_internal.h"
#include "sdq_layout.h"
#include "sdq_linear.h"
#include "sdq_ptx.cuh"

namespace sdq {

constexpr int GRP_THREADS = 768;                 // 24 warps
constexpr int GRP_MAX_UNITS = 8;                 // units the ring may hold (and container sets tensor memory holds)
constexpr uint32_t GRP_TM_ACC = 0;               // per item parity 64 columns: O_i at +0, O_o at +32 (32 columns each)
constexpr uint32_t GRP_TM_I = 128;               // 2 x 12: E_in 4 | SFA_in 4 | SFB_in 4
constexpr uint32_t GRP_TM_SO = 152;              // 2 x 8: SFA_out 4 | SFB_out 4 (per item parity)
constexpr uint32_t GRP_TM_C = 168;               // per ring position 40: A_out of the unit's two 128-K stages 2 x 16 | E_out 2 x 4
constexpr uint32_t GRP_TM_C_COLS = 40;
constexpr uint32_t GRP_TMEM_COLS = 512;
constexpr int GRP_BAR_BYTES = (4 * GRP_MAX_UNITS + 4 + 2) * 8 + 8;
// activation-resident variant (16 tokens): per 256-K unit the tokens' 4-bit codes, their scale atom and the 8-bit codes of the
// unit's two 128-K stages, in the operand layouts of the quantizer's buffer; then one atom of token scales for the outlier
// product; then the quantizing warps' per-token maxima and the tokens' fp32 scales (int8 outliers)
constexpr uint32_t GRP_XU = 16 * 128 + SF_ATOM_BYTES + 2 * 16 * 128;   // 6656
constexpr int GRP_XQ_WARPS = 22;                                       // every warp but the two producers quantizes
constexpr int GRP_X_TAIL = SF_ATOM_BYTES + GRP_XQ_WARPS * 8 * 4 + 16 * 4 + 64;
__host__ __device__ inline int group_xres_bytes(int T2) { return T2 * (int)GRP_XU + GRP_X_TAIL; }

// inlier slot: | WI record | 4-bit codes of the tokens | their scale atom |
__host__ __device__ inline int group_is_bytes(int n_tile) { return WI_BYTES + n_tile * 128 + SF_ATOM_BYTES; }
// outlier slot: | two compact records (128 K each) | 8-bit codes of the tokens, 2 x 128 K |
__host__ __device__ inline int group_os_bytes(int n_tile) { return 2 * wc_bytes(1) + 2 * n_tile * 128; }
// beside the ring: alternating per item, the outlier row / token scale atoms (SFA_out | SFB_out)
constexpr int GRP_SIDE_BYTES = 2 * 2 * SF_ATOM_BYTES;

// matrix of work item `item` (items are numbered matrix by matrix)
__device__ __forceinline__ int group_mat_of(const GroupParams& p, int item) {
  int i = 0;
  while (i + 1 < p.n && item >= p.m[i + 1].item0) ++i;
  return i;
}

template <bool F32_OUT, bool XRES>
__global__ void __launch_bounds__(GRP_THREADS, 1)
sdq_linear_group_kernel(const __grid_constant__ GroupParams p)
{
  extern __shared__ uint8_t smem_raw[];
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint8_t* sm = smem_raw + ((128 - (ptx::smem_u32(smem_raw) & 127)) & 127);
  const uint32_t NU = (uint32_t)p.nslot;                                     // units in the ring
  // (activation-resident variant: the slots hold the weight records only)
  const uint32_t xb = (uint32_t)p.n_tile * 128u, isb = XRES ? (uint32_t)WI_BYTES : (uint32_t)group_is_bytes(p.n_tile);
  const uint32_t osb = p.out_n ? (XRES ? 2u * (uint32_t)wc_bytes(1) : (uint32_t)group_os_bytes(p.n_tile)) : 0u;
  const uint32_t ub = isb + osb;                                             // bytes of a unit: inlier slot, then outlier slot
  uint8_t* xres = sm + NU * ub;                                              // XRES: the quantized activations of all K
  const uint32_t xres_main = XRES ? (uint32_t)p.m[0].T2 * GRP_XU : 0u;
  uint8_t* x_sfb = xres + xres_main;                                         // XRES: token-scale atom of the outlier product
  float* x_part = reinterpret_cast<float*>(x_sfb + SF_ATOM_BYTES);           // XRES: [quantizing warp][token of its group] maxima
  float* x_sx = x_part + GRP_XQ_WARPS * 8;                                   // XRES: the tokens' fp32 scales (int8 outliers)
  uint8_t* sfbuf = xres + (XRES ? (uint32_t)group_xres_bytes(p.m[0].T2) : 0u);   // 2 x (SFA_out | SFB_out) of the item, alternating
  uint64_t* full_is = reinterpret_cast<uint64_t*>(sfbuf + (p.out_n ? GRP_SIDE_BYTES : 0));  // inlier slot of ring position v has landed
  uint64_t* full_os = full_is + GRP_MAX_UNITS;                               // outlier slot of ring position v has landed
  uint64_t* done = full_os + GRP_MAX_UNITS;                                  // the MMAs of the unit at ring position v have completed
  uint64_t* built = done + GRP_MAX_UNITS;                                    // the containers of the unit at ring position v are in tensor memory
  uint64_t* acc_full = built + GRP_MAX_UNITS;                                // [2]
  uint64_t* acc_empty = acc_full + 2;                                        // [2]
  uint64_t* sf_full = acc_empty + 2;                                         // [2] outlier scale atoms of the item have landed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sf_full + 2);
  volatile uint32_t* timed_out = tmem_slot + 1;                              // a container builder's wait gave up

  if (tid == 0) ptx::griddep_launch_dependents();
  if (tid == 0) {
    *timed_out = 0u;
    const uint32_t issuers = p.out_n ? 2u : 1u;   // MMA-issuing warps: both commit to `done` and `acc_full`
    for (uint32_t v = 0; v < NU; ++v) {
      ptx::mbar_init(&full_is[v], 1); ptx::mbar_init(&full_os[v], 1); ptx::mbar_init(&done[v], issuers); ptx::mbar_init(&built[v], 4);
    }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(&acc_full[a], issuers); ptx::mbar_init(&acc_empty[a], 4); ptx::mbar_init(&sf_full[a], 1); }
    ptx::fence_barrier_init();
  }
  if (warp == 1) ptx::tmem_alloc(tmem_slot, GRP_TMEM_COLS);
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const int first = (int)blockIdx.x, stride = (int)gridDim.x;

  if (XRES && warp != 0 && warp != 10) {
    // ---------------- activation-resident variant: every warp but the producers quantizes the shared X (up to 16 tokens x K)
    // into this CTA's shared memory, in the operand layouts and with the arithmetic of sdq_quantize_act (Section 5, Stage 3:
    // A_i as E2M1 with one scale per 64 K, A_o as E4M3 or int8 per token), while the producers already stream the first
    // weights.  A warp takes a group of 8 tokens and every 11th Q-Vector, 4 lanes per token as in the quantizer.
    ptx::griddep_wait();                         // X comes from an earlier kernel
    const uint32_t qw = warp - (warp > 10 ? 2u : 1u);      // 0..21
    const uint32_t tg = qw & 1u, t = lane >> 2, l = lane & 3;
    const uint32_t mtok = tg * 8 + t;
    const bool live = (int)mtok < p.x_M;
    const __nv_bfloat16* xrow = reinterpret_cast<const __nv_bfloat16*>(p.x_bf16) + (int64_t)mtok * p.x_ld;
    const int NB = p.m[0].T2 * 4;                // Q-Vectors of 64 per token
    // one read of X: a lane keeps its (up to six) 16-element pieces in registers across the maxima's barrier
    constexpr int XT = 6;                        // Q-Vectors per warp: K <= 4096 -> 64 / 11
    uint4 raw[XT][2];
    uint32_t qmax[XT];
    uint32_t m2 = 0;
#pragma unroll
    for (int i = 0; i < XT; ++i) {
      const int b = (int)(qw >> 1) + i * (GRP_XQ_WARPS / 2);
      raw[i][0] = raw[i][1] = make_uint4(0, 0, 0, 0);
      if (live && b < NB) {
        const uint4* src = reinterpret_cast<const uint4*>(xrow + (int64_t)b * 64 + l * 16);
        raw[i][0] = __ldg(src);
        raw[i][1] = __ldg(src + 1);
      }
    }
#pragma unroll
    for (int i = 0; i < XT; ++i) {
      const uint32_t r[8] = {raw[i][0].x, raw[i][0].y, raw[i][0].z, raw[i][0].w, raw[i][1].x, raw[i][1].y, raw[i][1].z, raw[i][1].w};
      uint32_t q = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) q = __vmaxu2(q, r[j] & 0x7FFF7FFFu);
      q = max(q & 0xFFFFu, q >> 16);             // > 0x7F7F: the lane holds an infinity (counts as the largest finite bf16)
      qmax[i] = q;
      m2 = max(m2, min(q, 0x7F7Fu));
    }
    float amax = __uint_as_float(m2 << 16);
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
    if (l == 0) x_part[qw * 8 + t] = amax;
    ptx::named_bar_sync(8, GRP_XQ_WARPS * 32);
    float ramax = 0.0f;
    for (uint32_t q2 = 0; q2 < GRP_XQ_WARPS / 2; ++q2) ramax = fmaxf(ramax, x_part[(2 * q2 + tg) * 8 + t]);
    const int e = fp8_scale_exp(ramax);
    const float s8 = pow2_neg(e), sx = int8_scale(ramax);
    const bool i8 = p.out_i8 != 0;
    if (qw < 2 && l == 0) {
      x_sx[mtok] = sx;
      *reinterpret_cast<uint32_t*>(x_sfb + sf_off(mtok, 0)) = (uint32_t)((i8 || !live) ? 127 : e + 127) * 0x01010101u;
    }
#pragma unroll
    for (int i = 0; i < XT; ++i) {
      const int b = (int)(qw >> 1) + i * (GRP_XQ_WARPS / 2);     // uniform over the warp
      if (b >= NB) break;
      const uint32_t r[8] = {raw[i][0].x, raw[i][0].y, raw[i][0].z, raw[i][0].w, raw[i][1].x, raw[i][1].y, raw[i][1].z, raw[i][1].w};
      float v[16];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        v[2 * j] = __uint_as_float(r[j] << 16);
        v[2 * j + 1] = __uint_as_float(r[j] & 0xFFFF0000u);
      }
      if (qmax[i] > 0x7F7Fu) {
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = sat(v[j]);
      }
      uint32_t bm = min(qmax[i], 0x7F7Fu);
      bm = max(bm, __shfl_xor_sync(0xffffffffu, bm, 1));
      bm = max(bm, __shfl_xor_sync(0xffffffffu, bm, 2));
      const uint32_t c = e8m0_scale_code(__uint_as_float(bm << 16), p.scale_rule);
      const float s4 = pow2_inv_e8m0(c);
      uint32_t q4[2] = {0, 0}, q8[4] = {0, 0, 0, 0};
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        q4[j >> 2] |= e2m1x2(v[2 * j] * s4, v[2 * j + 1] * s4) << (8 * (j & 3));
        q8[j >> 1] |= (i8 ? (int8_code(v[2 * j], sx) | (int8_code(v[2 * j + 1], sx) << 8)) : e4m3x2(v[2 * j] * s8, v[2 * j + 1] * s8)) << (16 * (j & 1));
      }
      const uint32_t k = (uint32_t)b * 64 + l * 16;          // first element of this lane
      uint8_t* xu = xres + (size_t)(k >> 8) * GRP_XU;
      *reinterpret_cast<uint2*>(xu + b_off(mtok, (k & 255) >> 1)) = make_uint2(q4[0], q4[1]);
      *reinterpret_cast<uint4*>(xu + 16 * 128 + SF_ATOM_BYTES + ((k >> 7) & 1) * 16 * 128 + b_off(mtok, k & 127)) = make_uint4(q8[0], q8[1], q8[2], q8[3]);
      if (l == 0) xu[16 * 128 + in_sf_off(false, mtok, (uint32_t)(b & 3))] = (uint8_t)c;
    }
    ptx::fence_proxy_async();                    // generic-proxy writes -> visible to the tensor core's operand reads
    ptx::named_bar_sync(8, GRP_XQ_WARPS * 32);
  }

  if (warp == 0 || warp == 10) {
    // ---------------- producers: warp 0 fills the inlier slots, warp 10 the outlier slots.  Six lanes each, in lockstep: lane
    // 2 c + l issues copy c (of three) of the units u = l, l + 2, ... of this CTA's sequence (NU is even, so a lane's ring
    // positions keep its parity) -- issuing a bulk copy costs its thread ~100 ns, so one instruction issues a copy for
    // each of the six lanes instead of one thread issuing six in a row.
    const bool outl = warp == 10;
    const uint32_t l = lane & 1, c = lane >> 1;
    // (activation-resident variant: one copy per inlier slot; per outlier slot the compact records, and lane c = 1 the row-scale
    // atom of each item)
    if (c < (XRES ? (outl ? 2u : 1u) : 3u) && (!outl || p.out_n)) {
      if (!XRES) ptx::griddep_wait();            // activations come from an earlier kernel
      bool ok = true;
      int item = first, k2 = (int)l;             // this lane's position: work item and 256-K unit inside the item
      int mat = -1, rt = 0, T2 = 0;
      uint32_t iseq = 0;                         // number of the item in this CTA's sequence
      uint32_t v = l, wrapped = 0, ph = 0;       // ring position, whether the ring has wrapped, parity of `done` to wait for
      const uint32_t wcb = 2u * (uint32_t)wc_bytes(1);
      for (;;) {
        for (;;) {                               // advance to the item that holds unit k2
          if (item >= p.total_items) break;
          if (mat < 0) { mat = group_mat_of(p, item); rt = item - p.m[mat].item0; T2 = p.m[mat].T2; }
          if (k2 < T2) break;
          k2 -= T2; item += stride; mat = -1; ++iseq;
        }
        if (item >= p.total_items) break;
        const GroupMat& m = p.m[mat];
        if (wrapped && !(ok = ptx::mbar_wait(&done[v], ph ^ 1))) break;
        uint8_t* st = sm + (size_t)v * ub + (outl ? isb : 0u);
        if (XRES) {
          if (!outl) {
            ptx::mbar_expect_tx(&full_is[v], WI_BYTES);
            ptx::bulk_g2s(st, m.w + m.wi + ((size_t)rt * m.T2 + k2) * WI_BYTES, WI_BYTES, &full_is[v]);
          } else if (c == 0) {
            ptx::mbar_expect_tx(&full_os[v], wcb);
            ptx::bulk_g2s(st, m.w + m.wc + ((size_t)rt * 2 * m.T2 + 2 * k2) * (size_t)wc_bytes(1), wcb, &full_os[v]);
          } else if (k2 == 0 && !p.out_i8) {     // the item's row-scale atom (see below); the tokens' atom is resident
            const uint32_t sb = iseq & 1;
            if (iseq >= 2 && !(ok = ptx::mbar_wait(&acc_full[sb], ((iseq >> 1) - 1) & 1))) break;
            ptx::mbar_expect_tx(&sf_full[sb], SF_ATOM_BYTES);
            ptx::bulk_g2s(sfbuf + sb * 2 * SF_ATOM_BYTES, m.w + m.sfa_out + (size_t)rt * SF_ATOM_BYTES, SF_ATOM_BYTES, &sf_full[sb]);
          }
        } else if (!outl) {
          const uint8_t* xi = m.x + m.xi + (size_t)k2 * XI_BYTES;
          if (c == 0) ptx::mbar_expect_tx(&full_is[v], WI_BYTES + xb + SF_ATOM_BYTES);
          const uint8_t* src = c == 0 ? m.w + m.wi + ((size_t)rt * m.T2 + k2) * WI_BYTES : (c == 1 ? xi : xi + B4_BYTES);
          const uint32_t off = c == 0 ? 0u : (c == 1 ? (uint32_t)WI_BYTES : (uint32_t)WI_BYTES + xb);
          ptx::bulk_g2s(st + off, src, c == 0 ? (uint32_t)WI_BYTES : (c == 1 ? xb : (uint32_t)SF_ATOM_BYTES), &full_is[v]);
        } else {
          const uint8_t* xo = m.x + m.xo + (size_t)(2 * k2) * XO_BYTES;
          if (c == 0) ptx::mbar_expect_tx(&full_os[v], wcb + 2 * xb);
          const uint8_t* src = c == 0 ? m.w + m.wc + ((size_t)rt * 2 * m.T2 + 2 * k2) * (size_t)wc_bytes(1) : (c == 1 ? xo : xo + XO_BYTES);
          ptx::bulk_g2s(st + (c == 0 ? 0u : wcb + (c - 1) * xb), src, c == 0 ? wcb : xb, &full_os[v]);
          if (k2 == 0 && c >= 1 && !p.out_i8) {     // (int8 outliers take fp32 scales in the epilogue: no scale atoms)
            // the item's outlier scale atoms (lane c = 1: of the weight rows, c = 2: of the tokens): a buffer and a barrier
            // of their own per item parity.  The buffer is free once every MMA of the item two back has completed (`acc_full`
            // of that item: it cannot complete again before these atoms land, since the next item on that accumulator needs
            // them) -- the ring alone does not say so when an item has fewer units than half the ring.
            const uint32_t sb = iseq & 1;
            if (iseq >= 2 && !(ok = ptx::mbar_wait(&acc_full[sb], ((iseq >> 1) - 1) & 1))) break;
            uint8_t* sf = sfbuf + sb * 2 * SF_ATOM_BYTES;
            if (c == 1) ptx::mbar_expect_tx(&sf_full[sb], 2u * SF_ATOM_BYTES);
            ptx::bulk_g2s(sf + (c - 1) * SF_ATOM_BYTES, c == 1 ? m.w + m.sfa_out + (size_t)rt * SF_ATOM_BYTES : m.x + m.sfb_out, SF_ATOM_BYTES,
                          &sf_full[sb]);
          }
        }
        k2 += 2;
        v += 2;
        if (v >= NU) { v -= NU; wrapped = 1; ph ^= 1; }
      }
      if (!ok) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
    }
  } else if (warp == 1 || warp == 23) {
    // ---------------- MMA issuers: warp 1 the inlier product O_i, warp 23 the outlier product O_o, each into its own
    // accumulator (the epilogue adds them: O = O_i + O_o) -- a tcgen05 instruction costs its issuing thread ~45 cycles, and
    // all of a 256-K unit's in one thread were the longest serial piece of the kernel.  Warp-uniform loops, one elected
    // lane issues (descriptors and TMEM addresses are uniform-register operands).  tcgen05.cp and tcgen05.mma of one
    // thread execute in issue order, so the inlier metadata and the scales need no barrier of their own; their TMEM buffers
    // alternate.  The outlier product takes its A operand and metadata from tensor memory, where the builders put them.
    // The unit is released when both warps' commits have arrived.
    const bool outw = warp == 23;
    if (!outw || p.out_n) {
      bool ok = true;
      const uint32_t smb = ptx::smem_u32(sm);
      const uint32_t id4[2] = {ptx::idesc_block_scaled(128, (uint32_t)p.n_tile, 1, true, 0, 0), ptx::idesc_block_scaled(128, (uint32_t)p.n_tile, 1, true, 2, 2)};
      const uint32_t id8 = p.out_i8 ? ptx::idesc_i8(128, (uint32_t)p.n_tile, true) : ptx::idesc_block_scaled(128, (uint32_t)p.n_tile, 0, true, 0, 0);
      const uint32_t wcb = 2u * (uint32_t)wc_bytes(1);
      uint32_t v = 0, ph = 0, itc = 0;             // ring position and its lap parity, item count
      for (int item = first; item < p.total_items && ok; item += stride, ++itc) {
        const int T2 = p.m[group_mat_of(p, item)].T2;
        const uint32_t ab = itc & 1, acc_col = tmem + GRP_TM_ACC + 64u * ab + (outw ? 32u : 0u), so = tmem + GRP_TM_SO + 8u * ab;
        if (itc >= 2) {    // the epilogue has read this accumulator pair's previous item
          ok = __all_sync(0xffffffffu, ptx::mbar_wait(&acc_empty[ab], ((itc >> 1) - 1) & 1));
          if (!ok) break;
        }
        for (int k2 = 0; k2 < T2 && ok;) {
          // Up to four units of the item per trip: lane i tests unit k2 + i (for the outlier product: its containers are in
          // tensor memory, which implies that its slot has landed -- the builders waited for that), lane 4 the item's scale
          // atoms; the units ready in a row from k2 on are issued together.  A trip costs several hundred cycles beside the
          // instructions it issues (test, vote, fence, election, reconvergence), so taking what is ready in one trip keeps
          // the issuer ahead whenever it has fallen behind.  With nothing ready it waits for unit k2 and votes again.
          const int nb = T2 - k2 < 4 ? T2 - k2 : 4;
          uint32_t vi = v + lane, phi = ph;
          if (vi >= NU) { vi -= NU; phi ^= 1; }
          const bool sf_lane = outw && k2 == 0 && lane == 4 && !p.out_i8;
          uint64_t* bar = sf_lane ? &sf_full[ab] : (outw ? &built[vi < NU ? vi : 0] : &full_is[vi < NU ? vi : 0]);
          const uint32_t par = sf_lane ? ((itc >> 1) & 1) : phi;
          const bool mine = (int)lane < nb || sf_lane;
          const uint32_t ready = __ballot_sync(0xffffffffu, mine ? ptx::mbar_test(bar, par) : (lane == 4));
          int n = __ffs((int)~ready) - 1;          // units ready in a row (lane 4 votes yes when it has nothing to test)
          if (n > nb) n = nb;
          if (!(ready & 16u)) n = 0;
          if (n == 0) {
            ok = __all_sync(0xffffffffu, (lane == 0 || sf_lane) ? ptx::mbar_wait(bar, par) : true);
            continue;
          }
          ptx::tc_fence_after();
          if (ptx::elect_one()) {
            uint32_t vv = v;
            for (int i = 0; i < n; ++i) {
              const int kk = k2 + i;
              const uint32_t sb = smb + vv * ub;
              // the tokens' operands of unit kk: in the slot behind the weight records, or resident
              const uint32_t xu = ptx::smem_u32(xres) + (uint32_t)kk * GRP_XU;
              const uint32_t b4 = XRES ? xu : sb + WI_BYTES, sf4 = XRES ? xu + 16 * 128 : sb + WI_BYTES + xb;
              if (!outw) {
                const uint32_t mb = tmem + GRP_TM_I + 12u * (uint32_t)(kk & 1);
                ptx::tc_cp_128x128b(mb, ptx::smem_desc(sb + A_IN_BYTES, 0, 128));
                ptx::tc_cp_32x128b_warpx4(mb + 4, ptx::smem_desc(sb + A_IN_BYTES + E_IN_BYTES, 0, 128));
                ptx::tc_cp_32x128b_warpx4(mb + 8, ptx::smem_desc(sf4, 0, 128));
                ptx::mma_sp_mxf4(acc_col, ptx::smem_desc(sb, 128, 256), ptx::smem_desc(b4, 128, 1024), id4[0], mb, mb + 4, mb + 8,
                                 kk ? 1u : 0u);
                ptx::mma_sp_mxf4(acc_col, ptx::smem_desc(sb + 4096, 128, 256), ptx::smem_desc(b4 + 512, 128, 1024), id4[1], mb + 2,
                                 mb + 4, mb + 8, 1u);
              } else {
                if (kk == 0 && !p.out_i8) {
                  const uint32_t sf = ptx::smem_u32(sfbuf) + ab * 2 * SF_ATOM_BYTES;
                  ptx::tc_cp_32x128b_warpx4(so, ptx::smem_desc(sf, 0, 128));
                  ptx::tc_cp_32x128b_warpx4(so + 4, ptx::smem_desc(XRES ? ptx::smem_u32(x_sfb) : sf + SF_ATOM_BYTES, 0, 128));
                }
#pragma unroll
                for (uint32_t h = 0; h < 2; ++h) {
                  const uint32_t ca = tmem + GRP_TM_C + GRP_TM_C_COLS * vv + 16u * h, eb = tmem + GRP_TM_C + GRP_TM_C_COLS * vv + 32u + 4u * h;
                  const uint32_t xa = XRES ? xu + 16 * 128 + SF_ATOM_BYTES + h * 16 * 128 : sb + isb + wcb + h * xb;
                  if (p.out_i8) {     // the same containers and token codes as integers, int32 accumulator
                    ptx::mma_sp_i8_ta(acc_col, ca, ptx::smem_desc(xa, 128, 1024), id8, eb, (kk | (int)h) ? 1u : 0u);
                    ptx::mma_sp_i8_ta(acc_col, ca + 8, ptx::smem_desc(xa + 512, 128, 1024), id8, eb + 2, 1u);
                  } else {
                    ptx::mma_sp_mxf8_ta(acc_col, ca, ptx::smem_desc(xa, 128, 1024), id8, eb, so, so + 4, (kk | (int)h) ? 1u : 0u);
                    ptx::mma_sp_mxf8_ta(acc_col, ca + 8, ptx::smem_desc(xa + 512, 128, 1024), id8, eb + 2, so, so + 4, 1u);
                  }
                }
              }
              ptx::tc_commit(&done[vv]);
              if (kk == T2 - 1) ptx::tc_commit(&acc_full[ab]);
              if (++vv == NU) vv = 0;
            }
          }
          __syncwarp();
          k2 += n;
          v += (uint32_t)n;
          if (v >= NU) { v -= NU; ph ^= 1; }
        }
      }
      if (!ok && lane == 0) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
    }
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
      // one thread polls the barrier and releases the other 127 through a hardware barrier: many threads polling an mbarrier
      // slow every other barrier operation of the CTA down
      if (warp == 2 && lane == 0 && !ptx::mbar_wait(&acc_full[ab], (itc >> 1) & 1)) *timed_out = 1u;
      ptx::named_bar_sync(3, 128);
      if (*timed_out) { ok = false; break; }
      ptx::tc_fence_after();
      // int8 outliers: O_o = s_w[row] s_x[token] (exact int32 sum of code products); this thread's row scale
      const float sw = p.out_i8 ? __ldg(reinterpret_cast<const float*>(m.w + m.wsc) + n0 + qd * 32 + lane) : 0.0f;
      const float* sxp = reinterpret_cast<const float*>(m.x + m.xsc);
      uint32_t val[32];
      {
        // O = O_i + O_o: the two partial products of the item, added in fp32
        uint32_t a[16], b[16];
        const uint32_t tb = tmem + ((qd * 32u) << 16) + GRP_TM_ACC + 64u * ab;
#pragma unroll
        for (uint32_t c = 0; c < 32; c += 16) {
          if (c < (uint32_t)p.n_tile) {
            ptx::tmem_ld_32x32b_x16(tb + c, a);
            if (p.out_n) ptx::tmem_ld_32x32b_x16(tb + 32 + c, b);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 16; ++i) val[c + i] = p.out_n ? __float_as_uint(__uint_as_float(a[i]) + __uint_as_float(b[i])) : a[i];
            if (p.out_i8) {      // b holds exact int32 sums: scale them, tokens that exist only
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                const float o = (int)(c + i) < m.M ? (float)(int)b[i] * (sw * (XRES ? x_sx[c + i] : __ldg(sxp + c + i))) : 0.0f;
                val[c + i] = __float_as_uint(__uint_as_float(a[i]) + o);
              }
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) val[c + i] = 0u;
          }
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&acc_empty[ab]);
#pragma unroll
      for (int t = 0; t < 32; ++t) {
        if (t < m.M) {
          const int64_t idx = (int64_t)t * m.ldy + n0 + qd * 32 + lane;
          if (F32_OUT) reinterpret_cast<float*>(m.Y)[idx] = __uint_as_float(val[t]);
          else reinterpret_cast<__nv_bfloat16*>(m.Y)[idx] = __float2bfloat16_rn(__uint_as_float(val[t]));
        }
      }
    }
    if (!ok && lane == 0) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
  } else if (p.out_n && warp >= 6 && warp <= 22) {
    // ---------------- outlier container builders: up to four groups of four warps (6..9, 11..14, 15..18, 19..22); group g
    // rebuilds the containers of the units u = g, g + G, ... -- straight into tensor memory, where the outlier MMAs read their
    // A operand and metadata: shared memory is written once (by the bulk copies) and never again.  A warp can reach the 32
    // TMEM lanes 32 (warp % 4) .., so its thread `lane` rebuilds weight row 32 (warp % 4) + lane, both 128-K stages of the
    // unit, each from 16 codes + 16 positions: per S-Vector of 8 the code goes to the 2:4 slot of its group of 4 (two
    // ascending slot indices per 4: (p, 3) with the value first, or (0, 3) with the value second when p = 3; a group without
    // outlier gets (0, 1) and zeros), the form the packer writes for the many-token kernels.  A row's 64 stored bytes per
    // stage are 16 columns of its lane, its 16 metadata bytes 4 columns.  Several groups, because a trip is mostly latency
    // (measured ~1800 cycles, a tenth of it arithmetic): they overlap in time.  G divides the ring, so that every phase of
    // a slot's barrier is seen by the same group.  Container set v is free when the unit's outlier slot has landed at ring
    // position v: the producer refills a position only after the MMAs of its previous unit have completed.
    const uint32_t bw = warp - (warp >= 11 ? 7u : 6u);       // 0..15
    const uint32_t grp = bw >> 2;
    const uint32_t G = (NU & 3u) == 0 ? 4u : (NU % 3u == 0 ? 3u : 2u);
    const uint32_t r = (warp & 3) * 32 + lane;
    const bool poller = (bw & 3u) == 0;
    bool ok = true;
    uint32_t v = 0, ph = 0, gu = 0;              // position of the unit in the ring, lap parity, unit count modulo G
    const uint32_t tlane = tmem + (((warp & 3) * 32u) << 16) + GRP_TM_C;
    for (int item = first; item < p.total_items && ok && grp < G; item += stride) {
      const int T2 = p.m[group_mat_of(p, item)].T2;
      for (int k2 = 0; k2 < T2; ++k2) {
        if (gu == grp) {
          // Only ONE thread of the group waits on the mbarrier and then releases the others through a hardware barrier: with
          // every warp waiting on the same mbarrier some of them noticed its completion more than a microsecond late.
          if (poller && lane == 0 && !ptx::mbar_wait(&full_os[v], ph)) *timed_out = 1u;
          ptx::named_bar_sync(4 + grp, 128);   // (barrier 3 belongs to the epilogue)
          if (*timed_out) { ok = false; break; }
          const uint8_t* st = sm + (size_t)v * ub + isb;
          const uint32_t tc = tlane + GRP_TM_C_COLS * v;
#pragma unroll
          for (uint32_t h = 0; h < 2; ++h) {
            const uint4 codes = *reinterpret_cast<const uint4*>(st + h * (uint32_t)wc_bytes(1) + r * 16);
            const uint2 pos = *reinterpret_cast<const uint2*>(st + h * (uint32_t)wc_bytes(1) + WC_CODE_BYTES + r * 8);
            const uint32_t cw[4] = {codes.x, codes.y, codes.z, codes.w}, pw[2] = {pos.x, pos.y};
            // position ps (0..7) of the outlier in its S-Vector: it sits in the group of 4 number ps >> 2 at p = ps & 3.  Stored
            // bytes of the S-Vector (two per group of 4): the code moves to byte (p == 3) + 2 (ps >> 2); metadata byte = the two
            // groups' slot-index nibbles, (p, 3) or (0, 3) for p = 3 where the outlier is, (0, 1) elsewhere.  Both come from
            // 8-entry byte tables held in two registers each, and one byte-permute looks up four S-Vectors at a time: the four
            // position nibbles of a 16-bit piece of the position word are its selector.
            uint32_t stored[16], meta[4], shw[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const uint32_t sel = pw[i >> 1] >> (16 * (i & 1));
              meta[i] = __byte_perm(0x4C4E4D4Cu, 0xC4E4D4C4u, sel);
              shw[i] = __byte_perm(0x08000000u, 0x18101010u, sel);
            }
#pragma unroll
            for (int g = 0; g < 16; ++g)
              stored[g] = __funnelshift_l(0u, __byte_perm(cw[g >> 2], 0u, 0x4440u + (uint32_t)(g & 3)), shw[g >> 2] >> (8 * (g & 3)));   // (shift count mod 32: the byte's 0 / 8 / 16 / 24)
            // columns 0..7 of the stage: the row's stored bytes of K-block 0 (the first MMA's A), 8..15: of K-block 1
            ptx::tmem_st_32x32b_x16(tc + 16u * h, stored);
            ptx::tmem_st_32x32b_x4(tc + 32u + 4u * h, meta);
          }
          ptx::tmem_st_wait();
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&built[v]);      // one arrival per warp
        }
        if (++gu == G) gu = 0;
        if (++v == NU) { v = 0; ph ^= 1; }
      }
    }
    if (!ok && lane == 0) atomicOr(&p.flags[FLAG_TIMEOUT], 1u);
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) ptx::tmem_dealloc(tmem, GRP_TMEM_COLS);
}

// units the ring holds for `n_tile` tokens per tile: as many as fit (an even number)
static int group_units(int n_tile, int out_n, int xres_bytes, int unit_bytes) {
  const int avail = 232448 - 128 - (out_n ? GRP_SIDE_BYTES : 0) - GRP_BAR_BYTES - xres_bytes;
  int n = avail / unit_bytes;
  n &= ~1;
  return n > GRP_MAX_UNITS ? GRP_MAX_UNITS : n;
}

// shared-memory budget of the activation-resident variant: does a ring of at least six units fit beside X of K / 256 = T2 units?
bool group_xres_fits(int T2, int out_n) {
  const int unit = WI_BYTES + (out_n ? 2 * wc_bytes(1) : 0);
  return group_units(16, out_n, group_xres_bytes(T2), unit) >= 6;
}

cudaError_t launch_linear_group(GroupParams p, bool f32_out, int sm_count, cudaStream_t stream, uint32_t* attr_done)
{
  const bool xres = p.x_bf16 != nullptr;
  const int xbytes = xres ? group_xres_bytes(p.m[0].T2) : 0;
  p.slot_bytes = xres ? WI_BYTES + (p.out_n ? 2 * wc_bytes(1) : 0) : group_is_bytes(p.n_tile) + (p.out_n ? group_os_bytes(p.n_tile) : 0);
  p.nslot = group_units(p.n_tile, p.out_n, xbytes, p.slot_bytes);
  const int smem = p.nslot * p.slot_bytes + xbytes + (p.out_n ? GRP_SIDE_BYTES : 0) + GRP_BAR_BYTES + 128;
  if (!*attr_done) {
    const cudaFuncAttribute a = cudaFuncAttributeMaxDynamicSharedMemorySize;
    if (cudaFuncSetAttribute(sdq_linear_group_kernel<false, false>, a, 232448) != cudaSuccess ||
        cudaFuncSetAttribute(sdq_linear_group_kernel<true, false>, a, 232448) != cudaSuccess ||
        cudaFuncSetAttribute(sdq_linear_group_kernel<false, true>, a, 232448) != cudaSuccess ||
        cudaFuncSetAttribute(sdq_linear_group_kernel<true, true>, a, 232448) != cudaSuccess)
      return cudaErrorUnknown;
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
  if (xres) return f32_out ? cudaLaunchKernelEx(&lc, sdq_linear_group_kernel<true, true>, p) : cudaLaunchKernelEx(&lc, sdq_linear_group_kernel<false, true>, p);
  return f32_out ? cudaLaunchKernelEx(&lc, sdq_linear_group_kernel<true, false>, p) : cudaLaunchKernelEx(&lc, sdq_linear_group_kernel<false, false>, p);
}

}  // namespace sdq
