// Launch parameters of the fused GEMM kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "sdq_internal.h"
#include "sdq_layout.h"

namespace sdq {

struct LinearParams {
  const uint8_t* w;      // packed weights
  const uint8_t* x;      // quantized activations
  PackedOffsets poff;
  ActOffsets aoff;
  int64_t M, N, K;
  int out_n;
  int n_tile;            // tokens per tile: 16, 32, 64, 128 or 256
  int n_mtiles;          // ceil(M / n_tile)
  int total_tiles;       // (N / 128) * n_mtiles * ksplit
  int nslot, slot_bytes; // shared-memory ring geometry (depends on n_tile)
  int ring_bytes;        // nslot * slot_bytes; the transpose buffer and the barriers follow
  int release;           // 1: ring slots are reused (producer waits on `empty`, MMA issuer commits to it)
  int tmem_cols;         // TMEM columns to allocate (128, 256 or 512)
  int meta_col;          // first TMEM column of the metadata / scale buffers
  int b32;               // 1: one inlier / activation scale per 32 K (kind::mxf4nvf4 .block16), runtime geometry only
  // two-level scaling (E4M3 Q-Vector scale codes): the accumulator of row n and token m is in units of 2^(tw[n] + tx[m]);
  // the epilogue multiplies that factor back in.  tw == nullptr: not in use.
  const int32_t* tw;     // [N] exponents of the rows' inlier factors (packed weights)
  const int32_t* tx;     // [tokens] exponents of the tokens' 8-bit scales (quantized activations)
  int dense;             // 1: dense inliers (no Stage 1): 4 dense kind::mxf4 MMAs of 64 K per stage, runtime geometry only
  int ksplit;            // CTAs sharing the K range of one row tile (1 = no split)
  int cluster_ks;        // > 1: those CTAs form a cluster and reduce through distributed shared memory
  uint32_t* ws_counter;  // split-K workspace: arrival counters [row tile], zero between calls
  float* ws_partial;     // split-K workspace: fp32 partial tiles [row tile][split][token][128 rows]
  void* Y;
  int64_t ldy;
  uint32_t* flags;
};

// Grouped few-token kernel (sdq_linear_group.cu): one persistent launch over the (matrix, 128-row tile) work items of
// up to GROUP_MAX independent linear layers.
constexpr int GROUP_MAX = 32;
struct GroupMat {
  const uint8_t* w;      // packed weights
  const uint8_t* x;      // quantized activations
  void* Y;
  int64_t ldy;
  uint64_t wi, wc, sfa_out;       // sections of w: inlier stages, compact outlier stages, outlier row-scale atoms
  uint64_t xi, xo, sfb_out;       // sections of x: 4-bit stages, 8-bit stages, token-scale atom
  uint64_t wsc, xsc;              // int8 outliers: the fp32 row scales [N] of w and token scales [M] of x
  int M, T2;             // tokens, K / 256
  int item0;             // number of the matrix's first work item (= row tiles of the matrices before it)
};
struct GroupParams {
  int n, n_tile, nslot, slot_bytes, total_items;
  int out_n;             // outliers per S-Vector, the same for every matrix of the call (0 or 1)
  int out_i8;            // the outlier operands are int8 with fp32 scales (else E4M3 with power-of-two scale atoms)
  // activation-resident variant (launch_linear_group with x_bf16 set): all matrices share one bf16 X [x_M][K], which every
  // CTA quantizes into its own shared memory before it starts; GroupMat::x and its section offsets are then unused
  const void* x_bf16;
  int64_t x_ld;
  int x_M, scale_rule;
  uint32_t* flags;
  GroupMat m[GROUP_MAX];
};
cudaError_t launch_linear_group(GroupParams p, bool f32_out, int sm_count, cudaStream_t stream, uint32_t* attr_done);
bool group_xres_fits(int T2, int out_n);   // the activation-resident variant's shared-memory budget for K = 256 T2

// CTA-pair (tcgen05 cta_group::2) many-token kernel: tiles of 256 weight rows x 256 tokens (sdq_linear_pair.cu).
// `attr_mask` is the calling device's record of which instantiations already carry their shared-memory attribute.
bool pair_kernel_applies(int64_t M, int64_t N, int64_t K, int out_n);
cudaError_t launch_linear_pair(LinearParams p, bool f32_out, int sm_count, cudaStream_t stream, uint32_t* attr_mask);

}  // namespace sdq
