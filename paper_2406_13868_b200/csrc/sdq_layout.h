// Tiled device layouts shared by the packer, the activation quantizer, the exporters and the GEMM.
//
// Everything the GEMM streams is stored so that one contiguous byte range IS the shared-memory image
// of one pipeline stage: operands sit in the un-swizzled K-major "core matrix" form the tcgen05
// shared-memory descriptors address (8 rows x 16 bytes = 128 contiguous bytes per core matrix, the
// core matrices of one 8-row group adjacent along K), so a plain bulk copy (cp.async.bulk) brings a
// stage in and no tensor map or swizzle is involved.  Keeping the K-adjacent core matrices of a row
// group contiguous (LBO = 128) matters: the tensor core then fetches 256 consecutive bytes per row
// group per instruction instead of two 128-byte pieces that collide on the same banks.
//
// Weight buffer (per 128-row tile rt; T2 = K/256 inlier stages k2, T1 = K/128 outlier stages k1)
//   section WI[rt][k2] = | A_in 8192 | E_in 2048 | SFA_in 512 |                         (10752 B)
//     A_in : two K-blocks j (128 logical K each) of 128 rows x 32 B (64 kept E2M1 codes, low nibble =
//            lower k): byte(j, row r, b) at j*4096 + (r/8)*256 + (b/16)*128 + (r%8)*16 + b%16
//     E_in : 128 rows x 16 B  (one 4-bit pair-index pair per 8 logical K over 256 K)
//     SFA_in: 4 E8M0 scales (one per 64 K) of 128 rows: byte(r, s) at (r%32)*16 + (r/32)*4 + s
//             (one scale per 32 K: two such atoms, one per 128-K block, 4 scales each; the record is 11264 B)
//   no pruning (dense inliers, one scale per 32 K): WI[rt][k2] = | A_in 16384 | SFA_in 2 x 512 |   (17408 B)
//     A_in : four K-blocks j (64 K each) of 128 rows x 32 B (all 64 E2M1 codes; outlier positions hold +0), same
//            addressing; no E_in
//   section WO[rt][k1] = | A_out 8192 | E_out 2048 |                                     (10240 B)
//     A_out: two K-blocks j (64 logical K each) of 128 rows x 32 B (stored E4M3 bytes of the 2:4
//            embedding of the 1:8 / 2:8 outliers), same addressing as A_in
//     E_out: 128 rows x 16 B  (one 4-bit index pair per 4 logical K over 128 K)
//   section SFA_out[rt]: 512 B, the per-row outlier scale as an E8M0 code, scale-atom form, 4 copies
//   section WC[rt][k1] = | codes 128 rows x 16 out_n B | positions 128 rows x 8 out_n B |   (3072 out_n B)
//     the outliers in the form the method states them (one 8-bit code + one 3-bit position per S-Vector of 8 and
//     outlier, 12 of the 11 algorithmic bits): row r, S-Vector g (0..15 inside the 128-K stage), outlier t: code byte at
//     r * 16 out_n + g * out_n + t; position (0..7) in nibble (g * out_n + t) & 1 of byte
//     2048 out_n + r * 8 out_n + (g * out_n + t) / 2.  Few-token calls stream this section instead of WO and rebuild
//     the 2:4 form in shared memory; the exporter reads it.
//   sections row scale exponents [N] i32, inlier row-factor exponents [N] i32 (two-level scaling with E4M3 Q-Vector
//   scales; zeros otherwise); element-wise 2:4 inliers with one scale per 32 K are stored like dense inliers, plus their
//   kept indices [N][K/4] u8 for the exporter
//
// Activation buffer (per 128-token tile mt)
//   section XI[mt][k2] = | B4 16384 | SFB_in 512 |            (one scale per 32 K: SFB_in 2 x 512, as for the weights)
//     B4: 128 tokens x 128 B (256 K): byte(t, b) at (t/8)*1024 + (b/16)*128 + (t%8)*16 + b%16
//   section XO[mt][k1] = | B8 16384 |
//     B8: 128 tokens x 128 B (128 K): same addressing
//   section SFB_out[mt] 512 B (per-token 8-bit scale as E8M0, 4 copies), then exponents [MT*128] i32
#pragma once
#include <stdint.h>
#include <stddef.h>

namespace sdq {

constexpr int TILE_ROWS = 128;     // weight rows per tile (= MMA M)
constexpr int TILE_TOK = 128;      // tokens per activation tile
constexpr int K1 = 128;            // logical K per pipeline stage
constexpr int K2 = 256;            // logical K per metadata / scale atom

constexpr int A_IN_BYTES = 8192;      // per 256 K
constexpr int E_IN_BYTES = 2048;
constexpr int SF_ATOM_BYTES = 512;
constexpr int WI_BYTES = A_IN_BYTES + E_IN_BYTES + SF_ATOM_BYTES;   // 10752
constexpr int A_OUT_BYTES = 8192;     // per 128 K
constexpr int E_OUT_BYTES = 2048;
constexpr int WO_BYTES = A_OUT_BYTES + E_OUT_BYTES;                  // 10240
constexpr int WC_CODE_BYTES = 2048;   // per 128 K and outlier of the S-Vector: 128 rows x 16 code bytes
constexpr int WC_POS_BYTES = 1024;    //                                        128 rows x 16 position nibbles
__host__ __device__ inline int wc_bytes(int out_n) { return (WC_CODE_BYTES + WC_POS_BYTES) * out_n; }
constexpr int B4_BYTES = 16384;       // 128 tokens x 256 K
constexpr int XI_BYTES = B4_BYTES + SF_ATOM_BYTES;                   // 16896
constexpr int B8_BYTES = 16384;       // 128 tokens x 128 K
constexpr int XO_BYTES = B8_BYTES;
// One scale per 32 logical K (in_block = 32, run by kind::mxf4nvf4 .block16) doubles the scale atoms of the inlier
// records: one atom per 128-K block (4 scales of 32 K each) instead of one per 256 K (4 scales of 64 K each).
__host__ __device__ inline int sf_atoms(bool b32) { return b32 ? 2 : 1; }
// dense inliers (no Stage 1): twice the codes, no pattern metadata
__host__ __device__ inline int a_in_bytes(bool dense) { return dense ? 2 * A_IN_BYTES : A_IN_BYTES; }
__host__ __device__ inline int e_in_bytes(bool dense) { return dense ? 0 : E_IN_BYTES; }
__host__ __device__ inline int wi_bytes(bool b32, bool dense = false) {
  return a_in_bytes(dense) + e_in_bytes(dense) + sf_atoms(b32) * SF_ATOM_BYTES;
}
__host__ __device__ inline int xi_bytes(bool b32) { return B4_BYTES + sf_atoms(b32) * SF_ATOM_BYTES; }
// byte of the inlier scale of scale block `blk` (counted inside its 256-K record) of row / token `row` inside the
// record's scale atoms: block 64 -> atom 0, slot blk (0..3); block 32 -> atom blk / 4, slot blk % 4
__host__ __device__ inline uint32_t in_sf_off(bool b32, uint32_t row, uint32_t blk) {
  return (b32 ? (blk >> 2) * SF_ATOM_BYTES : 0u) + (row & 31) * 16 + (row >> 5) * 4 + (blk & 3);
}

// byte offset inside an operand block of K-blocks of `kb_bytes` whose rows carry `row_bytes` per K-block
//   A operands: row_bytes 32, kb_bytes 4096 (LBO 128, SBO 256);  B operands: one block, row_bytes 128 (SBO 1024)
__host__ __device__ inline uint32_t a_off(uint32_t row, uint32_t byte /*0..63; dense inliers 0..127*/) {
  const uint32_t j = byte >> 5, b = byte & 31;
  return j * 4096 + (row >> 3) * 256 + (b >> 4) * 128 + (row & 7) * 16 + (b & 15);
}
__host__ __device__ inline uint32_t b_off(uint32_t tok, uint32_t byte /*0..127*/) {
  return (tok >> 3) * 1024 + (byte >> 4) * 128 + (tok & 7) * 16 + (byte & 15);
}
__host__ __device__ inline uint32_t sf_off(uint32_t row, uint32_t s) { return (row & 31) * 16 + (row >> 5) * 4 + s; }

constexpr size_t HEADER_BYTES = 256;
// What the first HEADER_BYTES of a packed buffer hold (the rest of the 256 bytes is zero): enough to rebuild the host
// descriptor from the bytes alone.
constexpr uint64_t BLOB_MAGIC = 0x0030303242514453ull;   // "SDQB200\0", little endian
constexpr uint32_t BLOB_VERSION = 3;                     // layout version: 2 = compact outlier records tiled per 128 K (WC); 3 = six configuration words
struct BlobHeader {
  uint64_t magic;
  uint32_t version, header_bytes;
  int32_t cfg[6];          // out_n, in_gran, in_block, scale_rule, out_order, out_fmt
  uint32_t tiled;          // 1: stage-tiled tensor-core layout, 2: the same without the 2:4 outlier containers (compact),
                           // 0: canonical arrays (decompose-only reading)
  int64_t N, K;
  uint64_t total;          // bytes of the whole buffer
  uint64_t off[8];         // the section offsets of sdq_packed_t
};
static_assert(sizeof(BlobHeader) <= HEADER_BYTES, "header fits its reservation");

struct PackedOffsets {
  size_t wi, wo, sfa_out, wc, osexp, wtexp, emeta, total;
};
// compact: the buffer carries no 2:4 outlier containers (section WO empty), only the compact records -- the form the grouped
// few-token kernel streams; 4.2 instead of 9.1 bits per weight
inline PackedOffsets packed_offsets(int64_t N, int64_t K, int out_n, bool b32 = false, bool dense = false, bool elem = false, bool compact = false) {
  PackedOffsets o;
  const size_t RT = (size_t)(N / TILE_ROWS), T1 = (size_t)(K / K1), T2 = (size_t)(K / K2);
  auto al = [](size_t x) { return (x + 255) & ~(size_t)255; };
  o.wi = HEADER_BYTES;
  o.wo = al(o.wi + RT * T2 * (size_t)wi_bytes(b32, dense));
  o.sfa_out = al(o.wo + ((out_n && !compact) ? RT * T1 * WO_BYTES : 0));
  o.wc = al(o.sfa_out + RT * SF_ATOM_BYTES);
  o.osexp = al(o.wc + RT * T1 * (size_t)wc_bytes(out_n));
  o.wtexp = al(o.osexp + (size_t)N * 4);                          // inlier row-factor exponents [N] i32 (two-level scaling)
  o.emeta = al(o.wtexp + (size_t)N * 4);                          // element-wise 2:4 stored dense: kept indices [N][K/4] u8
  o.total = al(o.emeta + (elem ? (size_t)N * (size_t)(K / 4) : 0));
  return o;
}

struct ActOffsets {
  size_t xi, xo, sfb_out, sexp, amax, total;
  int64_t MT;
};
inline ActOffsets act_offsets(int64_t M, int64_t K, bool b32 = false) {
  ActOffsets o;
  const size_t MT = (size_t)((M + TILE_TOK - 1) / TILE_TOK), T1 = (size_t)(K / K1), T2 = (size_t)(K / K2);
  auto al = [](size_t x) { return (x + 255) & ~(size_t)255; };
  o.MT = (int64_t)MT;
  o.xi = 0;
  o.xo = al(o.xi + MT * T2 * (size_t)xi_bytes(b32));
  o.sfb_out = al(o.xo + MT * T1 * XO_BYTES);
  o.sexp = al(o.sfb_out + MT * SF_ATOM_BYTES);
  o.amax = al(o.sexp + MT * TILE_TOK * 4);                       // per-token chunk maxima [MT*128][ceil(K/1024)] f32
  o.total = al(o.amax + MT * TILE_TOK * ((size_t)(K + 1023) / 1024) * 4);
  return o;
}

}  // namespace sdq
