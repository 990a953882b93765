// Tiled device layouts shared by the packer, the activation quantizer, the exporters and the GEMM.
//
// Everything the GEMM streams is stored so that one contiguous byte range IS the shared-memory image
// of one pipeline stage (128 logical K of one 128-row weight tile / one 128-token activation tile):
// operands sit in the un-swizzled K-major "core matrix" form the tcgen05 shared-memory descriptors
// address (8 rows x 16 bytes = 128 contiguous bytes per core matrix), so a plain bulk copy
// (cp.async.bulk) brings a stage in and no tensor map or swizzle is involved.
//
// Weight buffer (per 128-row tile rt, T1 = K/128 stages k1, T2 = K/256 metadata atoms k2)
//   section INLIER/OUTLIER stages  W1[rt][k1] = | A_in 4096 | A_out 8192 | E_out 2048 |   (out_n > 0)
//                                  W1[rt][k1] = | A_in 4096 |                             (out_n = 0)
//     A_in : 128 rows x 32 B  (64 kept E2M1 codes of the 128 logical K; low nibble = lower k)
//            byte(row r, b) at (b/16)*2048 + (r/8)*128 + (r%8)*16 + b%16
//     A_out: 128 rows x 64 B  (64 stored E4M3 bytes: the 2:4 embedding of the 1:8 / 2:8 outliers)
//            byte(row r, b) at (b/16)*2048 + (r/8)*128 + (r%8)*16 + b%16
//     E_out: 128 rows x 16 B  (one 4-bit index pair per 4 logical K, low nibble = lower chunk)
//   section META                   W2[rt][k2] = | E_in 2048 | SFA_in 512 |
//     E_in : 128 rows x 16 B  (one 4-bit pair-index pair per 8 logical K over 256 K)
//     SFA_in: 4 E8M0 scales (one per 64 K) of 128 rows: byte(r, s) at (r%32)*16 + (r/32)*4 + s
//   section SFA_out[rt]: 512 B, the per-row outlier scale as an E8M0 code, same atom form, 4 copies
//   sections compact outlier codes/indices [N][K/8][out_n] u8 and row scale exponents [N] i32
//
// Activation buffer (per 128-token tile mt)
//   X1[mt][k1] = | B4 8192 | B8 16384 |
//     B4: 128 tokens x 64 B: byte(t, b) at (t/8)*512  + (b/16)*128 + (t%8)*16 + b%16
//     B8: 128 tokens x 128 B: byte(t, b) at (t/8)*1024 + (b/16)*128 + (t%8)*16 + b%16
//   X2[mt][k2] = | SFB_in 512 |   (same atom form as SFA_in, row = token)
//   SFB_out[mt] 512 B (per-token 8-bit scale as E8M0, 4 copies), then xq8 exponents [Mpad] i32
#pragma once
#include <stdint.h>
#include <stddef.h>

namespace sdq {

constexpr int TILE_ROWS = 128;     // weight rows per tile (= MMA M)
constexpr int TILE_TOK = 128;      // tokens per activation tile
constexpr int K1 = 128;            // logical K per pipeline stage
constexpr int K2 = 256;            // logical K per metadata / scale atom

constexpr int A_IN_BYTES = 4096;
constexpr int A_OUT_BYTES = 8192;
constexpr int E_OUT_BYTES = 2048;
constexpr int E_IN_BYTES = 2048;
constexpr int SF_ATOM_BYTES = 512;
constexpr int W2_BYTES = E_IN_BYTES + SF_ATOM_BYTES;   // 2560
constexpr int B4_BYTES = 8192;
constexpr int B8_BYTES = 16384;
constexpr int X1_BYTES = B4_BYTES + B8_BYTES;           // 24576
constexpr int X2_BYTES = SF_ATOM_BYTES;

__host__ __device__ inline int w1_bytes(int out_n) { return out_n ? (A_IN_BYTES + A_OUT_BYTES + E_OUT_BYTES) : A_IN_BYTES; }

// offsets inside a core-matrix tile whose K-adjacent core matrices are `lbo` bytes apart and whose
// row-group-adjacent core matrices are `sbo` bytes apart
__host__ __device__ inline uint32_t core_off(uint32_t row, uint32_t byte, uint32_t lbo, uint32_t sbo) {
  return (byte >> 4) * lbo + (row >> 3) * sbo + (row & 7) * 16 + (byte & 15);
}
__host__ __device__ inline uint32_t a_off(uint32_t row, uint32_t byte) { return core_off(row, byte, 2048, 128); }
__host__ __device__ inline uint32_t b4_off(uint32_t tok, uint32_t byte) { return core_off(tok, byte, 128, 512); }
__host__ __device__ inline uint32_t b8_off(uint32_t tok, uint32_t byte) { return core_off(tok, byte, 128, 1024); }
__host__ __device__ inline uint32_t sf_off(uint32_t row, uint32_t s) { return (row & 31) * 16 + (row >> 5) * 4 + s; }

constexpr size_t HEADER_BYTES = 256;

struct PackedOffsets {
  size_t w1, w2, sfa_out, ocode, oidx, osexp, total;
};
inline PackedOffsets packed_offsets(int64_t N, int64_t K, int out_n) {
  PackedOffsets o;
  const size_t RT = (size_t)(N / TILE_ROWS), T1 = (size_t)(K / K1), T2 = (size_t)(K / K2);
  auto al = [](size_t x) { return (x + 255) & ~(size_t)255; };
  o.w1 = HEADER_BYTES;
  o.w2 = al(o.w1 + RT * T1 * (size_t)w1_bytes(out_n));
  o.sfa_out = al(o.w2 + RT * T2 * W2_BYTES);
  o.ocode = al(o.sfa_out + RT * SF_ATOM_BYTES);
  o.oidx = al(o.ocode + (size_t)N * (size_t)(K / 8) * (size_t)out_n);
  o.osexp = al(o.oidx + (size_t)N * (size_t)(K / 8) * (size_t)out_n);
  o.total = al(o.osexp + (size_t)N * 4);
  return o;
}

struct ActOffsets {
  size_t x1, x2, sfb_out, sexp, total;
  int64_t MT;
};
inline ActOffsets act_offsets(int64_t M, int64_t K) {
  ActOffsets o;
  const size_t MT = (size_t)((M + TILE_TOK - 1) / TILE_TOK), T1 = (size_t)(K / K1), T2 = (size_t)(K / K2);
  auto al = [](size_t x) { return (x + 255) & ~(size_t)255; };
  o.MT = (int64_t)MT;
  o.x1 = 0;
  o.x2 = al(o.x1 + MT * T1 * X1_BYTES);
  o.sfb_out = al(o.x2 + MT * T2 * X2_BYTES);
  o.sexp = al(o.sfb_out + MT * SF_ATOM_BYTES);
  o.total = al(o.sexp + MT * TILE_TOK * 4);
  return o;
}

}  // namespace sdq
