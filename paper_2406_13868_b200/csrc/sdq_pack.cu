// Offline weight decomposition + packing (Section 5, Stage 2 -> Stage 1 -> Stage 3) and its exporter.
//
// One CTA per weight row; one thread per S-Vector of 8 consecutive K (a single 16-byte load).
// Pass 1 finds the row's largest outlier magnitude (the per-row power-of-two scale); pass 2 selects
// outliers, prunes the rest pair-wise, derives the Q-Vector scales by an 8-lane shuffle reduction
// (8 S-Vectors = 64 K), encodes, and scatters into the stage-tiled layout of sdq_layout.h.  Without Stage 1 (dense
// inliers) every position that is not an outlier is encoded, with one scale per 32 K.
#include <cstring>

#include "sdq_codec.cuh"
#include "sdq_internal.h"
#include "sdq_layout.h"
#include "sdq_plain.h"

namespace sdq {

struct GroupSel {
  uint32_t key[8];   // 15-bit magnitude keys
  int o0, o1;        // outlier positions (ascending), -1 if absent
};

// S-Vectors of 4: the most significant of positions 0..3 and of positions 4..7 (ties to the lower index)
__device__ __forceinline__ void select_outliers_per_4(const uint32_t (&key)[8], bool small, int& o0, int& o1) {
  o0 = 0; o1 = 4;
#pragma unroll
  for (int i = 1; i < 4; ++i) {
    if (small ? key[i] < key[o0] : key[i] > key[o0]) o0 = i;
    if (small ? key[4 + i] < key[o1] : key[4 + i] > key[o1]) o1 = 4 + i;
  }
}

// Stage 1, pair-wise 4:8: the 2 pairs (of 4) with the largest summed significance among the non-outliers (one fp32 add
// per pair, largest first, ties to the lower index), ascending
__device__ __forceinline__ void select_pairs(const uint32_t (&key)[8], const uint32_t (&skey)[8], bool weighted, int o0, int o1,
                                             int& j0, int& j1) {
  float score[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float a0 = (2 * j == o0 || 2 * j == o1) ? 0.0f : key_value(key[2 * j], skey[2 * j], weighted);
    const float a1 = (2 * j + 1 == o0 || 2 * j + 1 == o1) ? 0.0f : key_value(key[2 * j + 1], skey[2 * j + 1], weighted);
    score[j] = __fadd_rn(a0, a1);
  }
  j0 = 0;
#pragma unroll
  for (int j = 1; j < 4; ++j)
    if (score[j] > score[j0]) j0 = j;
  j1 = -1;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    if (j == j0) continue;
    if (j1 < 0 || score[j] > score[j1]) j1 = j;
  }
  if (j0 > j1) { int t = j0; j0 = j1; j1 = t; }
}

__global__ void __launch_bounds__(128)
pack_kernel(const __nv_bfloat16* __restrict__ W, int64_t N, int64_t K, int64_t ldw, sdq_config_t cfg, const float* __restrict__ colw,
            uint8_t* __restrict__ blob, PackedOffsets off, uint32_t* __restrict__ flags)
{
  const int64_t n = blockIdx.x;
  const int tid = threadIdx.x;
  const int G = (int)(K / 8);
  const int out_n = cfg.out_n;
  const __nv_bfloat16* wrow = W + n * ldw;
  __shared__ uint32_t s_red[4], s_red_in[4];
  __shared__ int s_e, s_t;
  const bool sv4 = cfg.in_gran == SDQ_GRAN_3OF4;          // S-Vectors of 4: one outlier and two inliers per 4
  const bool small = cfg.out_order == SDQ_ORDER_SMALL;   // Stage 2 takes the least significant values (study control)
  const bool ue = cfg.scale_rule == SDQ_SCALE_UE4M3;     // two-level scaling with E4M3 Q-Vector scales (pair-wise, block 32)
  const bool i8 = cfg.out_fmt == SDQ_OUT_INT8;           // int8 outliers with an fp32 row scale

  // ---- pass 1: largest outlier magnitude of the row (and, for two-level scaling, largest kept inlier), non-finite check
  uint32_t okey_max = 0, ikey_max = 0, bad = 0;
  for (int g = tid; g < G; g += 128) {
    uint32_t bits[8], key[8];
    load_group(wrow + 8 * g, bits);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      key[i] = bits[i] & 0x7FFFu;
      bad |= (key[i] >= 0x7F80u);
    }
    uint32_t skey[8];
    bad |= selection_keys(key, colw, g, skey);
    int o0, o1;
    if (sv4 && out_n) select_outliers_per_4(skey, small, o0, o1); else select_outliers(skey, out_n, small, o0, o1);
    if (o0 >= 0) okey_max = max(okey_max, key[o0]);
    if (o1 >= 0) okey_max = max(okey_max, key[o1]);
    if (ue) {
      int j0, j1;
      select_pairs(key, skey, colw != nullptr, o0, o1, j0, j1);
      const int pos[4] = {2 * j0, 2 * j0 + 1, 2 * j1, 2 * j1 + 1};
#pragma unroll
      for (int s = 0; s < 4; ++s)
        if (pos[s] != o0 && pos[s] != o1) ikey_max = max(ikey_max, key[pos[s]]);
    }
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) {
    okey_max = max(okey_max, __shfl_xor_sync(0xffffffffu, okey_max, s));
    ikey_max = max(ikey_max, __shfl_xor_sync(0xffffffffu, ikey_max, s));
    bad |= __shfl_xor_sync(0xffffffffu, bad, s);
  }
  if ((tid & 31) == 0) { s_red[tid >> 5] = okey_max; s_red_in[tid >> 5] = ikey_max; }
  if (bad && (tid & 31) == 0) atomicOr(&flags[FLAG_NONFINITE], 1u);
  __syncthreads();
  if (tid == 0) {
    uint32_t m = max(max(s_red[0], s_red[1]), max(s_red[2], s_red[3]));
    // int8 outliers: the row's fp32 scale amax / 127 travels as its bit pattern in the place of the exponent
    s_e = i8 ? __float_as_int(int8_scale(bf16_bits_to_float(m))) : fp8_scale_exp(bf16_bits_to_float(m));
    const uint32_t mi = max(max(s_red_in[0], s_red_in[1]), max(s_red_in[2], s_red_in[3]));
    s_t = ue ? fp8_scale_exp(bf16_bits_to_float(mi)) : 0;   // exponent of the row's inlier factor 2^t
  }
  __syncthreads();
  const int e = s_e, tw = s_t;

  const int64_t rt = n / TILE_ROWS;
  const uint32_t r = (uint32_t)(n % TILE_ROWS);
  const int T1 = (int)(K / K1), T2 = (int)(K / K2);
  const bool b32 = cfg.in_block == 32, dense = is_dense_layout(cfg);
  const bool elem = cfg.in_gran == SDQ_GRAN_ELEM;        // element-wise 2:4: the 2 most significant non-outliers of every 4
  const bool grp4 = sv4 || elem;                         // Stage 1 ranks inside groups of 4
  // dense family: inliers kept per group (8 - out_n without Stage 1; groups of 4: 3 minus the outlier, or 2 for 2:4)
  const int keep_in = elem ? 2 : (sv4 ? (out_n ? 2 : 3) : 10 - cfg.in_gran - out_n);
  const int wib = wi_bytes(b32, dense);
  uint8_t* wi_base = blob + off.wi + (size_t)rt * T2 * wib;
  uint8_t* wo_base = blob + off.wo + (size_t)rt * T1 * WO_BYTES;

  if (tid == 0) {
    reinterpret_cast<int32_t*>(blob + off.osexp)[n] = e;
    reinterpret_cast<int32_t*>(blob + off.wtexp)[n] = tw;
    // the accumulator of a row is kept in units of 2^tw (the inlier scale codes leave that factor out), so the outlier
    // row scale is 2^(e - tw); the GEMM's epilogue multiplies the factor back in
    const uint32_t c = i8 ? 127u : (uint32_t)min(max(e - tw + 127, 0), 254);    // (int8: the epilogue applies the scales)
    *reinterpret_cast<uint32_t*>(blob + off.sfa_out + (size_t)rt * SF_ATOM_BYTES + sf_off(r, 0)) = c * 0x01010101u;
  }

  // ---- pass 2 (G is a multiple of 32, so whole warps iterate together)
  for (int g = tid; g < G; g += 128) {
    uint32_t bits[8], key[8];
    load_group(wrow + 8 * g, bits);
#pragma unroll
    for (int i = 0; i < 8; ++i) key[i] = bits[i] & 0x7FFFu;
    uint32_t skey[8];
    selection_keys(key, colw, g, skey);
    int o0, o1;
    if (sv4 && out_n) select_outliers_per_4(skey, small, o0, o1); else select_outliers(skey, out_n, small, o0, o1);
    const int k1 = g >> 4, k2 = g >> 5;
    uint8_t* wi = wi_base + (size_t)k2 * wib;
    uint8_t* wo = wo_base + (size_t)k1 * WO_BYTES;

    if (dense) {
      // all eight positions are inlier slots; an outlier position holds +0, and so does a value that Stage 1 drops: a
      // non-outlier survives if fewer than keep_in non-outliers rank before it (more significant, or equal with a
      // lower index).  Stage 3 with one scale per 32 K = 4 S-Vectors = 4 lanes
      uint32_t gone = 0;        // bit i: position i holds +0
      uint32_t ikey = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        int before = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j)
          before += (j != o0 && j != o1 && (!grp4 || (j >> 2) == (i >> 2)) && (skey[j] > skey[i] || (skey[j] == skey[i] && j < i))) ? 1 : 0;
        if (i == o0 || i == o1 || before >= keep_in) gone |= 1u << i;
        else ikey = max(ikey, key[i]);
      }
      ikey = max(ikey, __shfl_xor_sync(0xffffffffu, ikey, 1));
      ikey = max(ikey, __shfl_xor_sync(0xffffffffu, ikey, 2));
      const uint32_t c = e8m0_scale_code(bf16_bits_to_float(ikey), cfg.scale_rule);
      uint32_t codes = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float v0 = ((gone >> (2 * i)) & 1) ? 0.0f : bf16_bits_to_float(bits[2 * i]) * pow2_inv_e8m0(c);
        const float v1 = ((gone >> (2 * i + 1)) & 1) ? 0.0f : bf16_bits_to_float(bits[2 * i + 1]) * pow2_inv_e8m0(c);
        codes |= e2m1x2(v0, v1) << (8 * i);
      }
      // 32 S-Vectors per 256-K stage, 4 code bytes each: bytes 32 j .. 32 j + 31 = K-block j (64 K)
      *reinterpret_cast<uint32_t*>(wi + a_off(r, (uint32_t)(g & 31) * 4)) = codes;
      if ((g & 3) == 0) wi[a_in_bytes(true) + in_sf_off(true, r, (uint32_t)((g >> 2) & 7))] = (uint8_t)c;
      if (elem) {
        // the kept indices (two ascending 2-bit values per group of 4) are only needed by the exporter
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const uint32_t kept = (~(gone >> (4 * h))) & 15u;            // exactly two bits
          const int i0 = __ffs((int)kept) - 1, i1 = 31 - __clz((int)kept);
          blob[off.emeta + (size_t)n * (size_t)(K / 4) + 2 * g + h] = (uint8_t)(i0 | (i1 << 2));
        }
      }
    } else {
    // Stage 1 on the remaining values: keep the 2 pairs (of 4) with the largest summed significance
    int j0, j1;
    select_pairs(key, skey, colw != nullptr, o0, o1, j0, j1);
    const int slot_pos[4] = {2 * j0, 2 * j0 + 1, 2 * j1, 2 * j1 + 1};

    // Stage 3, inliers: Q-Vector (64 K = 8 S-Vectors = 8 lanes, or 32 K = 4 lanes) largest kept magnitude -> E8M0 scale
    uint32_t ikey = 0;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const int p = slot_pos[s];
      if (p != o0 && p != o1) ikey = max(ikey, key[p]);
    }
    ikey = max(ikey, __shfl_xor_sync(0xffffffffu, ikey, 1));
    ikey = max(ikey, __shfl_xor_sync(0xffffffffu, ikey, 2));
    if (!b32) ikey = max(ikey, __shfl_xor_sync(0xffffffffu, ikey, 4));
    const uint32_t c = ue ? ue4m3_scale_code(bf16_bits_to_float(ikey), tw) : e8m0_scale_code(bf16_bits_to_float(ikey), cfg.scale_rule);
    const float sv = ue ? ue4m3_scale_value(c, tw) : 0.0f;
    float v[4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const int p = slot_pos[s];
      const float w = bf16_bits_to_float(bits[p]);
      v[s] = (p == o0 || p == o1) ? 0.0f : (ue ? (c ? __fdiv_rn(w, sv) : 0.0f) : w * pow2_inv_e8m0(c));
    }
    const uint32_t codes = e2m1x2(v[0], v[1]) | (e2m1x2(v[2], v[3]) << 8);

    // 32 S-Vectors per 256-K stage, 2 code bytes each: bytes 0..31 = K-block 0, 32..63 = K-block 1
    *reinterpret_cast<uint16_t*>(wi + a_off(r, (uint32_t)(g & 31) * 2)) = (uint16_t)codes;
    // metadata nibble j0 | j1<<2; two S-Vectors share a byte (even one in the low nibble)
    uint32_t nib = (uint32_t)(j0 | (j1 << 2));
    const uint32_t nib_hi = __shfl_down_sync(0xffffffffu, nib, 1);
    if ((g & 1) == 0) wi[A_IN_BYTES + r * 16 + ((g & 31) >> 1)] = (uint8_t)(nib | (nib_hi << 4));
    if (b32) { if ((g & 3) == 0) wi[A_IN_BYTES + E_IN_BYTES + in_sf_off(true, r, (uint32_t)((g >> 2) & 7))] = (uint8_t)c; }
    else if ((g & 7) == 0) wi[A_IN_BYTES + E_IN_BYTES + in_sf_off(false, r, (uint32_t)((g >> 3) & 3))] = (uint8_t)c;
    }

    if (out_n > 0) {
      // Stage 3, outliers: E4M3 codes of w / 2^e; compact arrays plus the 2:4 embedding the sparse
      // FP8 tensor-core path consumes (per 4 K: two ascending slot indices, unused slots hold +0)
      // (or int8 codes of w / s, Section 5.1)
      const uint32_t c0 = i8 ? int8_code(bf16_bits_to_float(bits[o0]), __int_as_float(e)) : e4m3x1(bf16_bits_to_float(bits[o0]) * pow2_neg(e));
      const uint32_t c1 = (o1 >= 0) ? (i8 ? int8_code(bf16_bits_to_float(bits[o1]), __int_as_float(e)) : e4m3x1(bf16_bits_to_float(bits[o1]) * pow2_neg(e))) : 0u;
      // compact record of the 128-K stage: codes, then position nibbles (two S-Vectors share a byte when out_n = 1)
      uint8_t* wc = blob + off.wc + ((size_t)rt * T1 + k1) * (size_t)wc_bytes(out_n);
      const uint32_t gi = (uint32_t)(g & 15);
      if (out_n == 1) {
        wc[r * 16 + gi] = (uint8_t)c0;
        const uint32_t pos_hi = __shfl_down_sync(0xffffffffu, (uint32_t)o0, 1);
        if ((g & 1) == 0) wc[WC_CODE_BYTES + r * 8 + (gi >> 1)] = (uint8_t)((uint32_t)o0 | (pos_hi << 4));
      } else {
        *reinterpret_cast<uint16_t*>(wc + r * 32 + gi * 2) = (uint16_t)(c0 | (c1 << 8));
        wc[2 * WC_CODE_BYTES + r * 16 + gi] = (uint8_t)((uint32_t)o0 | ((uint32_t)o1 << 4));
      }
      uint32_t stored = 0, meta = 0;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int a = (o0 >= 4 * h && o0 < 4 * h + 4) ? (o0 - 4 * h) : -1;
        const int b = (o1 >= 4 * h && o1 < 4 * h + 4) ? (o1 - 4 * h) : -1;
        int i0, i1;
        uint32_t s0 = 0, s1 = 0;
        if (a >= 0 && b >= 0) { i0 = a; i1 = b; s0 = c0; s1 = c1; }
        else if (a >= 0 || b >= 0) {
          const int p = (a >= 0) ? a : b;
          const uint32_t cc = (a >= 0) ? c0 : c1;
          if (p < 3) { i0 = p; i1 = 3; s0 = cc; } else { i0 = 0; i1 = 3; s1 = cc; }
        } else { i0 = 0; i1 = 1; }
        stored |= (s0 | (s1 << 8)) << (16 * h);
        meta |= (uint32_t)(i0 | (i1 << 2)) << (4 * h);
      }
      // 16 S-Vectors per 128-K stage, 4 stored bytes each: bytes 0..31 = K-block 0 (64 K), 32..63 = K-block 1
      *reinterpret_cast<uint32_t*>(wo + a_off(r, (uint32_t)(g & 15) * 4)) = stored;
      wo[A_OUT_BYTES + r * 16 + (g & 15)] = (uint8_t)meta;
    }
  }
}

// outlier t of S-Vector g of row r in row tile rt, from the compact records: code and position
__device__ __forceinline__ uint8_t wc_code(const uint8_t* blob, const PackedOffsets& off, int64_t rt, int T1, uint32_t r, int g, int out_n, int t) {
  const uint8_t* wc = blob + off.wc + ((size_t)rt * T1 + (g >> 4)) * (size_t)wc_bytes(out_n);
  return wc[r * 16 * out_n + (g & 15) * out_n + t];
}
__device__ __forceinline__ uint8_t wc_pos(const uint8_t* blob, const PackedOffsets& off, int64_t rt, int T1, uint32_t r, int g, int out_n, int t) {
  const uint8_t* wc = blob + off.wc + ((size_t)rt * T1 + (g >> 4)) * (size_t)wc_bytes(out_n);
  const int e = (g & 15) * out_n + t;
  return (uint8_t)((wc[WC_CODE_BYTES * out_n + r * 8 * out_n + (e >> 1)] >> (4 * (e & 1))) & 15);
}

// packed buffer -> canonical arrays (one code per byte)
__global__ void __launch_bounds__(128)
export_packed_kernel(const uint8_t* __restrict__ blob, int64_t N, int64_t K, sdq_config_t cfg, PackedOffsets off, sdq_canonical_t out)
{
  const int64_t n = blockIdx.x;
  const int G = (int)(K / 8), out_n = cfg.out_n;
  const int64_t rt = n / TILE_ROWS;
  const uint32_t r = (uint32_t)(n % TILE_ROWS);
  const int T1 = (int)(K / K1), T2 = (int)(K / K2);
  const bool b32 = cfg.in_block == 32, dense = is_dense_layout(cfg), elem = cfg.in_gran == SDQ_GRAN_ELEM;
  const int wib = wi_bytes(b32, dense);
  const uint8_t* wi_base = blob + off.wi + (size_t)rt * T2 * wib;
  for (int g = threadIdx.x; g < G; g += 128) {
    const uint8_t* wi = wi_base + (size_t)(g >> 5) * wib;
    if (dense) {
      const uint32_t codes = *reinterpret_cast<const uint32_t*>(wi + a_off(r, (uint32_t)(g & 31) * 4));
      if (elem) {
        // element-wise 2:4: the canonical arrays hold the two kept slots of every 4 and their indices
        uint8_t* ic = out.in_code + (size_t)n * (K / 2) + 4 * g;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const uint32_t mb = blob[off.emeta + (size_t)n * (size_t)(K / 4) + 2 * g + h];
          out.in_meta[(size_t)n * (K / 4) + 2 * g + h] = (uint8_t)mb;
          ic[2 * h] = (codes >> (4 * (4 * h + (mb & 3)))) & 15;
          ic[2 * h + 1] = (codes >> (4 * (4 * h + ((mb >> 2) & 3)))) & 15;
        }
      } else {
      uint8_t* ic = out.in_code + (size_t)n * K + 8 * g;
#pragma unroll
      for (int i = 0; i < 8; ++i) ic[i] = (codes >> (4 * i)) & 15;
      }
      if ((g & 3) == 0) out.in_scale[(size_t)n * (K / 32) + (g >> 2)] = wi[a_in_bytes(true) + in_sf_off(true, r, (uint32_t)((g >> 2) & 7))];
      for (int t = 0; t < out_n; ++t) {
        out.out_code[((size_t)n * G + g) * out_n + t] = wc_code(blob, off, rt, T1, r, g, out_n, t);
        out.out_idx[((size_t)n * G + g) * out_n + t] = wc_pos(blob, off, rt, T1, r, g, out_n, t);
      }
      continue;
    }
    const uint32_t codes = *reinterpret_cast<const uint16_t*>(wi + a_off(r, (uint32_t)(g & 31) * 2));
    uint8_t* ic = out.in_code + (size_t)n * (K / 2) + 4 * g;
    ic[0] = codes & 15; ic[1] = (codes >> 4) & 15; ic[2] = (codes >> 8) & 15; ic[3] = (codes >> 12) & 15;
    const uint32_t mb = wi[A_IN_BYTES + r * 16 + ((g & 31) >> 1)];
    out.in_meta[(size_t)n * G + g] = (uint8_t)((g & 1) ? (mb >> 4) : (mb & 15));
    if (b32) { if ((g & 3) == 0) out.in_scale[(size_t)n * (K / 32) + (g >> 2)] = wi[A_IN_BYTES + E_IN_BYTES + in_sf_off(true, r, (uint32_t)((g >> 2) & 7))]; }
    else if ((g & 7) == 0) out.in_scale[(size_t)n * (K / 64) + (g >> 3)] = wi[A_IN_BYTES + E_IN_BYTES + in_sf_off(false, r, (uint32_t)((g >> 3) & 3))];
    for (int t = 0; t < out_n; ++t) {
      out.out_code[((size_t)n * G + g) * out_n + t] = wc_code(blob, off, rt, T1, r, g, out_n, t);
      out.out_idx[((size_t)n * G + g) * out_n + t] = wc_pos(blob, off, rt, T1, r, g, out_n, t);
    }
  }
  if (threadIdx.x == 0) {
    out.out_sexp[n] = reinterpret_cast<const int32_t*>(blob + off.osexp)[n];
    if (out.in_texp) out.in_texp[n] = reinterpret_cast<const int32_t*>(blob + off.wtexp)[n];
  }
}

}  // namespace sdq

using namespace sdq;

static bool cfg_ok(const sdq_config_t* c) {
  return c && c->out_n >= 0 && c->out_n <= 2 && c->in_gran >= 0 && c->in_gran <= SDQ_GRAN_3OF4 &&
         (c->out_order == SDQ_ORDER_LARGE || c->out_order == SDQ_ORDER_SMALL) &&
         (c->in_gran < SDQ_GRAN_DENSE || c->in_gran == SDQ_GRAN_3OF4 || 10 - c->in_gran > c->out_n) &&
         (c->in_gran != SDQ_GRAN_3OF4 || c->out_n != 1) &&
         (c->in_block == 32 || c->in_block == 64) && c->scale_rule >= SDQ_SCALE_OCP_FLOOR && c->scale_rule <= SDQ_SCALE_UE4M3 &&
         (c->out_fmt == SDQ_OUT_E4M3 || (c->out_fmt == SDQ_OUT_INT8 && c->scale_rule != SDQ_SCALE_UE4M3));
}
// valid configurations this kernel set does not carry out
static bool cfg_unsupported(const sdq_config_t* c) {
  return (c->in_gran >= SDQ_GRAN_DENSE && c->in_block != 32) ||
         (c->scale_rule == SDQ_SCALE_UE4M3 && !(c->in_gran == SDQ_GRAN_PAIR && c->in_block == 32)) ||
         (c->out_fmt == SDQ_OUT_INT8 && !(c->in_gran == SDQ_GRAN_PAIR && c->in_block == 64));   // int8 outliers: the primary format only
}

static void fill_header(BlobHeader* h, const sdq_packed_t& d, bool tiled) {
  h->magic = BLOB_MAGIC;
  h->version = BLOB_VERSION;
  h->header_bytes = (uint32_t)HEADER_BYTES;
  h->cfg[0] = d.cfg.out_n; h->cfg[1] = d.cfg.in_gran; h->cfg[2] = d.cfg.in_block; h->cfg[3] = d.cfg.scale_rule; h->cfg[4] = d.cfg.out_order; h->cfg[5] = d.cfg.out_fmt;
  h->tiled = tiled ? 1u : 0u;
  h->N = d.N; h->K = d.K;
  h->total = d.bytes;
  for (int i = 0; i < 8; ++i) h->off[i] = d.off[i];
}

extern "C" sdq_status_t sdq_packed_size(int64_t N, int64_t K, const sdq_config_t* cfg, size_t* bytes, size_t* algorithmic_bytes)
{
  if (!cfg_ok(cfg)) return SDQ_ERR_INVALID_ARG;
  if (cfg_unsupported(cfg)) return SDQ_ERR_UNSUPPORTED;
  if (N <= 0 || K <= 0 || N % TILE_ROWS || K % K2) return SDQ_ERR_SHAPE;
  if (bytes) *bytes = is_tensor_core_reading(*cfg) ? tiled_offsets(N, K, *cfg).total : plain_packed_offsets(N, K, *cfg).total;
  if (algorithmic_bytes) {
    // per weight: 4-bit values on half the positions (2) + index metadata (pair-wise: two 2-bit pair indices per 8 =
    // 0.5; element-wise: two 2-bit indices per 4 = 1) + one 8-bit scale per Q-Vector + out_n * (8 value + 3 index
    // bits) per 8; plus one 32-bit row scale
    // (dense storage: a 4-bit value on every position and no index metadata)
    const double inl = cfg->in_gran >= SDQ_GRAN_DENSE ? 4.0 : 2.0 + (cfg->in_gran == SDQ_GRAN_PAIR ? 0.5 : 1.0);   // 2:4: the paper's form
    const double bits = inl + 8.0 / cfg->in_block + cfg->out_n * 11.0 / 8.0;
    *algorithmic_bytes = (size_t)((double)N * (double)K * bits / 8.0) + (cfg->out_n ? (size_t)N * 4 : 0);
  }
  return SDQ_OK;
}

extern "C" sdq_status_t sdq_decompose(const void* W, int64_t N, int64_t K, int64_t ldw, const sdq_config_t* cfg, void* packed_buf,
                                      size_t packed_bytes, sdq_packed_t* out, void* stream)
{ return sdq_decompose_metric(W, N, K, ldw, cfg, nullptr, packed_buf, packed_bytes, out, stream); }

extern "C" sdq_status_t sdq_decompose_metric(const void* W, int64_t N, int64_t K, int64_t ldw, const sdq_config_t* cfg,
                                             const float* col_weight, void* packed_buf, size_t packed_bytes, sdq_packed_t* out,
                                             void* stream)
{
  if (!W || !packed_buf || !out || !cfg_ok(cfg)) return SDQ_ERR_INVALID_ARG;
  if (cfg_unsupported(cfg)) return SDQ_ERR_UNSUPPORTED;
  if ((uintptr_t)col_weight & 15) return SDQ_ERR_ALIGNMENT;
  if (N <= 0 || K <= 0 || N % TILE_ROWS || K % K2 || ldw < K) return SDQ_ERR_SHAPE;
  if (((uintptr_t)W & 15) || ((uintptr_t)packed_buf & 15) || (ldw % 8)) return SDQ_ERR_ALIGNMENT;
  const bool tc = is_tensor_core_reading(*cfg);
  const PackedOffsets off = tiled_offsets(N, K, *cfg);
  const PlainPackedOffsets poff = plain_packed_offsets(N, K, *cfg);
  if (packed_bytes < (tc ? off.total : poff.total)) return SDQ_ERR_BUFFER_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  uint32_t* flags = device_flags();
  if (!flags) return SDQ_ERR_CUDA;
  if (cudaMemsetAsync(flags + FLAG_NONFINITE, 0, sizeof(uint32_t), st) != cudaSuccess) return SDQ_ERR_CUDA;
  if (tc) pack_kernel<<<(unsigned)N, 128, 0, st>>>((const __nv_bfloat16*)W, N, K, ldw, *cfg, col_weight, (uint8_t*)packed_buf, off, flags);
  else launch_pack_plain(W, N, K, ldw, *cfg, col_weight, packed_buf, flags, st);
  if (cudaGetLastError() != cudaSuccess) return SDQ_ERR_CUDA;
  uint32_t nonfinite = 0;
  if (cudaMemcpyAsync(&nonfinite, flags + FLAG_NONFINITE, sizeof(uint32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SDQ_ERR_CUDA;
  out->dev = packed_buf;
  out->bytes = tc ? off.total : poff.total;
  out->N = N;
  out->K = K;
  out->cfg = *cfg;
  for (int i = 0; i < 8; ++i) out->off[i] = 0;
  if (tc) {
    out->off[0] = off.wi; out->off[1] = off.wo; out->off[2] = off.sfa_out;
    out->off[3] = off.wc; out->off[4] = 0; out->off[5] = off.osexp; out->off[6] = off.wtexp;
  } else {
    out->off[0] = poff.in_code; out->off[1] = poff.in_meta; out->off[2] = poff.in_scale;
    out->off[3] = poff.out_code; out->off[4] = poff.out_idx; out->off[5] = poff.osexp;
  }
  // the self-describing header (read back by sdq_packed_attach); the copy is complete before `hdr` goes out of scope
  // because the stream is synchronised below
  alignas(16) unsigned char hdr[HEADER_BYTES] = {0};
  fill_header(reinterpret_cast<BlobHeader*>(hdr), *out, tc);
  if (cudaMemcpyAsync(packed_buf, hdr, HEADER_BYTES, cudaMemcpyHostToDevice, st) != cudaSuccess) return SDQ_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return SDQ_ERR_CUDA;
  return nonfinite ? SDQ_ERR_NONFINITE : SDQ_OK;
}

extern "C" sdq_status_t sdq_packed_attach(const void* dev, size_t bytes, sdq_packed_t* out, void* stream)
{
  if (!dev || !out) return SDQ_ERR_INVALID_ARG;
  if ((uintptr_t)dev & 15) return SDQ_ERR_ALIGNMENT;
  if (bytes < HEADER_BYTES) return SDQ_ERR_BUFFER_TOO_SMALL;
  alignas(16) unsigned char raw[HEADER_BYTES];
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(raw, dev, HEADER_BYTES, cudaMemcpyDeviceToHost, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
    return SDQ_ERR_CUDA;
  const BlobHeader* h = reinterpret_cast<const BlobHeader*>(raw);
  if (h->magic != BLOB_MAGIC || h->version != BLOB_VERSION || h->header_bytes != HEADER_BYTES) return SDQ_ERR_UNSUPPORTED;
  sdq_config_t cfg;
  cfg.out_n = h->cfg[0]; cfg.in_gran = h->cfg[1]; cfg.in_block = h->cfg[2]; cfg.scale_rule = h->cfg[3]; cfg.out_order = h->cfg[4]; cfg.out_fmt = h->cfg[5];
  if (!cfg_ok(&cfg) || cfg_unsupported(&cfg)) return SDQ_ERR_SHAPE;
  if (h->N <= 0 || h->K <= 0 || h->N % TILE_ROWS || h->K % K2) return SDQ_ERR_SHAPE;
  // the sections must sit where this library puts them for that configuration and shape
  const bool tc = is_tensor_core_reading(cfg);
  if ((h->tiled != 0) != tc) return SDQ_ERR_SHAPE;
  sdq_packed_t d;
  d.dev = const_cast<void*>(dev);
  d.N = h->N; d.K = h->K; d.cfg = cfg;
  for (int i = 0; i < 8; ++i) d.off[i] = 0;
  if (tc) {
    const bool compact = h->tiled == 2;
    if (h->tiled > 2 || (compact && cfg.out_n == 0)) return SDQ_ERR_SHAPE;
    const PackedOffsets off = tiled_offsets(h->N, h->K, cfg, compact);
    d.bytes = off.total;
    d.off[0] = off.wi; d.off[1] = compact ? 0 : off.wo; d.off[2] = off.sfa_out; d.off[3] = off.wc; d.off[5] = off.osexp; d.off[6] = off.wtexp;
  } else {
    const PlainPackedOffsets poff = plain_packed_offsets(h->N, h->K, cfg);
    d.bytes = poff.total;
    d.off[0] = poff.in_code; d.off[1] = poff.in_meta; d.off[2] = poff.in_scale; d.off[3] = poff.out_code; d.off[4] = poff.out_idx; d.off[5] = poff.osexp;
  }
  if (h->total != d.bytes) return SDQ_ERR_SHAPE;
  for (int i = 0; i < 8; ++i)
    if (h->off[i] != d.off[i]) return SDQ_ERR_SHAPE;
  if (bytes < d.bytes) return SDQ_ERR_BUFFER_TOO_SMALL;
  *out = d;
  return SDQ_OK;
}

extern "C" sdq_status_t sdq_packed_compact_size(int64_t N, int64_t K, const sdq_config_t* cfg, size_t* bytes)
{
  if (!cfg_ok(cfg) || !bytes) return SDQ_ERR_INVALID_ARG;
  if (cfg_unsupported(cfg) || !is_tensor_core_reading(*cfg) || cfg->out_n == 0) return SDQ_ERR_UNSUPPORTED;
  if (N <= 0 || K <= 0 || N % TILE_ROWS || K % K2) return SDQ_ERR_SHAPE;
  *bytes = tiled_offsets(N, K, *cfg, true).total;
  return SDQ_OK;
}

extern "C" sdq_status_t sdq_packed_compact(const sdq_packed_t* P, void* dst, size_t dst_bytes, sdq_packed_t* out, void* stream)
{
  if (!P || !P->dev || !dst || !out) return SDQ_ERR_INVALID_ARG;
  if (!cfg_ok(&P->cfg)) return SDQ_ERR_INVALID_ARG;
  if (!is_tensor_core_reading(P->cfg) || P->cfg.out_n == 0 || is_compact(*P)) return SDQ_ERR_UNSUPPORTED;
  if ((uintptr_t)dst & 255) return SDQ_ERR_ALIGNMENT;
  const PackedOffsets src = tiled_offsets(P->N, P->K, P->cfg), off = tiled_offsets(P->N, P->K, P->cfg, true);
  if (dst_bytes < off.total) return SDQ_ERR_BUFFER_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  const uint8_t* s = (const uint8_t*)P->dev;
  uint8_t* d = (uint8_t*)dst;
  // every section but the 2:4 containers, each to its place in the shorter buffer
  bool ok = cudaMemcpyAsync(d + off.wi, s + src.wi, src.wo - src.wi, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(d + off.sfa_out, s + src.sfa_out, src.total - src.sfa_out, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  if (!ok) return SDQ_ERR_CUDA;
  sdq_packed_t q;
  q.dev = dst; q.bytes = off.total; q.N = P->N; q.K = P->K; q.cfg = P->cfg;
  for (int i = 0; i < 8; ++i) q.off[i] = 0;
  q.off[0] = off.wi; q.off[1] = 0; q.off[2] = off.sfa_out; q.off[3] = off.wc; q.off[5] = off.osexp; q.off[6] = off.wtexp;
  alignas(16) static thread_local unsigned char raw[HEADER_BYTES];
  memset(raw, 0, HEADER_BYTES);
  fill_header(reinterpret_cast<BlobHeader*>(raw), q, true);
  reinterpret_cast<BlobHeader*>(raw)->tiled = 2u;
  if (cudaMemcpyAsync(dst, raw, HEADER_BYTES, cudaMemcpyHostToDevice, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
    return SDQ_ERR_CUDA;
  *out = q;
  return SDQ_OK;
}

extern "C" sdq_status_t sdq_packed_export(const sdq_packed_t* P, const sdq_canonical_t* out, void* stream)
{
  if (!P || !out || !P->dev || !out->in_code || !out->in_scale || !out->out_sexp) return SDQ_ERR_INVALID_ARG;
  if (!out->in_meta && P->cfg.in_gran < SDQ_GRAN_DENSE) return SDQ_ERR_INVALID_ARG;   // PAIR and ELEM record their pattern
  if (P->cfg.out_n > 0 && (!out->out_code || !out->out_idx)) return SDQ_ERR_INVALID_ARG;
  if (!is_tensor_core_reading(P->cfg)) {
    // the buffer already holds the canonical arrays
    const PlainPackedOffsets o = plain_packed_offsets(P->N, P->K, P->cfg);
    const uint8_t* b = (const uint8_t*)P->dev;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t n = (size_t)P->N, k = (size_t)P->K, on = (size_t)P->cfg.out_n;
    bool ok = cudaMemcpyAsync(out->in_code, b + o.in_code, n * k / 2, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(out->in_meta, b + o.in_meta, n * (P->cfg.in_gran == SDQ_GRAN_PAIR ? k / 8 : k / 4), cudaMemcpyDeviceToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(out->in_scale, b + o.in_scale, n * k / (size_t)P->cfg.in_block, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
    if (on) {
      ok = ok && cudaMemcpyAsync(out->out_code, b + o.out_code, n * (k / 8) * on, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
      ok = ok && cudaMemcpyAsync(out->out_idx, b + o.out_idx, n * (k / 8) * on, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
    }
    ok = ok && cudaMemcpyAsync(out->out_sexp, b + o.osexp, n * 4, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
    return ok ? SDQ_OK : SDQ_ERR_CUDA;
  }
  const PackedOffsets off = tiled_offsets(*P);
  export_packed_kernel<<<(unsigned)P->N, 128, 0, (cudaStream_t)stream>>>((const uint8_t*)P->dev, P->N, P->K, P->cfg, off, *out);
  return cudaGetLastError() == cudaSuccess ? SDQ_OK : SDQ_ERR_CUDA;
}
