// The reading of the decomposition that the sparse FP4 tensor core cannot execute -- element-wise 2:4 inliers
// (SDQ_GRAN_ELEM), the literal "2:4" wording -- is decompose / export only.  Its buffer simply holds the canonical
// arrays (one code per byte, sections in the order of sdq_canonical_t); sdq_linear refuses it.
// Same algorithm as sdq_pack.cu (Section 5, Stage 2 -> Stage 1 -> Stage 3), same thread mapping: one thread per
// S-Vector of 8 weights.
#include "sdq_codec.cuh"
#include "sdq_internal.h"
#include "sdq_layout.h"
#include "sdq_plain.h"

namespace sdq {

__global__ void __launch_bounds__(128)
pack_plain_kernel(const __nv_bfloat16* __restrict__ W, int64_t N, int64_t K, int64_t ldw, sdq_config_t cfg, const float* __restrict__ colw,
                  uint8_t* __restrict__ blob, PlainPackedOffsets off, uint32_t* __restrict__ flags)
{
  const int64_t n = blockIdx.x;
  const int tid = threadIdx.x;
  const int G = (int)(K / 8), out_n = cfg.out_n, Bs = cfg.in_block;
  const bool pair = cfg.in_gran == SDQ_GRAN_PAIR;
  const __nv_bfloat16* wrow = W + n * ldw;
  __shared__ uint32_t s_red[4];
  __shared__ int s_e;

  uint32_t okey_max = 0, bad = 0;
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
    select_outliers(skey, out_n, cfg.out_order == SDQ_ORDER_SMALL, o0, o1);
    if (o0 >= 0) okey_max = max(okey_max, key[o0]);
    if (o1 >= 0) okey_max = max(okey_max, key[o1]);
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) {
    okey_max = max(okey_max, __shfl_xor_sync(0xffffffffu, okey_max, s));
    bad |= __shfl_xor_sync(0xffffffffu, bad, s);
  }
  if ((tid & 31) == 0) s_red[tid >> 5] = okey_max;
  if (bad && (tid & 31) == 0) atomicOr(&flags[FLAG_NONFINITE], 1u);
  __syncthreads();
  if (tid == 0) s_e = fp8_scale_exp(bf16_bits_to_float(max(max(s_red[0], s_red[1]), max(s_red[2], s_red[3]))));
  __syncthreads();
  const int e = s_e;
  if (tid == 0) reinterpret_cast<int32_t*>(blob + off.osexp)[n] = e;

  for (int g = tid; g < G; g += 128) {
    uint32_t bits[8], key[8];
    load_group(wrow + 8 * g, bits);
#pragma unroll
    for (int i = 0; i < 8; ++i) key[i] = bits[i] & 0x7FFFu;
    uint32_t skey[8];
    selection_keys(key, colw, g, skey);
    int o0, o1;
    select_outliers(skey, out_n, cfg.out_order == SDQ_ORDER_SMALL, o0, o1);
    int slot_pos[4];
    if (pair) {
      float score[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float a0 = (2 * j == o0 || 2 * j == o1) ? 0.0f : key_value(key[2 * j], skey[2 * j], colw != nullptr);
        const float a1 = (2 * j + 1 == o0 || 2 * j + 1 == o1) ? 0.0f : key_value(key[2 * j + 1], skey[2 * j + 1], colw != nullptr);
        score[j] = __fadd_rn(a0, a1);
      }
      int j0 = 0;
#pragma unroll
      for (int j = 1; j < 4; ++j)
        if (score[j] > score[j0]) j0 = j;
      int j1 = -1;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (j == j0) continue;
        if (j1 < 0 || score[j] > score[j1]) j1 = j;
      }
      if (j0 > j1) { int t = j0; j0 = j1; j1 = t; }
      slot_pos[0] = 2 * j0; slot_pos[1] = 2 * j0 + 1; slot_pos[2] = 2 * j1; slot_pos[3] = 2 * j1 + 1;
      blob[off.in_meta + (size_t)n * G + g] = (uint8_t)(j0 | (j1 << 2));
    } else {
      // element-wise 2:4: in each group of 4 keep the 2 most significant among the non-outlier positions
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        int i0 = -1, i1 = -1;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int p = 4 * h + i;
          if (p == o0 || p == o1) continue;
          if (i0 < 0 || skey[p] > skey[4 * h + i0]) i0 = i;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int p = 4 * h + i;
          if (p == o0 || p == o1 || i == i0) continue;
          if (i1 < 0 || skey[p] > skey[4 * h + i1]) i1 = i;
        }
        if (i0 > i1) { int t = i0; i0 = i1; i1 = t; }
        slot_pos[2 * h] = 4 * h + i0;
        slot_pos[2 * h + 1] = 4 * h + i1;
        blob[off.in_meta + (size_t)n * (2 * G) + 2 * g + h] = (uint8_t)(i0 | (i1 << 2));
      }
    }
    // Q-Vector maximum over the kept inlier values: Bs = 64 -> 8 S-Vectors (8 lanes); Bs = 32 -> 4 lanes
    uint32_t ikey = 0;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const int p = slot_pos[s];
      if (p != o0 && p != o1) ikey = max(ikey, key[p]);
    }
    ikey = max(ikey, __shfl_xor_sync(0xffffffffu, ikey, 1));
    ikey = max(ikey, __shfl_xor_sync(0xffffffffu, ikey, 2));
    if (Bs == 64) ikey = max(ikey, __shfl_xor_sync(0xffffffffu, ikey, 4));
    const uint32_t c = e8m0_scale_code(bf16_bits_to_float(ikey), cfg.scale_rule);
    const int lanes_per_q = Bs / 8;
    if ((g % lanes_per_q) == 0) blob[off.in_scale + (size_t)n * (K / Bs) + g / lanes_per_q] = (uint8_t)c;
    float v[4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const int p = slot_pos[s];
      v[s] = (p == o0 || p == o1) ? 0.0f : bf16_bits_to_float(bits[p]) * pow2_inv_e8m0(c);
    }
    const uint32_t c01 = e2m1x2(v[0], v[1]), c23 = e2m1x2(v[2], v[3]);
    uint8_t* ic = blob + off.in_code + (size_t)n * (K / 2) + 4 * g;
    ic[0] = c01 & 15; ic[1] = c01 >> 4; ic[2] = c23 & 15; ic[3] = c23 >> 4;
    if (out_n > 0) {
      uint8_t* oc = blob + off.out_code + ((size_t)n * G + g) * out_n;
      uint8_t* oi = blob + off.out_idx + ((size_t)n * G + g) * out_n;
      oc[0] = (uint8_t)e4m3x1(bf16_bits_to_float(bits[o0]) * pow2_neg(e));
      oi[0] = (uint8_t)o0;
      if (out_n == 2) {
        oc[1] = (uint8_t)e4m3x1(bf16_bits_to_float(bits[o1]) * pow2_neg(e));
        oi[1] = (uint8_t)o1;
      }
    }
  }
}

void launch_pack_plain(const void* W, int64_t N, int64_t K, int64_t ldw, const sdq_config_t& cfg, const float* col_weight, void* buf,
                       uint32_t* flags, cudaStream_t st)
{
  pack_plain_kernel<<<(unsigned)N, 128, 0, st>>>((const __nv_bfloat16*)W, N, K, ldw, cfg, col_weight, (uint8_t*)buf,
                                                 plain_packed_offsets(N, K, cfg), flags);
}
}  // namespace sdq
