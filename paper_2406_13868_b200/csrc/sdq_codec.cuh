// Device-side number-format helpers of the packer and the activation quantizer.
// E2M1 / E4M3 encoding uses the hardware converters (round to nearest even, saturate to the largest
// finite value); scales are powers of two so every scaling below is exact.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp4.h>
#include <cuda_fp8.h>
#include <stdint.h>

namespace sdq {

__device__ __forceinline__ float bf16_bits_to_float(uint32_t h) { return __uint_as_float(h << 16); }

// a = f * 2^p with f in [1, 2):  returns p and f (a > 0, finite; subnormals handled)
__device__ __forceinline__ void split_pow2(float a, int& p, float& f) {
  p = ilogbf(a);
  f = scalbnf(a, -p);
}

// E8M0 code of the Q-Vector scale of 4-bit values whose largest magnitude is amax
//   rule 0: E = floor(log2 amax) - 2      rule 1: E = smallest integer with amax <= 6 * 2^E
__device__ __forceinline__ uint32_t e8m0_scale_code(float amax, int rule) {
  if (amax == 0.0f) return 0u;
  int p;
  float f;
  split_pow2(amax, p, f);
  int E = (rule == 0) ? (p - 2) : ((f <= 1.5f) ? (p - 2) : (p - 1));
  int c = E + 127;
  return (uint32_t)min(max(c, 0), 254);
}

// int8 operands (Section 5.1: W_o and A_o in int8): scale amax / 127 (1 for an all-zero vector) and code = the integer
// nearest to x / s, ties to even, limited to +-127 -- both quotients in fp32, IEEE round-to-nearest divisions, the
// precision in which the code is decided; returns the code's byte
__device__ __forceinline__ float int8_scale(float amax) { return amax == 0.0f ? 1.0f : __fdiv_rn(amax, 127.0f); }
__device__ __forceinline__ uint32_t int8_code(float x, float s) {
  const float r = fminf(fmaxf(rintf(__fdiv_rn(x, s)), -127.0f), 127.0f);
  return (uint32_t)(int)r & 0xFFu;
}

// exponent e of the power-of-two scale of an 8-bit (E4M3, max 448 = 1.75 * 2^8) operand:
// the smallest integer with amax <= 448 * 2^e, limited to what an E8M0 byte can carry
__device__ __forceinline__ int fp8_scale_exp(float amax) {
  if (amax == 0.0f) return 0;
  int p;
  float f;
  split_pow2(amax, p, f);
  int e = (f <= 1.75f) ? (p - 8) : (p - 7);
  return min(max(e, -127), 127);
}

// 2^(127 - c) for an E8M0 code c <= 253 and 2^(-e) for an 8-bit scale exponent e in [-127, 120], built from
// the exponent field: multiplying by them is exact (the products here never overflow; results too small for
// fp32 are far below half of the smallest E2M1 / E4M3 step and round to zero either way)
__device__ __forceinline__ float pow2_inv_e8m0(uint32_t c) { return __uint_as_float((254u - c) << 23); }
__device__ __forceinline__ float pow2_neg(int e) { return __uint_as_float((uint32_t)(127 - e) << 23); }

// Two-level scaling (SDQ_SCALE_UE4M3): unsigned E4M3 code of the Q-Vector scale nearest to amax / (6 * 2^t), at least
// the smallest positive code unless amax == 0, and the value scale * 2^t the elements are divided by (0 for code 0).
// amax * 2^-t is exact (amax <= 448 * 2^t); the one rounding of the division is far from every E4M3 midpoint or
// lands on it exactly, so the converter's round-to-nearest-even is that of the exact quotient.
__device__ __forceinline__ uint32_t ue4m3_scale_code(float amax, int t) {
  if (amax == 0.0f) return 0u;
  const uint32_t c = (uint32_t)__nv_cvt_float_to_fp8(__fdiv_rn(scalbnf(amax, -t), 6.0f), __NV_SATFINITE, __NV_E4M3);
  return c == 0u ? 1u : c;
}
__device__ __forceinline__ float ue4m3_scale_value(uint32_t c, int t) {
  const __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)c, __NV_E4M3);
  return scalbnf(__half2float(__half(h)), t);
}

// two floats -> two E2M1 codes in one byte (x in the low nibble)
__device__ __forceinline__ uint32_t e2m1x2(float x, float y) {
  return (uint32_t)__nv_cvt_float2_to_fp4x2(make_float2(x, y), __NV_E2M1, cudaRoundNearest);
}
// two floats -> two E4M3 codes in 16 bits (x in the low byte)
__device__ __forceinline__ uint32_t e4m3x2(float x, float y) {
  return (uint32_t)__nv_cvt_float2_to_fp8x2(make_float2(x, y), __NV_SATFINITE, __NV_E4M3);
}
__device__ __forceinline__ uint32_t e4m3x1(float x) { return (uint32_t)__nv_cvt_float_to_fp8(x, __NV_SATFINITE, __NV_E4M3); }

// selection keys of one S-Vector: the 15-bit magnitude itself, or -- with a per-input-channel weight c[k] -- the bit
// pattern of the fp32 product |w| * c[k] (one round-to-nearest multiply; non-negative floats order like their bits).
// Returns nonzero if a channel weight is negative, infinite or NaN.
__device__ __forceinline__ uint32_t selection_keys(const uint32_t (&key)[8], const float* __restrict__ colw, int g, uint32_t (&skey)[8]) {
  if (!colw) {
#pragma unroll
    for (int i = 0; i < 8; ++i) skey[i] = key[i];
    return 0;
  }
  const float4 c0 = reinterpret_cast<const float4*>(colw + 8 * g)[0], c1 = reinterpret_cast<const float4*>(colw + 8 * g)[1];
  const float c[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
  uint32_t bad = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    bad |= !(c[i] >= 0.0f && c[i] <= 3.4028234663852886e38f);
    skey[i] = __float_as_uint(__fmul_rn(bf16_bits_to_float(key[i]), c[i]));
  }
  return bad;
}
// significance of position i as a float (for the pair score)
__device__ __forceinline__ float key_value(uint32_t key, uint32_t skey, bool weighted) {
  return weighted ? __uint_as_float(skey) : bf16_bits_to_float(key);
}

// |x| with +-Inf replaced by the largest finite bf16 (saturation)
__device__ __forceinline__ float sat_abs(float x) { return fminf(fabsf(x), 3.3895313892515355e38f); }
__device__ __forceinline__ float sat(float x) { return copysignf(sat_abs(x), x); }

// ---- Stage 2 helpers shared by the tiled and the plain packer (one thread per S-Vector of 8 weights) ----------
// the 8 bf16 bit patterns of an S-Vector (one 16-byte load)
__device__ __forceinline__ void load_group(const __nv_bfloat16* w, uint32_t (&bits)[8]) {
  const uint4 v = *reinterpret_cast<const uint4*>(w);
  const uint32_t r[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    bits[2 * i] = r[i] & 0xFFFFu;
    bits[2 * i + 1] = r[i] >> 16;
  }
}

// positions of the out_n most (small: least) significant values, ties to the lower index
__device__ __forceinline__ void select_outliers(const uint32_t (&key)[8], int out_n, bool small, int& o0, int& o1) {
  o0 = o1 = -1;
  if (out_n >= 1) {
    int b = 0;
#pragma unroll
    for (int i = 1; i < 8; ++i)
      if (small ? key[i] < key[b] : key[i] > key[b]) b = i;
    o0 = b;
  }
  if (out_n >= 2) {
    int b = -1;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (i == o0) continue;
      if (b < 0 || (small ? key[i] < key[b] : key[i] > key[b])) b = i;
    }
    o1 = b;
    if (o0 > o1) { int t = o0; o0 = o1; o1 = t; }
  }
}

}  // namespace sdq
