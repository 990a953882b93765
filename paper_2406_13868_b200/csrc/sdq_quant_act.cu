// Runtime activation quantization A -> A_i (E2M1 + E8M0 per 64 K) and A_o (E4M3 + per-token power-of-two
// scale), "we also quantize activations accordingly" (Section 5, Stage 3; A_o / A_i of Section 5.1).
//
// One CTA per token row, 16-byte loads (8 bf16 per thread per step).  Pass 1 reduces the row's largest
// magnitude (the 8-bit scale needs the whole row); pass 2 re-reads the row (L2 resident), reduces each
// 64-K Q-Vector over 8 lanes by warp shuffle, converts with the hardware E2M1 / E4M3 converters and
// stores packed codes straight into the stage-tiled layout the GEMM streams with bulk copies.
#include "sdq_codec.cuh"
#include "sdq_internal.h"
#include "sdq_layout.h"

namespace sdq {

constexpr int QA_THREADS = 256;

__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&x)[8]) {
  const uint4 v = *reinterpret_cast<const uint4*>(p);
  const uint32_t r[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    x[2 * i] = __uint_as_float(r[i] << 16);
    x[2 * i + 1] = __uint_as_float(r[i] & 0xFFFF0000u);
  }
}
// |x| with +-Inf replaced by the largest finite bf16 (saturation), as a float
__device__ __forceinline__ float sat_abs(float x) { return fminf(fabsf(x), 3.3895313892515355e38f); }
__device__ __forceinline__ float sat(float x) { return copysignf(sat_abs(x), x); }

__global__ void __launch_bounds__(QA_THREADS)
quant_act_kernel(const __nv_bfloat16* __restrict__ X, int64_t M, int64_t K, int64_t ldx, sdq_config_t cfg, uint8_t* __restrict__ buf,
                 ActOffsets off)
{
  const int64_t m = blockIdx.x;
  const int tid = threadIdx.x;
  const __nv_bfloat16* x = X + m * ldx;
  __shared__ float s_red[QA_THREADS / 32];
  __shared__ int s_e;

  float amax = 0.0f;
  for (int64_t k = (int64_t)tid * 8; k < K; k += QA_THREADS * 8) {
    float v[8];
    load8(x + k, v);
#pragma unroll
    for (int i = 0; i < 8; ++i) amax = fmaxf(amax, sat_abs(v[i]));
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, s));
  if ((tid & 31) == 0) s_red[tid >> 5] = amax;
  __syncthreads();
  if (tid == 0) {
    float a = 0.0f;
#pragma unroll
    for (int i = 0; i < QA_THREADS / 32; ++i) a = fmaxf(a, s_red[i]);
    s_e = fp8_scale_exp(a);
  }
  __syncthreads();
  const int e = s_e;

  const int64_t mt = m / TILE_TOK;
  const uint32_t t = (uint32_t)(m % TILE_TOK);
  const int T1 = (int)(K / K1), T2 = (int)(K / K2);
  uint8_t* xi_base = buf + off.xi + (size_t)mt * T2 * XI_BYTES;
  uint8_t* xo_base = buf + off.xo + (size_t)mt * T1 * XO_BYTES;
  if (tid == 0) {
    reinterpret_cast<int32_t*>(buf + off.sexp)[m] = e;
    *reinterpret_cast<uint32_t*>(buf + off.sfb_out + (size_t)mt * SF_ATOM_BYTES + sf_off(t, 0)) = (uint32_t)(e + 127) * 0x01010101u;
  }

  // K is a multiple of 256, so every warp-iteration covers whole 64-K Q-Vectors (8 lanes each)
  for (int64_t k = (int64_t)tid * 8; k < K; k += QA_THREADS * 8) {
    float v[8];
    load8(x + k, v);
    float bmax = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      v[i] = sat(v[i]);
      bmax = fmaxf(bmax, fabsf(v[i]));
    }
    bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 1));
    bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 2));
    bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 4));
    const uint32_t c = e8m0_scale_code(bmax, cfg.scale_rule);
    uint32_t q4 = 0, q8lo = 0, q8hi = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      q4 |= e2m1x2(scalbnf(v[2 * i], 127 - (int)c), scalbnf(v[2 * i + 1], 127 - (int)c)) << (8 * i);
      const uint32_t p = e4m3x2(scalbnf(v[2 * i], -e), scalbnf(v[2 * i + 1], -e));
      if (i < 2) q8lo |= p << (16 * i); else q8hi |= p << (16 * (i - 2));
    }
    const int k1 = (int)(k >> 7), k2 = (int)(k >> 8);
    uint8_t* xi = xi_base + (size_t)k2 * XI_BYTES;
    uint8_t* xo = xo_base + (size_t)k1 * XO_BYTES;
    *reinterpret_cast<uint32_t*>(xi + b_off(t, (uint32_t)(k & 255) >> 1)) = q4;
    *reinterpret_cast<uint2*>(xo + b_off(t, (uint32_t)(k & 127))) = make_uint2(q8lo, q8hi);
    if ((k & 63) == 0) xi[B4_BYTES + sf_off(t, (uint32_t)((k >> 6) & 3))] = (uint8_t)c;
  }
}

__global__ void __launch_bounds__(QA_THREADS)
export_act_kernel(const uint8_t* __restrict__ buf, int64_t M, int64_t K, ActOffsets off, sdq_act_canonical_t out)
{
  const int64_t m = blockIdx.x;
  const int64_t mt = m / TILE_TOK;
  const uint32_t t = (uint32_t)(m % TILE_TOK);
  const int T1 = (int)(K / K1), T2 = (int)(K / K2);
  const uint8_t* xi_base = buf + off.xi + (size_t)mt * T2 * XI_BYTES;
  const uint8_t* xo_base = buf + off.xo + (size_t)mt * T1 * XO_BYTES;
  for (int64_t k = threadIdx.x; k < K; k += QA_THREADS) {
    const uint8_t* xi = xi_base + (size_t)(k >> 8) * XI_BYTES;
    const uint8_t* xo = xo_base + (size_t)(k >> 7) * XO_BYTES;
    const uint32_t b = xi[b_off(t, (uint32_t)(k & 255) >> 1)];
    out.xq4_code[(size_t)m * K + k] = (uint8_t)((k & 1) ? (b >> 4) : (b & 15));
    out.xq8_code[(size_t)m * K + k] = xo[b_off(t, (uint32_t)(k & 127))];
    if ((k & 63) == 0) out.xq4_scale[(size_t)m * (K / 64) + (k >> 6)] = xi[B4_BYTES + sf_off(t, (uint32_t)((k >> 6) & 3))];
  }
  if (threadIdx.x == 0) out.xq8_sexp[m] = reinterpret_cast<const int32_t*>(buf + off.sexp)[m];
}

}  // namespace sdq

using namespace sdq;

static bool act_cfg_ok(const sdq_config_t* c) {
  return c && c->out_n >= 0 && c->out_n <= 2 && (c->in_block == 32 || c->in_block == 64) &&
         (c->scale_rule == SDQ_SCALE_OCP_FLOOR || c->scale_rule == SDQ_SCALE_CEIL_NOSAT);
}

extern "C" sdq_status_t sdq_act_size(int64_t M, int64_t K, const sdq_config_t* cfg, size_t* bytes)
{
  if (!act_cfg_ok(cfg) || !bytes) return SDQ_ERR_INVALID_ARG;
  if (M <= 0 || K <= 0 || K % K2) return SDQ_ERR_SHAPE;
  if (cfg->in_block != 64) return SDQ_ERR_UNSUPPORTED;
  *bytes = act_offsets(M, K).total;
  return SDQ_OK;
}

extern "C" sdq_status_t sdq_quantize_act(const void* X, int64_t M, int64_t K, int64_t ldx, const sdq_config_t* cfg, void* xq_buf,
                                         size_t xq_bytes, sdq_act_t* out, void* stream)
{
  if (!X || !xq_buf || !out || !act_cfg_ok(cfg)) return SDQ_ERR_INVALID_ARG;
  if (M <= 0 || K <= 0 || K % K2 || ldx < K) return SDQ_ERR_SHAPE;
  if (cfg->in_block != 64) return SDQ_ERR_UNSUPPORTED;
  if (((uintptr_t)X & 15) || ((uintptr_t)xq_buf & 15) || (ldx % 8)) return SDQ_ERR_ALIGNMENT;
  const ActOffsets off = act_offsets(M, K);
  if (xq_bytes < off.total) return SDQ_ERR_BUFFER_TOO_SMALL;
  quant_act_kernel<<<(unsigned)M, QA_THREADS, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)X, M, K, ldx, *cfg, (uint8_t*)xq_buf, off);
  if (cudaGetLastError() != cudaSuccess) return SDQ_ERR_CUDA;
  out->dev = xq_buf;
  out->bytes = off.total;
  out->M = M;
  out->K = K;
  out->cfg = *cfg;
  for (int i = 0; i < 6; ++i) out->off[i] = 0;
  out->off[0] = off.xi; out->off[1] = off.xo; out->off[2] = off.sfb_out; out->off[3] = off.sexp;
  return SDQ_OK;
}

extern "C" sdq_status_t sdq_act_export(const sdq_act_t* Xq, const sdq_act_canonical_t* out, void* stream)
{
  if (!Xq || !out || !Xq->dev || !out->xq4_code || !out->xq4_scale || !out->xq8_code || !out->xq8_sexp) return SDQ_ERR_INVALID_ARG;
  const ActOffsets off = act_offsets(Xq->M, Xq->K);
  export_act_kernel<<<(unsigned)Xq->M, QA_THREADS, 0, (cudaStream_t)stream>>>((const uint8_t*)Xq->dev, Xq->M, Xq->K, off, *out);
  return cudaGetLastError() == cudaSuccess ? SDQ_OK : SDQ_ERR_CUDA;
}
