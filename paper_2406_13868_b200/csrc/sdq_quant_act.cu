// Runtime activation quantization A -> A_i (E2M1 + E8M0 per 64 K) and A_o (E4M3 + per-token power-of-two
// scale), "we also quantize activations accordingly" (Section 5, Stage 3; A_o / A_i of Section 5.1).
//
// The per-token 8-bit scale needs the whole row before anything can be stored.  Rows up to 16384 long take one
// launch (`quant_act_fused_kernel`): the CTAs of a thread-block cluster split the Q-Vectors of a group of 8 tokens,
// keep their elements in registers, exchange the per-token maxima through distributed shared memory and encode.
// Longer rows take two launches: `act_amax_kernel` reduces, per token, the largest magnitude of each 1024-K chunk,
// `quant_act_kernel` then encodes, one CTA per (group of 8 tokens = one row group of the tiled operand layout,
// 1024-K chunk).  In both a warp works on one 64-K Q-Vector of all 8 tokens at a time: 4 lanes per token, 16
// elements (two 16-byte loads) per lane, so the Q-Vector maximum is a 4-lane shuffle and every store instruction
// writes whole 128-byte lines of the stage-tiled layout (8 tokens x 16 B per core matrix).  Codes come from the
// hardware E2M1 / E4M3 converters and go straight into the layout the GEMM streams.
#include "sdq_codec.cuh"
#include "sdq_internal.h"
#include "sdq_layout.h"
#include "sdq_plain.h"

namespace sdq {

constexpr int QA_THREADS = 256;
constexpr int QA_WARPS = QA_THREADS / 32;
constexpr int QA_CHUNK_QV = 16;                          // Q-Vectors (64 K each) per CTA: 1024 K

__device__ __forceinline__ void load16(const __nv_bfloat16* p, float (&x)[16]) {
  const uint4 a = reinterpret_cast<const uint4*>(p)[0], b = reinterpret_cast<const uint4*>(p)[1];
  const uint32_t r[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    x[2 * i] = __uint_as_float(r[i] << 16);
    x[2 * i + 1] = __uint_as_float(r[i] & 0xFFFF0000u);
  }
}

// partial[m][chunk] = max |x| of token m over its 1024-K chunk
__global__ void __launch_bounds__(QA_THREADS)
act_amax_kernel(const __nv_bfloat16* __restrict__ X, int64_t M, int64_t K, int64_t ldx, float* __restrict__ partial, int n_chunks)
{
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int t = lane >> 2, l = lane & 3;
  const int64_t m = (int64_t)blockIdx.x * 8 + t;
  const bool live = m < M;
  const int NB = (int)(K / 64);
  const int b0 = blockIdx.y * QA_CHUNK_QV;
  __shared__ float s_amax[QA_WARPS][8];
  float amax = 0.0f;
#pragma unroll
  for (int i = 0; i < QA_CHUNK_QV / QA_WARPS; ++i) {
    const int b = b0 + warp + i * QA_WARPS;
    if (live && b < NB) {
      float v[16];
      load16(X + m * ldx + (int64_t)b * 64 + l * 16, v);
#pragma unroll
      for (int j = 0; j < 16; ++j) amax = fmaxf(amax, sat_abs(v[j]));
    }
  }
  amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
  amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
  if (l == 0) s_amax[warp][t] = amax;
  __syncthreads();
  if (tid < 8 && (int64_t)blockIdx.x * 8 + tid < M) {
    float a = 0.0f;
#pragma unroll
    for (int w = 0; w < QA_WARPS; ++w) a = fmaxf(a, s_amax[w][tid]);
    partial[((int64_t)blockIdx.x * 8 + tid) * n_chunks + blockIdx.y] = a;
  }
}

template <bool UE>                                      // UE: two-level scaling with E4M3 Q-Vector scales
__global__ void __launch_bounds__(QA_THREADS)
quant_act_kernel(const __nv_bfloat16* __restrict__ X, int64_t M, int64_t K, int64_t ldx, sdq_config_t cfg, uint8_t* __restrict__ buf,
                 ActOffsets off, const float* __restrict__ partial, int n_chunks)
{
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int t = lane >> 2, l = lane & 3;                 // token within the group of 8, quarter of the Q-Vector
  // a following sdq_linear may start its set-up and weight copies now; it waits for this grid before reading codes
  if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int64_t m = (int64_t)blockIdx.x * 8 + t;
  const bool live = m < M;
  const int NB = (int)(K / 64);                           // Q-Vectors per row
  const int b0 = blockIdx.y * QA_CHUNK_QV;

  // per-token 8-bit scale from the chunk maxima of the whole row
  float ramax = 0.0f;
  if (live)
    for (int c = l; c < n_chunks; c += 4) ramax = fmaxf(ramax, partial[m * n_chunks + c]);
  ramax = fmaxf(ramax, __shfl_xor_sync(0xffffffffu, ramax, 1));
  ramax = fmaxf(ramax, __shfl_xor_sync(0xffffffffu, ramax, 2));
  const int e = fp8_scale_exp(ramax);
  const float s8 = pow2_neg(e);
  const bool i8 = cfg.out_fmt == SDQ_OUT_INT8;       // A_o in int8: fp32 token scale amax / 127, handed on as its bit pattern
  const float sx = int8_scale(ramax);

  const int64_t mt = m / TILE_TOK;
  const uint32_t tk = (uint32_t)(m % TILE_TOK);
  const int T1 = (int)(K / K1), T2 = (int)(K / K2);
  const bool b32 = cfg.in_block == 32;               // one scale per 32 K: a Q-Vector is a lane pair
  constexpr bool ue = UE;
  const int xib = xi_bytes(b32);
  uint8_t* xi_base = buf + off.xi + (size_t)mt * T2 * xib;
  uint8_t* xo_base = buf + off.xo + (size_t)mt * T1 * XO_BYTES;
  if (live && blockIdx.y == 0 && warp == 0 && l == 0) {
    reinterpret_cast<int32_t*>(buf + off.sexp)[m] = i8 ? __float_as_int(sx) : e;
    // two-level scaling keeps a token's accumulator column in units of 2^e (the 4-bit scale codes leave that factor out):
    // the 8-bit product then takes the scale 1 here and the GEMM's epilogue multiplies 2^e back in
    *reinterpret_cast<uint32_t*>(buf + off.sfb_out + (size_t)mt * SF_ATOM_BYTES + sf_off(tk, 0)) = (uint32_t)((ue || i8) ? 127 : e + 127) * 0x01010101u;
  }

#pragma unroll
  for (int i = 0; i < QA_CHUNK_QV / QA_WARPS; ++i) {
    const int b = b0 + warp + i * QA_WARPS;              // uniform over the warp
    if (b >= NB) break;
    float v[16];
    if (live) load16(X + m * ldx + (int64_t)b * 64 + l * 16, v);
    else {
#pragma unroll
      for (int j = 0; j < 16; ++j) v[j] = 0.0f;
    }
    float bmax = 0.0f;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      v[j] = sat(v[j]);
      bmax = fmaxf(bmax, fabsf(v[j]));
    }
    bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 1));
    if (!b32) bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 2));
    const uint32_t c = ue ? ue4m3_scale_code(bmax, e) : e8m0_scale_code(bmax, cfg.scale_rule);
    uint32_t q4[2] = {0, 0}, q8[4] = {0, 0, 0, 0};
    if (!ue) {
      const float s4 = pow2_inv_e8m0(c);
#pragma unroll
      for (int j = 0; j < 8; ++j) q4[j >> 2] |= e2m1x2(v[2 * j] * s4, v[2 * j + 1] * s4) << (8 * (j & 3));
    } else if (c) {
      // two-level scaling: the Q-Vector scale E4M3(c) * 2^e is not a power of two, the elements are divided by it
      const float sv = ue4m3_scale_value(c, e);
#pragma unroll
      for (int j = 0; j < 8; ++j) q4[j >> 2] |= e2m1x2(__fdiv_rn(v[2 * j], sv), __fdiv_rn(v[2 * j + 1], sv)) << (8 * (j & 3));
    }
#pragma unroll
    for (int j = 0; j < 8; ++j)
      q8[j >> 1] |= (i8 ? (int8_code(v[2 * j], sx) | (int8_code(v[2 * j + 1], sx) << 8)) : e4m3x2(v[2 * j] * s8, v[2 * j + 1] * s8)) << (16 * (j & 1));
    if (!live) continue;
    const uint32_t k = (uint32_t)b * 64 + l * 16;          // first element of this lane
    uint8_t* xi = xi_base + (size_t)(k >> 8) * xib;
    uint8_t* xo = xo_base + (size_t)(k >> 7) * XO_BYTES;
    *reinterpret_cast<uint2*>(xi + b_off(tk, (k & 255) >> 1)) = make_uint2(q4[0], q4[1]);
    *reinterpret_cast<uint4*>(xo + b_off(tk, k & 127)) = make_uint4(q8[0], q8[1], q8[2], q8[3]);
    if (b32) { if ((l & 1) == 0) xi[B4_BYTES + in_sf_off(true, tk, (k >> 5) & 7)] = (uint8_t)c; }
    else if (l == 0) xi[B4_BYTES + in_sf_off(false, tk, (uint32_t)(b & 3))] = (uint8_t)c;
  }
}

// Single pass: the CTAs of a cluster share one group of 8 tokens and split its Q-Vectors; every thread keeps its
// elements in registers (packed bf16) from the one read of X, the per-token maxima meet through distributed shared
// memory, and the codes are produced from the registers.  Same arithmetic as the two-kernel path, which stays for
// rows too long for the register budget (K > 64 * QA_WARPS * QF_MAX_IT * 8 = 16384); both scale-block sizes run here.
constexpr int QF_MAX_IT = 4;                             // Q-Vectors per warp
template <int IT, bool UE>
__global__ void __launch_bounds__(QA_THREADS, UE ? 3 : 4)
quant_act_fused_kernel(const __nv_bfloat16* __restrict__ X, int64_t M, int64_t K, int64_t ldx, sdq_config_t cfg, uint8_t* __restrict__ buf,
                       ActOffsets off)
{
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int t = lane >> 2, l = lane & 3;                 // token within the group of 8, quarter of the Q-Vector
  // launched with programmatic stream serialization: X may still be being written by the previous kernel
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const uint32_t cx = gridDim.x, rank = blockIdx.x;      // cluster = the gridDim.x CTAs of one token group
  const int64_t m = (int64_t)blockIdx.y * 8 + t;
  const bool live = m < M;
  const int NB = (int)(K / 64);
  const int per_cta = (NB + (int)cx - 1) / (int)cx;
  const int b_begin = (int)rank * per_cta, b_end = min(NB, b_begin + per_cta);
  __shared__ float s_warp[QA_WARPS][8];
  __shared__ float s_all[8][8];                          // [cluster rank][token]: every CTA's maxima, pushed by their owners

  // magnitudes are compared as 15-bit integers, two per 32-bit word (max.u16x2); +-Inf counts as the largest finite
  // bf16: the maxima are clamped once, the elements only in the (rare) lanes that hold an infinity
  uint4 raw[IT][2];
  uint32_t qmax[IT];                                      // this lane's largest magnitude bits of Q-Vector i (16 elements)
  uint32_t m2 = 0;
#pragma unroll
  for (int i = 0; i < IT; ++i) {
    const int b = b_begin + warp + i * QA_WARPS;
    raw[i][0] = raw[i][1] = make_uint4(0, 0, 0, 0);
    if (live && b < b_end) {
      const uint4* p = reinterpret_cast<const uint4*>(X + m * ldx + (int64_t)b * 64 + l * 16);
      raw[i][0] = p[0];
      raw[i][1] = p[1];
    }
  }
#pragma unroll
  for (int i = 0; i < IT; ++i) {
    const uint32_t r[8] = {raw[i][0].x, raw[i][0].y, raw[i][0].z, raw[i][0].w, raw[i][1].x, raw[i][1].y, raw[i][1].z, raw[i][1].w};
    uint32_t q = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) q = __vmaxu2(q, r[j] & 0x7FFF7FFFu);
    q = max(q & 0xFFFFu, q >> 16);                       // > 0x7F7F: the lane holds an infinity (clamped where used)
    qmax[i] = q;
    m2 = max(m2, min(q, 0x7F7Fu));
  }
  float amax = __uint_as_float(m2 << 16);
  amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
  amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
  if (l == 0) s_warp[warp][t] = amax;
  __syncthreads();
  if (tid < 8 * (int)cx) {
    // thread (peer, token): this CTA's maximum of the token goes into row `rank` of the peer's table
    const int tok = tid & 7;
    const uint32_t peer = (uint32_t)tid >> 3;
    float a = 0.0f;
#pragma unroll
    for (int w = 0; w < QA_WARPS; ++w) a = fmaxf(a, s_warp[w][tok]);
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"((uint32_t)__cvta_generic_to_shared(&s_all[rank][tok])), "r"(peer));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(ra), "f"(a) : "memory");
  }
  // one barrier: every push is visible after it, and nobody touches another CTA's memory afterwards
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  float ramax = 0.0f;
  for (uint32_t c = 0; c < cx; ++c) ramax = fmaxf(ramax, s_all[c][t]);
  const int e = fp8_scale_exp(ramax);
  const float s8 = pow2_neg(e);
  const bool i8 = cfg.out_fmt == SDQ_OUT_INT8;       // A_o in int8: fp32 token scale amax / 127, handed on as its bit pattern
  const float sx = int8_scale(ramax);

  const int64_t mt = m / TILE_TOK;
  const uint32_t tk = (uint32_t)(m % TILE_TOK);
  const int T1 = (int)(K / K1), T2 = (int)(K / K2);
  const bool b32 = cfg.in_block == 32;               // one scale per 32 K: a Q-Vector is a lane pair
  constexpr bool ue = UE;
  const int xib = xi_bytes(b32);
  uint8_t* xi_base = buf + off.xi + (size_t)mt * T2 * xib;
  uint8_t* xo_base = buf + off.xo + (size_t)mt * T1 * XO_BYTES;
  if (live && rank == 0 && warp == 0 && l == 0) {
    reinterpret_cast<int32_t*>(buf + off.sexp)[m] = i8 ? __float_as_int(sx) : e;
    // two-level scaling keeps a token's accumulator column in units of 2^e (the 4-bit scale codes leave that factor out):
    // the 8-bit product then takes the scale 1 here and the GEMM's epilogue multiplies 2^e back in
    *reinterpret_cast<uint32_t*>(buf + off.sfb_out + (size_t)mt * SF_ATOM_BYTES + sf_off(tk, 0)) = (uint32_t)((ue || i8) ? 127 : e + 127) * 0x01010101u;
  }
#pragma unroll
  for (int i = 0; i < IT; ++i) {
    const int b = b_begin + warp + i * QA_WARPS;          // uniform over the warp
    if (b >= b_end) break;
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
    if (!b32) bm = max(bm, __shfl_xor_sync(0xffffffffu, bm, 2));
    const float bmax = __uint_as_float(bm << 16);
    const uint32_t c = ue ? ue4m3_scale_code(bmax, e) : e8m0_scale_code(bmax, cfg.scale_rule);
    uint32_t q4[2] = {0, 0}, q8[4] = {0, 0, 0, 0};
    if (!ue) {
      const float s4 = pow2_inv_e8m0(c);
#pragma unroll
      for (int j = 0; j < 8; ++j) q4[j >> 2] |= e2m1x2(v[2 * j] * s4, v[2 * j + 1] * s4) << (8 * (j & 3));
    } else if (c) {
      // two-level scaling: the Q-Vector scale E4M3(c) * 2^e is not a power of two, the elements are divided by it
      const float sv = ue4m3_scale_value(c, e);
#pragma unroll
      for (int j = 0; j < 8; ++j) q4[j >> 2] |= e2m1x2(__fdiv_rn(v[2 * j], sv), __fdiv_rn(v[2 * j + 1], sv)) << (8 * (j & 3));
    }
#pragma unroll
    for (int j = 0; j < 8; ++j)
      q8[j >> 1] |= (i8 ? (int8_code(v[2 * j], sx) | (int8_code(v[2 * j + 1], sx) << 8)) : e4m3x2(v[2 * j] * s8, v[2 * j + 1] * s8)) << (16 * (j & 1));
    if (!live) continue;
    const uint32_t k = (uint32_t)b * 64 + l * 16;          // first element of this lane
    uint8_t* xi = xi_base + (size_t)(k >> 8) * xib;
    uint8_t* xo = xo_base + (size_t)(k >> 7) * XO_BYTES;
    *reinterpret_cast<uint2*>(xi + b_off(tk, (k & 255) >> 1)) = make_uint2(q4[0], q4[1]);
    *reinterpret_cast<uint4*>(xo + b_off(tk, k & 127)) = make_uint4(q8[0], q8[1], q8[2], q8[3]);
    if (b32) { if ((l & 1) == 0) xi[B4_BYTES + in_sf_off(true, tk, (k >> 5) & 7)] = (uint8_t)c; }
    else if (l == 0) xi[B4_BYTES + in_sf_off(false, tk, (uint32_t)(b & 3))] = (uint8_t)c;
  }
}

__global__ void __launch_bounds__(QA_THREADS)
export_act_kernel(const uint8_t* __restrict__ buf, int64_t M, int64_t K, int in_block, ActOffsets off, sdq_act_canonical_t out)
{
  const int64_t m = blockIdx.x;
  const int64_t mt = m / TILE_TOK;
  const uint32_t t = (uint32_t)(m % TILE_TOK);
  const int T1 = (int)(K / K1), T2 = (int)(K / K2);
  const bool b32 = in_block == 32;
  const int xib = xi_bytes(b32);
  const uint8_t* xi_base = buf + off.xi + (size_t)mt * T2 * xib;
  const uint8_t* xo_base = buf + off.xo + (size_t)mt * T1 * XO_BYTES;
  for (int64_t k = threadIdx.x; k < K; k += QA_THREADS) {
    const uint8_t* xi = xi_base + (size_t)(k >> 8) * xib;
    const uint8_t* xo = xo_base + (size_t)(k >> 7) * XO_BYTES;
    const uint32_t b = xi[b_off(t, (uint32_t)(k & 255) >> 1)];
    out.xq4_code[(size_t)m * K + k] = (uint8_t)((k & 1) ? (b >> 4) : (b & 15));
    out.xq8_code[(size_t)m * K + k] = xo[b_off(t, (uint32_t)(k & 127))];
    if (b32) { if ((k & 31) == 0) out.xq4_scale[(size_t)m * (K / 32) + (k >> 5)] = xi[B4_BYTES + in_sf_off(true, t, (uint32_t)((k >> 5) & 7))]; }
    else if ((k & 63) == 0) out.xq4_scale[(size_t)m * (K / 64) + (k >> 6)] = xi[B4_BYTES + in_sf_off(false, t, (uint32_t)((k >> 6) & 3))];
  }
  if (threadIdx.x == 0) out.xq8_sexp[m] = reinterpret_cast<const int32_t*>(buf + off.sexp)[m];
}

}  // namespace sdq

using namespace sdq;

static bool act_cfg_ok(const sdq_config_t* c) {
  return c && c->out_n >= 0 && c->out_n <= 2 && (c->in_block == 32 || c->in_block == 64) &&
         c->scale_rule >= SDQ_SCALE_OCP_FLOOR && c->scale_rule <= SDQ_SCALE_UE4M3 &&
         (c->out_fmt == SDQ_OUT_E4M3 || (c->out_fmt == SDQ_OUT_INT8 && c->scale_rule != SDQ_SCALE_UE4M3));
}

extern "C" sdq_status_t sdq_act_size(int64_t M, int64_t K, const sdq_config_t* cfg, size_t* bytes)
{
  if (!act_cfg_ok(cfg) || !bytes) return SDQ_ERR_INVALID_ARG;
  if (cfg->scale_rule == SDQ_SCALE_UE4M3 && cfg->in_block != 32) return SDQ_ERR_UNSUPPORTED;
  if (M <= 0 || K <= 0 || K % K2) return SDQ_ERR_SHAPE;
  *bytes = act_offsets(M, K, cfg->in_block == 32).total;
  return SDQ_OK;
}

extern "C" sdq_status_t sdq_quantize_act(const void* X, int64_t M, int64_t K, int64_t ldx, const sdq_config_t* cfg, void* xq_buf,
                                         size_t xq_bytes, sdq_act_t* out, void* stream)
{
  if (!X || !xq_buf || !out || !act_cfg_ok(cfg)) return SDQ_ERR_INVALID_ARG;
  if (cfg->scale_rule == SDQ_SCALE_UE4M3 && cfg->in_block != 32) return SDQ_ERR_UNSUPPORTED;
  if (M <= 0 || K <= 0 || K % K2 || ldx < K) return SDQ_ERR_SHAPE;
  if (((uintptr_t)X & 15) || ((uintptr_t)xq_buf & 15) || (ldx % 8)) return SDQ_ERR_ALIGNMENT;
  const bool b32 = cfg->in_block == 32;
  const ActOffsets off = act_offsets(M, K, b32);
  if (xq_bytes < off.total) return SDQ_ERR_BUFFER_TOO_SMALL;
  const int n_chunks = (int)((K / 64 + QA_CHUNK_QV - 1) / QA_CHUNK_QV);
  float* partial = reinterpret_cast<float*>((uint8_t*)xq_buf + off.amax);
  const dim3 grid((unsigned)((M + 7) / 8), (unsigned)n_chunks);
  // cluster size for the single-pass kernel: enough CTAs per token group that a warp keeps at most QF_MAX_IT Q-Vectors
  const int NB = (int)(K / 64);
  const int cx = (NB + QA_WARPS * QF_MAX_IT - 1) / (QA_WARPS * QF_MAX_IT);
  if (cx <= 8) {
    const int it = ((NB + cx - 1) / cx + QA_WARPS - 1) / QA_WARPS;      // 1..QF_MAX_IT
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)cx, (unsigned)((M + 7) / 8));
    lc.blockDim = dim3(QA_THREADS);
    lc.stream = (cudaStream_t)stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cx;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 2;
    const __nv_bfloat16* Xb = (const __nv_bfloat16*)X;
    uint8_t* bufp = (uint8_t*)xq_buf;
    cudaError_t le;
    if (cfg->scale_rule == SDQ_SCALE_UE4M3) {
      switch (it) {
        case 1: le = cudaLaunchKernelEx(&lc, quant_act_fused_kernel<1, true>, Xb, M, K, ldx, *cfg, bufp, off); break;
        case 2: le = cudaLaunchKernelEx(&lc, quant_act_fused_kernel<2, true>, Xb, M, K, ldx, *cfg, bufp, off); break;
        case 3: le = cudaLaunchKernelEx(&lc, quant_act_fused_kernel<3, true>, Xb, M, K, ldx, *cfg, bufp, off); break;
        default: le = cudaLaunchKernelEx(&lc, quant_act_fused_kernel<4, true>, Xb, M, K, ldx, *cfg, bufp, off); break;
      }
    } else {
      switch (it) {
        case 1: le = cudaLaunchKernelEx(&lc, quant_act_fused_kernel<1, false>, Xb, M, K, ldx, *cfg, bufp, off); break;
        case 2: le = cudaLaunchKernelEx(&lc, quant_act_fused_kernel<2, false>, Xb, M, K, ldx, *cfg, bufp, off); break;
        case 3: le = cudaLaunchKernelEx(&lc, quant_act_fused_kernel<3, false>, Xb, M, K, ldx, *cfg, bufp, off); break;
        default: le = cudaLaunchKernelEx(&lc, quant_act_fused_kernel<4, false>, Xb, M, K, ldx, *cfg, bufp, off); break;
      }
    }
    if (le != cudaSuccess || cudaGetLastError() != cudaSuccess) return SDQ_ERR_CUDA;
  } else {
  act_amax_kernel<<<grid, QA_THREADS, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)X, M, K, ldx, partial, n_chunks);
  if (cfg->scale_rule == SDQ_SCALE_UE4M3)
    quant_act_kernel<true><<<grid, QA_THREADS, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)X, M, K, ldx, *cfg, (uint8_t*)xq_buf, off, partial, n_chunks);
  else
    quant_act_kernel<false><<<grid, QA_THREADS, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)X, M, K, ldx, *cfg, (uint8_t*)xq_buf, off, partial, n_chunks);
  if (cudaGetLastError() != cudaSuccess) return SDQ_ERR_CUDA;
  }
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
  const ActOffsets off = act_offsets(Xq->M, Xq->K, Xq->cfg.in_block == 32);
  export_act_kernel<<<(unsigned)Xq->M, QA_THREADS, 0, (cudaStream_t)stream>>>((const uint8_t*)Xq->dev, Xq->M, Xq->K, Xq->cfg.in_block, off, *out);
  return cudaGetLastError() == cudaSuccess ? SDQ_OK : SDQ_ERR_CUDA;
}
