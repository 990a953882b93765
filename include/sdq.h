/*
 * sdq.h -- C-ABI of the B200 (sm_100a) SDQ decomposed linear layer
 *
 *     Y = A_i * W_i^T + A_o * W_o^T
 *
 * following "SDQ: Sparse Decomposed Quantization for LLM Inference" (arXiv 2406.13868):
 *   Section 5, Stage 1 (N:M magnitude sparsification), Stage 2 (local N:M outlier extraction per
 *   S-Vector), Stage 3 (different number formats for inliers and outliers, activations quantized
 *   accordingly) and the paragraph "LLM inference performance" (O = O_o + O_i).
 *
 * Conventions
 *   W [N, K] bf16, row-major (row = output feature, K contiguous);  X [M, K] bf16;  Y [M, N].
 *   "device" pointers are CUDA device memory of the current device; "host" pointers are plain
 *   host memory.  The library never allocates or frees device memory: every buffer is owned by the
 *   caller and sized with the *_size queries.  All launches go to the caller's stream; nothing
 *   synchronises unless stated.  Every function returns a status code; nothing throws or aborts.
 *   Preconditions: N % 128 == 0, K % 256 == 0 (the inlier metadata and scale atoms of the sparse 4-bit tensor-core
 *   kind cover 256 K: a record of the packed layout is one such atom), M >= 1, 16-byte aligned pointers, finite weights.
 */
#ifndef SDQ_H_
#define SDQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SDQ_OK = 0,
  SDQ_ERR_INVALID_ARG = 1,      /* null pointer, bad enum value                              */
  SDQ_ERR_SHAPE = 2,            /* N, K, M violate the preconditions or operands disagree    */
  SDQ_ERR_ALIGNMENT = 3,        /* pointer or leading dimension not 16-byte aligned          */
  SDQ_ERR_UNSUPPORTED = 4,      /* valid config that this kernel set cannot execute          */
  SDQ_ERR_BUFFER_TOO_SMALL = 5, /* caller buffer smaller than the matching *_size query      */
  SDQ_ERR_NONFINITE = 6,        /* Inf/NaN weight (or bad channel weight) seen by sdq_decompose */
  SDQ_ERR_CUDA = 7,             /* a CUDA runtime call failed (launch error etc.)            */
  SDQ_ERR_TIMEOUT = 8           /* a bounded device-side wait gave up (sticky device status) */
} sdq_status_t;

enum { SDQ_GRAN_PAIR = 0, SDQ_GRAN_ELEM = 1, SDQ_GRAN_DENSE = 2 }; /* inlier pattern            */
#define SDQ_GRAN_KEEP(n) (2 + (8 - (n)))  /* n:8 sparsification, n = 2..8; SDQ_GRAN_KEEP(8) == SDQ_GRAN_DENSE */
#define SDQ_GRAN_3OF4 9                   /* S-Vectors of 4: 3:4 = 1:4 outliers + 2:4 inliers                 */
enum { SDQ_SCALE_OCP_FLOOR = 0, SDQ_SCALE_CEIL_NOSAT = 1, SDQ_SCALE_UE4M3 = 2 }; /* Q-Vector scale rule */
enum { SDQ_ORDER_LARGE = 0, SDQ_ORDER_SMALL = 1 };          /* Stage 2 takes the most / least significant values */
/* 8-bit format of the outlier operands.  SDQ_OUT_E4M3: FP8 E4M3 with a power-of-two scale per weight row / token, applied by
 * the tensor core, so that O_i and O_o can share an accumulator.  SDQ_OUT_INT8 (Section 5.1 "quantize 1:8 W_o as int8 ...
 * A would be quantized to int8 A_o"): symmetric int8, one fp32 scale amax / 127 per weight row and per token (1 for an
 * all-zero vector), code = integer nearest to x / s (ties to even, |code| <= 127), both quotients formed in fp32; O_o is
 * accumulated exactly in int32 and scaled in the epilogue.  Pair-wise 4:8 inliers with in_block 64 only; computed by
 * sdq_linear_group's fused kernel (other calls return SDQ_ERR_UNSUPPORTED for it).  out_sexp / xq8_sexp of the canonical
 * exports then hold the bit patterns of the fp32 scales. */
enum { SDQ_OUT_E4M3 = 0, SDQ_OUT_INT8 = 1 };

/* "pattern, formats" of the decomposition (Section 5, Stages 1-3).
 *   out_n      outliers extracted per S-Vector of 8 consecutive K (Stage 2): 0, 1 or 2; stored as
 *              FP8-E4M3 with one power-of-two scale per weight row.
 *   in_gran    how the remaining values are pruned to 50% (Stage 1, magnitude metric):
 *              SDQ_GRAN_PAIR keeps the 2 adjacent pairs (of 4) with the largest |a|+|b| in every 8
 *              (the pattern the sparse FP4 tensor core consumes); SDQ_GRAN_ELEM keeps the 2 largest
 *              of every 4 (with in_block = 32 the inliers are stored and executed like the dense
 *              pattern below, the dropped positions holding +0; with in_block = 64 decompose / export
 *              only: the buffer then holds the canonical arrays and sdq_linear returns
 *              SDQ_ERR_UNSUPPORTED).  SDQ_GRAN_DENSE skips Stage 1: every value that
 *              is not an outlier stays an inlier (the evaluation's configuration 8:8 = 1:8 outliers +
 *              7:8 inliers); sdq_linear runs W_i as a dense 4-bit operand.  SDQ_GRAN_KEEP(n), n > out_n:
 *              Stage 1 keeps the n most significant values of every S-Vector of 8, of which the out_n most
 *              significant are the outliers and the other n - out_n the inliers, at whatever positions
 *              they have (the evaluation's flexible N:M configurations, e.g. 7:8 = 1:8 + 6:8; largest
 *              first, ties to the lower k); stored and executed like the dense pattern, the dropped
 *              positions holding +0.  SDQ_GRAN_3OF4 (the evaluation's 3:4 = 1:4 + 2:4): per 4 consecutive K
 *              the most significant value is the outlier (out_n must be 2, i.e. two per 8, or 0), the
 *              next two stay inliers, the last is dropped; stored and executed like the dense pattern.
 *              The dense 4-bit tensor-core kind has one scale per 32 K only, so
 *              these patterns require in_block = 32 (with 64 every call returns SDQ_ERR_UNSUPPORTED).
 *   in_block   Q-Vector length: logical K sharing one E8M0 scale, for W_i and for the 4-bit
 *              activations: 64 or 32.  Both are executed by sdq_linear (64: kind::mxf4 .block32, the
 *              faster kernel; 32: kind::mxf4nvf4 .block16 with E8M0 scale codes).
 *   scale_rule E8M0 exponent from the Q-Vector's largest magnitude a: OCP_FLOOR = floor(log2 a) - 2,
 *              CEIL_NOSAT = smallest E with a <= 6 * 2^E.  SDQ_SCALE_UE4M3 (the quantization-stage study's
 *              preferred scale-factor format, fp8-e4m3): two-level scaling -- a vector (the kept inliers
 *              of a weight row; a token) has a power-of-two factor 2^t, t = smallest integer with its
 *              largest magnitude <= 448 * 2^t (for a token: the exponent of its 8-bit scale); a Q-Vector's
 *              scale code is the unsigned E4M3 value nearest to a / (6 * 2^t) (ties to even, at least the
 *              smallest positive one unless a = 0); an element is the E2M1 value nearest to x / (scale *
 *              2^t).  Requires in_gran = SDQ_GRAN_PAIR and in_block = 32 (kind::mxf4nvf4 .block16 with
 *              UE4M3 scale codes), else every call returns SDQ_ERR_UNSUPPORTED; rows or tokens whose largest
 *              magnitude is below 2^-100 are outside its range.
 */
typedef struct {
  int32_t out_n;
  int32_t in_gran;
  int32_t in_block;
  int32_t scale_rule;
  int32_t out_order;   /* SDQ_ORDER_LARGE (the method) or SDQ_ORDER_SMALL: outliers in ascending order of the
                          metric, the decomposition-stage study's control; sdq_quantize_act ignores it */
  int32_t out_fmt;     /* SDQ_OUT_E4M3, or SDQ_OUT_INT8: the 8-bit operands W_o and A_o in int8 (Section 5.1; the
                          evaluation's "1:8int8" configurations) */
} sdq_config_t;

/* Host-side descriptor of a packed weight matrix (filled by sdq_decompose; plain data, may be
 * copied; `dev` stays owned by the caller).  off[] are byte offsets of the sections inside dev:
 *   0 inlier stages  1 outlier stages (tensor-core 2:4 form)  2 outlier row-scale atoms
 *   3 outlier stages in compact form (8-bit code + position nibble per outlier; tiled configurations; the
 *     decompose-only reading keeps plain code / index arrays at 3 and 4)  4 see 3  5 outlier scale exponents
 *   6 inlier row-factor exponents (SDQ_SCALE_UE4M3; zeros otherwise)  7 reserved */
typedef struct {
  void* dev;
  size_t bytes;
  int64_t N, K;
  sdq_config_t cfg;
  size_t off[8];
} sdq_packed_t;

/* Host-side descriptor of a quantized activation matrix (filled by sdq_quantize_act).
 *   off: 0 activation stages (4-bit codes | 8-bit codes | 4-bit scales per 128-token x 256-K tile)
 *        1 per-token 8-bit scale atoms   2 per-token 8-bit scale exponents   3.. reserved */
typedef struct {
  void* dev;
  size_t bytes;
  int64_t M, K;
  sdq_config_t cfg;
  size_t off[6];
} sdq_act_t;

/* Layout-free copies of the packed arrays, one code per byte, for bit-exact comparison
 * (all pointers: device memory, caller-owned, sizes in elements given beside each field). */
typedef struct {
  uint8_t* in_code;   /* [N][K/2]   E2M1 codes of the kept inlier slots in ascending k
                         (DENSE / KEEP: [N][K], every position; outlier and dropped ones hold +0)                */
  uint8_t* in_meta;   /* [N][K/8] (PAIR) or [N][K/4] (ELEM): i0 | i1<<2, kept indices, ascending
                         (DENSE / KEEP: not written, may be NULL)                                         */
  uint8_t* in_scale;  /* [N][K/in_block] E8M0 codes                                               */
  uint8_t* out_code;  /* [N][K/8][out_n] E4M3 codes                                               */
  uint8_t* out_idx;   /* [N][K/8][out_n] position 0..7 in the S-Vector, ascending                 */
  int32_t* out_sexp;  /* [N] exponent e of the row scale 2^e                                      */
  int32_t* in_texp;   /* [N] SDQ_SCALE_UE4M3: exponent t of the row's inlier factor 2^t (in_scale then
                         holds unsigned E4M3 codes); zeros otherwise; may be NULL                  */
} sdq_canonical_t;

typedef struct {
  uint8_t* xq4_code;  /* [M][K] E2M1 codes           */
  uint8_t* xq4_scale; /* [M][K/in_block] E8M0 codes (SDQ_SCALE_UE4M3: unsigned E4M3 codes, times 2^xq8_sexp[m]) */
  uint8_t* xq8_code;  /* [M][K] E4M3 codes           */
  int32_t* xq8_sexp;  /* [M] exponent e of the per-token scale 2^e */
} sdq_act_canonical_t;

/* Size of the packed-weight buffer for an N x K matrix.  *bytes: what sdq_decompose needs;
 * *algorithmic_bytes: the paper's accounting (Section 3.3: values + one index per non-zero + one
 * scale per Q-Vector), the numerator of the decode GB/s metric.  Either out pointer may be NULL. */
sdq_status_t sdq_packed_size(int64_t N, int64_t K, const sdq_config_t* cfg, size_t* bytes,
                             size_t* algorithmic_bytes);

/* Section 5, Stages 2 -> 1 -> 3 on one weight matrix: per S-Vector of 8 along K take the out_n
 * largest |w| as outliers, prune the rest to the inlier N:M pattern by magnitude, quantize
 * outliers to E4M3 with a per-row power-of-two scale and inliers to E2M1 with an E8M0 scale per
 * Q-Vector, and write codes, scales and sparsity metadata in the tiled layout sdq_linear streams.
 *   W (device) [N][ldw] bf16, ldw >= K elements; packed_buf (device) >= *bytes of sdq_packed_size;
 *   out (host) receives the descriptor.  Enqueues on `stream`, then synchronises that stream once
 *   to read back the non-finite flag.  Errors: INVALID_ARG, SHAPE, ALIGNMENT, BUFFER_TOO_SMALL,
 *   NONFINITE (buffer contents undefined), CUDA. */
sdq_status_t sdq_decompose(const void* W_bf16, int64_t N, int64_t K, int64_t ldw, const sdq_config_t* cfg,
                           void* packed_buf, size_t packed_bytes, sdq_packed_t* out, void* stream);

/* The same decomposition with the weight-activation product as the significance metric (Section 5,
 * Stage 1, calibration-based metrics: a small weight that meets a large activation matters; the
 * decomposition-stage study finds product-based outlier extraction best): the selections -- which
 * out_n values of an S-Vector are outliers and which inlier pairs / elements survive pruning -- rank
 * by |w[n][k]| * col_weight[k] (one fp32 round-to-nearest multiply, largest first, ties to the lower
 * k; a pair's score is the fp32 sum of its two products) instead of |w|.  Values, scales and formats
 * are untouched by the metric.
 *   col_weight (device) [K] fp32, 16-byte aligned, every entry finite and >= 0 -- typically the norm
 *   of input channel k over a calibration set (any per-channel saliency weight fits: an error-based
 *   saliency w^2 / [H^-1]_kk ranks like |w| * c[k] with c[k] = [H^-1]_kk^(-1/2)).  NULL gives sdq_decompose exactly.
 *   Errors as sdq_decompose; a negative, infinite or NaN channel weight reports NONFINITE. */
sdq_status_t sdq_decompose_metric(const void* W_bf16, int64_t N, int64_t K, int64_t ldw, const sdq_config_t* cfg,
                                  const float* col_weight, void* packed_buf, size_t packed_bytes,
                                  sdq_packed_t* out, void* stream);

/* Calibration helper for sdq_decompose_metric (Section 5, Stage 1: metrics that use calibration data):
 * col_norm[k] = sqrt(sum over the M tokens of X[m][k]^2), the Euclidean norm of input channel k, accumulated
 * in token order in fp64 and rounded to fp32 (reproducible).
 *   X (device) [M][ldx] bf16, 4-byte aligned, ldx >= K, K and ldx even; col_norm (device) [K] fp32.
 *   Asynchronous on `stream`.  Errors: INVALID_ARG, SHAPE, ALIGNMENT, CUDA. */
sdq_status_t sdq_channel_norm(const void* X_bf16, int64_t M, int64_t K, int64_t ldx, float* col_norm, void* stream);

/* Untile a packed weight buffer into the canonical arrays (parity surface). Asynchronous. */
sdq_status_t sdq_packed_export(const sdq_packed_t* P, const sdq_canonical_t* out, void* stream);

/* Packed buffers are self-describing: sdq_decompose writes a 256-byte header (magic, layout version, configuration, N,
 * K, total bytes, section offsets) in front of the sections, so a buffer can be saved and restored with plain memcpy
 * (device -> file -> device, or to another process) and turned back into a descriptor without the original weights.
 *   sdq_packed_attach: `dev` (device, 16-byte aligned) holds `bytes` bytes of a packed buffer.  Reads the header
 *   (synchronises `stream`), checks magic, version, configuration, shape and that the recorded section offsets are the
 *   ones this library computes for that configuration and shape, and fills *out.  The buffer stays owned by the caller.
 *   Errors: INVALID_ARG (null pointer), ALIGNMENT, UNSUPPORTED (not a packed buffer of this layout version),
 *   SHAPE (header inconsistent with itself), BUFFER_TOO_SMALL (bytes < the size the header records), CUDA. */
sdq_status_t sdq_packed_attach(const void* dev, size_t bytes, sdq_packed_t* out, void* stream);

/* The packed matrix without its 2:4 outlier containers: inlier records, compact outlier records (8-bit code + position per
 * outlier), scales -- 4.2 instead of 9.1 bits per weight for the 1:8 + 4:8 configuration, i.e. what Section 3.3 counts plus
 * the tensor core's metadata and padding.  This is all the fused few-token kernel of sdq_linear_group / sdq_linear_group_x
 * streams (it rebuilds the containers in tensor memory), so a deployment that only decodes keeps just this form resident;
 * calls that need the containers (sdq_linear and its variants, the layer-by-layer fallback of sdq_linear_group) return
 * SDQ_ERR_UNSUPPORTED for it.  sdq_packed_export, sdq_packed_attach (the header says which form a buffer holds) and the
 * grouped calls accept both forms; off[1] of a compact descriptor is 0.
 *   sdq_packed_compact_size: bytes of the compact form (tiled configurations with out_n >= 1; SDQ_ERR_UNSUPPORTED otherwise).
 *   sdq_packed_compact: copies P's sections into dst (device, 256-byte aligned, >= that many bytes, caller-owned, must not
 *   overlap P->dev), writes its header and fills *out.  Device-to-device copies on `stream`, then one stream
 *   synchronisation; allocates nothing.  P itself is unchanged and may be freed afterwards. */
sdq_status_t sdq_packed_compact_size(int64_t N, int64_t K, const sdq_config_t* cfg, size_t* bytes);
sdq_status_t sdq_packed_compact(const sdq_packed_t* P, void* dst, size_t dst_bytes, sdq_packed_t* out, void* stream);

/* Size of the quantized-activation buffer for M tokens of K features. */
sdq_status_t sdq_act_size(int64_t M, int64_t K, const sdq_config_t* cfg, size_t* bytes);

/* activation quantization (Section 5, Stage 3; A -> A_o, A_i in Section 5.1):
 * per token and Q-Vector an E8M0 scale and E2M1 codes (A_i); per token a power-of-two scale and
 * E4M3 codes (A_o).  X (device) [M][ldx] bf16; xq_buf (device) >= sdq_act_size bytes; out (host).
 * +-Inf saturates, NaN input is undefined.  Asynchronous on `stream`; for K <= 16384 the one kernel it
 * enqueues carries programmatic stream serialization and waits for the previous kernel of the stream
 * before it reads X. */
sdq_status_t sdq_quantize_act(const void* X_bf16, int64_t M, int64_t K, int64_t ldx, const sdq_config_t* cfg,
                              void* xq_buf, size_t xq_bytes, sdq_act_t* out, void* stream);

/* Untile a quantized activation buffer into canonical arrays (parity surface). Asynchronous. */
sdq_status_t sdq_act_export(const sdq_act_t* Xq, const sdq_act_canonical_t* out, void* stream);

/* The decomposed product of Section 5.1, O = O_o + O_i, both sparse products accumulated in fp32 in
 * one accumulator: Y[m][n] = sum_k A_i[m][k] W_i[n][k] + sum_k A_o[m][k] W_o[n][k].
 *   Xq, P (host descriptors; K and cfg must agree); Y (device) [M][ldy] bf16 (round to nearest even
 *   of the fp32 accumulator); ldy >= N elements, ldy % 8 == 0.  Asynchronous on `stream`.
 *   The kernel is enqueued with programmatic stream serialization: it may begin (set-up, reading the packed
 *   weights) while the previous kernel of the stream is still finishing, and waits for that kernel before it
 *   reads Xq or writes Y.  The packed weights must therefore be complete before the call is enqueued
 *   (sdq_decompose synchronises its stream, so a buffer it returned always is).
 *   Errors: INVALID_ARG, SHAPE, ALIGNMENT, UNSUPPORTED (in_gran == ELEM with in_block == 64), CUDA. */
sdq_status_t sdq_linear(const sdq_act_t* Xq, const sdq_packed_t* P, void* Y_bf16, int64_t ldy, void* stream);

/* Same product, storing the fp32 accumulator itself (the value the bf16 output is rounded from). */
sdq_status_t sdq_linear_f32(const sdq_act_t* Xq, const sdq_packed_t* P, float* Y_f32, int64_t ldy, void* stream);

/* The same product with a caller-owned scratch buffer (device).  With few tokens (M <= 128) a weight row
 * tile has too little work for one thread block per SM, so the K range of every row tile is split over
 * several blocks; each writes an fp32 partial tile to the workspace and the last one to arrive adds them in
 * split order, so the result does not depend on timing (O = O_o + O_i of Section 5.1 is unchanged; only the
 * summation over K is regrouped, hence Y may differ from sdq_linear in the last fp32 bits).
 *   sdq_workspace_size: bytes needed for (M, N, K) on the current device (0 when no split would be used).
 *   sdq_workspace_init: zeroes a workspace once after allocation (asynchronous); calls leave it zeroed.  A call that
 *   ended with SDQ_ERR_TIMEOUT (sdq_device_status) or SDQ_ERR_CUDA may leave arrival counters behind: initialise the
 *   workspace again before it is reused, or the next call adds incomplete partial tiles.
 *   A workspace must not be shared by calls that can overlap on the GPU.  ws may be NULL (no split).
 *   Errors as sdq_linear, plus BUFFER_TOO_SMALL. */
sdq_status_t sdq_workspace_size(int64_t M, int64_t N, int64_t K, const sdq_config_t* cfg, size_t* bytes);
sdq_status_t sdq_workspace_init(void* ws, size_t ws_bytes, void* stream);
sdq_status_t sdq_linear_ws(const sdq_act_t* Xq, const sdq_packed_t* P, void* Y_bf16, int64_t ldy, void* ws, size_t ws_bytes,
                           void* stream);
sdq_status_t sdq_linear_f32_ws(const sdq_act_t* Xq, const sdq_packed_t* P, float* Y_f32, int64_t ldy, void* ws, size_t ws_bytes,
                               void* stream);

/* Several independent layers in one call: Y[i] = A_i,in W_i,in^T + A_i,out W_i,out^T for i = 0 .. n - 1
 * (Section 5.1, O = O_i + O_o, once per layer; Section 5, Stage 3 supplies each layer's quantized operands).  The
 * layers must not depend on one another (q / k / v projections or gate / up, which may share one Xq; the layers of a
 * benchmark rotation): they may run in any order and concurrently.
 *   Xq, P, Y, ldy: host arrays of n entries (descriptors and pointers as for sdq_linear; the arrays themselves are read
 *   during the call only).  Outputs must not overlap.
 *   When every layer has at most 32 tokens, K >= 1024, the primary format (SDQ_GRAN_PAIR, in_block 64, out_n <= 1,
 *   power-of-two scales), n <= 32 and the layers together have at least half as many 128-row tiles as the GPU has SMs, the
 *   call is ONE persistent kernel launch that streams all weights once, the outlier part in its compact form (8-bit code +
 *   position per S-Vector, rebuilt into the tensor core's 2:4 form in tensor memory); the summation order over K of an output differs
 *   from sdq_linear's split-K paths, so results agree to fp32 rounding, not bit for bit.  Otherwise the layers are
 *   enqueued one after the other exactly as sdq_linear would.
 *   Asynchronous on `stream`; allocates nothing.  Errors as sdq_linear (the first failing layer's). */
sdq_status_t sdq_linear_group(int n, const sdq_act_t* const* Xq, const sdq_packed_t* const* P, void* const* Y_bf16,
                              const int64_t* ldy, void* stream);
sdq_status_t sdq_linear_group_f32(int n, const sdq_act_t* const* Xq, const sdq_packed_t* const* P, float* const* Y_f32,
                                  const int64_t* ldy, void* stream);

/* sdq_linear_group with the activation quantization inside the kernel (Section 5, Stage 3 fused into the linear layers'
 * load path): Y_i = Q(X) W_i,in^T + Q'(X) W_i,out^T for n independent layers that read the SAME activations -- q / k / v, or
 * gate / up, of a few tokens.
 *   X_bf16: device, [M][K] bf16, row stride ldx elements (16-byte aligned, ldx % 8 == 0), M <= 16.  Every CTA of the one
 *   persistent launch quantizes X into its own shared memory (the codes, scales and arithmetic of sdq_quantize_act, so
 *   the results are bit-identical to sdq_quantize_act followed by sdq_linear_group) while the first weights stream in;
 *   no quantized buffer exists in device memory and no second kernel runs.
 *   P, Y, ldy as for sdq_linear_group; every P[i]->K == K.  The 8-bit format of A_o is the weights' (cfg.out_fmt).
 *   Range: the fused kernel's (primary format, out_n <= 1, power-of-two scales, n <= 32, at least half as many 128-row
 *   tiles as SMs) with 1024 <= K <= 4096 (X has to fit beside the weight ring); outside it the call returns
 *   SDQ_ERR_UNSUPPORTED and launches nothing: quantize with sdq_quantize_act and use sdq_linear_group then.
 *   Asynchronous on `stream`; allocates nothing. */
sdq_status_t sdq_linear_group_x(int n, const void* X_bf16, int64_t M, int64_t K, int64_t ldx, const sdq_packed_t* const* P,
                                void* const* Y_bf16, const int64_t* ldy, void* stream);
sdq_status_t sdq_linear_group_x_f32(int n, const void* X_bf16, int64_t M, int64_t K, int64_t ldx, const sdq_packed_t* const* P,
                                    float* const* Y_f32, const int64_t* ldy, void* stream);

/* Built-in scratch variant of sdq_linear_ws (the paper has no counterpart: this is a packaging choice of the
 * library, not part of the method).
 *   For callers that hold nothing but their input and output pointers and cannot obtain device memory: a
 *   plug-in running inside someone else's inference server whose memory pool was handed out at start-up, a
 *   host thread on a latency path where a device allocation (which may synchronise the whole device) is not
 *   acceptable, or any caller that must not call cudaMalloc.  The split-K scratch is a fixed array of
 *   SDQ_STATIC_WS_BYTES inside the library's device image; every GPU that loads the library carries it until
 *   the process exits.  The call allocates and frees nothing.
 *   Same arguments, result and errors as sdq_linear; the result equals sdq_linear_ws with a caller workspace
 *   bit for bit.  Shapes whose scratch need (sdq_workspace_size) exceeds SDQ_STATIC_WS_BYTES are refused with
 *   SDQ_ERR_BUFFER_TOO_SMALL; shapes that need no scratch run as sdq_linear.
 *   The first call on each device looks up the device address of the array (cudaGetSymbolAddress with that
 *   device current); make that first call before any stream capture begins.  All calls on a device share the
 *   one array and it keeps the previous call's contents (the counters are cleared on the stream at the start of
 *   every call): two calls that can overlap on the GPU (different streams) race on it -- serialise them or use
 *   sdq_linear_ws with separate workspaces. */
#define SDQ_STATIC_WS_BYTES (4u << 20)
sdq_status_t sdq_linear_noalloc(const sdq_act_t* Xq, const sdq_packed_t* P, void* Y_bf16, int64_t ldy, void* stream);

/* Synchronises `stream` and returns the sticky device-side status (SDQ_OK or SDQ_ERR_TIMEOUT when a
 * bounded wait inside a kernel gave up), clearing it. */
sdq_status_t sdq_device_status(void* stream);

const char* sdq_status_string(sdq_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* SDQ_H_ */
