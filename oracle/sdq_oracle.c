/*
 * SDQ oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, obviously-correct CPU statement of what the SDQ decomposed linear layer computes
 * (arXiv 2406.13868, Section 5: Stage 1 sparsification, Stage 2 decomposition, Stage 3
 * quantization, and the "LLM inference performance" paragraph O = O_o + O_i).  It shares no code,
 * header, table or helper with the CUDA library; only tests, the smoke check and the CPU-baseline
 * leg of the benchmark may call it.
 *
 * Everything is written in the order and notation of the paper's stages:
 *   W  --(local N:M outlier extraction per S-Vector of 8 along K)-->  W_o  (outliers, 8-bit float)
 *      --(N:M magnitude pruning of the remaining values)          -->  W_i  (inliers, 4-bit float)
 *   A  --> A_o (8-bit float), A_i (4-bit float with per-Q-Vector power-of-two scale)
 *   O  = A_o * W_o^T + A_i * W_i^T                     accumulated in fp64
 *
 * Number formats are decoded/encoded by exhaustive nearest-value search over the list of
 * representable values in fp64 -- no bit tricks -- so that the rounding rule is visible:
 * round to nearest, ties to the code whose last bit is 0, saturate at the largest finite value.
 *
 * Pins (tests/ -m "not gpu"): exhaustive codec checks against closed forms and torch CPU casts,
 * N:M invariants from the paper, brute force over all C(8,n) selections, an independent dense
 * "definition" of the decomposition, brute-force matmul, one-hot read-back, exact power-of-two
 * scaling, the paper's printed bits-per-weight / throughput arithmetic, and for the E4M3 scale rule closed forms at every
 * representable scale and midpoint plus an independent definition built on torch's float8 cast.
 * The int8 outlier format is pinned by closed forms (codes of k * amax / 127 are k, the half-way points go to the even
 * integer, nothing exceeds 127), by numpy's own fp32 division and rint on random rows, and by a product that must equal an
 * exact integer matrix product times the two scales.
 * Parity unpinned: none of the functions in this file (model-quality numbers of the paper are not
 * computed here at all).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define SDQO_GRAN_PAIR 0 /* inlier pattern: keep 2 of the 4 adjacent pairs in every 8 (pair-wise 4:8) */
#define SDQO_GRAN_ELEM 1 /* inlier pattern: keep 2 of every 4 elements (element-wise 2:4)            */
#define SDQO_GRAN_DENSE 2 /* no Stage 1: every non-outlier value stays an inlier (8:8 = out_n:8 + (8-out_n):8) */
/* Stage 1 keeps the n most significant values of every S-Vector of 8 (n:8 sparsification, n = 2..8), of which out_n
   become outliers and n - out_n stay inliers at whatever positions they have (the paper's flexible N:M patterns, e.g.
   7:8 = 1:8 + 6:8); stored like the dense pattern, the dropped positions holding +0.  KEEP(8) is DENSE. */
#define SDQO_GRAN_KEEP(n) (2 + (8 - (n)))
/* S-Vectors of 4 (the evaluation's 3:4 = 1:4 + 2:4 configuration): Stage 1 keeps the 3 most significant of every 4,
   Stage 2 takes the most significant of every 4 as the outlier (out_n = 2 per 8 consecutive K; out_n = 0: none), the
   others stay inliers at whatever positions they have; stored like the dense pattern. */
#define SDQO_GRAN_3OF4 9
/* Stage 2 order (decomposition-stage study): "Large" takes the most significant values as outliers (the method),
   "Small" the least significant ones (the study's control: the wrong values in high precision) */
#define SDQO_ORDER_LARGE 0
#define SDQO_ORDER_SMALL 1
#define SDQO_SCALE_OCP_FLOOR 0  /* E = floor(log2 amax) - 2   (OCP MX rule, may saturate in (6,8)) */
#define SDQO_SCALE_CEIL_NOSAT 1 /* E = smallest integer with amax <= 6 * 2^E                        */
/* Two-level scaling with 8-bit floating-point Q-Vector scales (the quantization-stage study: scale factors in
   fp8-e4m3 work best): a vector (the kept inliers of a weight row, or a token) gets a power-of-two factor 2^t,
   t = the exponent of its 8-bit scale (smallest t with amax <= 448 * 2^t); a Q-Vector gets the unsigned E4M3 scale
   nearest to amax_q / (6 * 2^t) (ties to the even code; never below the smallest positive one unless the Q-Vector is
   all zero); an element is the E2M1 value nearest to x / (scale * 2^t), ties to even, saturating at 6. */
#define SDQO_SCALE_UE4M3 2
/* 8-bit format of the outlier operands W_o and A_o: E4M3 with a power-of-two scale per weight row / token, or the
   evaluation's int8 (Section 6 configuration names "1:8int8"; Section 5.1: "quantize 1:8 W_o as int8 ... A would be
   quantized to int8 A_o"): symmetric, one fp32 scale per weight row / token */
#define SDQO_OUT_E4M3 0
#define SDQO_OUT_INT8 1

typedef struct {
  int out_n;      /* outliers kept per S-Vector of 8 along K: 0, 1 or 2          */
  int in_gran;    /* SDQO_GRAN_*                                                */
  int in_block;   /* Q-Vector: logical K per inlier / 4-bit activation scale (32|64) */
  int scale_rule; /* SDQO_SCALE_*                                               */
  int out_order;  /* SDQO_ORDER_*: which end of the metric's order Stage 2 takes     */
  int out_fmt;    /* SDQO_OUT_*: 8-bit format of W_o and A_o                          */
} sdqo_config;

/* ------------------------------------------------------------------ number formats */

/* bf16 bit pattern -> value (bf16 is the upper half of an IEEE fp32) */
double sdqo_bf16_to_double(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* E2M1: 1 sign, 2 exponent (bias 1), 1 mantissa bit. Magnitudes by code 0..7. */
static const double E2M1_MAG[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};

double sdqo_e2m1_decode(uint8_t code) {
  double m = E2M1_MAG[code & 7];
  return (code & 8) ? -m : m;
}

/* E4M3 (OCP "FN" flavour): 1 sign, 4 exponent (bias 7), 3 mantissa; no infinity; magnitude codes
 * 0x00..0x7E are finite (0x7F is NaN); largest finite value 448. */
static double e4m3_mag(int mcode) {
  int e = (mcode >> 3) & 15, m = mcode & 7;
  if (e == 0) return ldexp((double)m / 8.0, -6);   /* subnormals: m/8 * 2^-6 */
  return ldexp(1.0 + (double)m / 8.0, e - 7);
}

double sdqo_e4m3_decode(uint8_t code) {
  double m = e4m3_mag(code & 0x7F);
  return (code & 0x80) ? -m : m;
}

/* E8M0: value 2^(code-127); code 255 (NaN) never produced here. */
double sdqo_e8m0_decode(uint8_t code) { return ldexp(1.0, (int)code - 127); }

/* nearest representable magnitude among n_codes ascending magnitudes; ties -> even code;
 * anything above the largest magnitude saturates to it. */
static int nearest_code(double a, int n_codes, double (*mag)(int)) {
  if (a >= mag(n_codes - 1)) return n_codes - 1;   /* saturate (also keeps huge inputs away from the tie rule) */
  int best = 0;
  double best_d = fabs(a - mag(0));
  for (int c = 1; c < n_codes; ++c) {
    double d = fabs(a - mag(c));
    if (d < best_d || (d == best_d && (c & 1) == 0)) { best = c; best_d = d; }
  }
  return best;
}
static double e2m1_mag_fn(int c) { return E2M1_MAG[c]; }

/* sign of v is kept even when the magnitude rounds to zero (so -0 encodes as 0x8 / 0x80) */
uint8_t sdqo_e2m1_encode(double v) {
  int c = nearest_code(fabs(v), 8, e2m1_mag_fn);
  return (uint8_t)(c | (signbit(v) ? 8 : 0));
}
uint8_t sdqo_e4m3_encode(double v) {
  int c = nearest_code(fabs(v), 127, e4m3_mag);
  return (uint8_t)(c | (signbit(v) ? 0x80 : 0));
}

/* smallest integer e with amax <= vmax * 2^e ; amax == 0 -> 0 */
static int ceil_exp(double amax, double vmax) {
  if (amax == 0.0) return 0;
  int e = -200;
  while (amax > ldexp(vmax, e)) ++e;
  return e;
}
/* floor(log2 amax) for amax > 0 */
static int floor_log2(double amax) {
  int e = -200;
  while (ldexp(1.0, e + 1) <= amax) ++e;
  return e;
}

/* E8M0 code of the Q-Vector scale for 4-bit values whose largest magnitude is amax */
uint8_t sdqo_e8m0_scale_code(double amax, int scale_rule) {
  if (amax == 0.0) return 0;
  int E = (scale_rule == SDQO_SCALE_OCP_FLOOR) ? floor_log2(amax) - 2 : ceil_exp(amax, 6.0);
  int c = E + 127;
  if (c < 0) c = 0;
  if (c > 254) c = 254;
  return (uint8_t)c;
}

/* exponent e of the power-of-two scale 2^e used for 8-bit (E4M3) operands: nothing saturates.
 * The scale must be expressible as an E8M0 byte (code e + 127 in 0..254), so e is limited to
 * [-127, 127]; only rows whose largest magnitude is below 448 * 2^-127 are affected. */
int sdqo_fp8_scale_exp(double amax) {
  int e = ceil_exp(amax, 448.0);
  if (e < -127) e = -127;
  if (e > 127) e = 127;
  return e;
}

/* int8 operands: scale s = amax / 127 (amax = 0: s = 1) and code = the integer nearest to x / s, ties to the even
 * integer, limited to [-127, 127].  The scale is not a power of two, so x / s rounds; both the scale and the quotient
 * are formed in fp32 (one IEEE division each, round to nearest even), the precision in which the code is decided.
 * x is a bf16 value (exact in fp32).  The scale is handed on as its fp32 bit pattern. */
float sdqo_int8_scale(double amax) { return amax == 0.0 ? 1.0f : (float)amax / 127.0f; }
int8_t sdqo_int8_encode(double x, float s) {
  volatile float q = (float)x / s;   /* fp32 quotient (volatile: no wider intermediate) */
  float r = nearbyintf(q);           /* default rounding mode: to nearest, ties to even */
  if (r > 127.0f) r = 127.0f;
  if (r < -127.0f) r = -127.0f;
  return (int8_t)r;
}
static int32_t float_bits(float f) { int32_t u; memcpy(&u, &f, 4); return u; }
static float bits_float(int32_t u) { float f; memcpy(&f, &u, 4); return f; }
/* value of an 8-bit operand code under the configuration's format; sexp = the exponent of the power-of-two scale
 * (E4M3) or the bit pattern of the fp32 scale (int8) */
static double out_value(const sdqo_config* cfg, uint8_t code, int32_t sexp) {
  if (cfg->out_fmt == SDQO_OUT_INT8) return (double)(int8_t)code * (double)bits_float(sexp);
  return ldexp(sdqo_e4m3_decode(code), sexp);
}

/* unsigned-E4M3 code (0x00..0x7E) of a Q-Vector scale under SDQO_SCALE_UE4M3, and the scaled E2M1 code of an element */
uint8_t sdqo_ue4m3_scale_code(double amax_q, int t) {
  if (amax_q == 0.0) return 0;
  uint8_t c = sdqo_e4m3_encode(ldexp(amax_q, -t) / 6.0);
  return c == 0 ? 1 : c;
}
static uint8_t e2m1_of_quotient(double x, uint8_t scale_code, int t) {
  if (scale_code == 0) return 0;
  return sdqo_e2m1_encode(x / ldexp(sdqo_e4m3_decode(scale_code), t));
}

/* magnitude key used by every "largest" selection: the 15 low bits of the bf16 pattern */

static int is_finite_bf16(uint16_t h) { return (h & 0x7F80) != 0x7F80; }

/* ------------------------------------------------------------------ Stage 2 + 1 + 3 on one weight matrix
 *
 * W        [N][K] bf16 bit patterns, row-major (row = output feature, K contiguous)
 * Canonical outputs, one code per byte (layout-free parity surface):
 *   in_code  [N][K/2]      E2M1 codes of the kept inlier slots in ascending k   (DENSE / KEEP(n): [N][K], every position)
 *   in_meta  [N][K/8] (PAIR: j0 | j1<<2, kept pair indices 0..3 of the group of 8)
 *            [N][K/4] (ELEM: i0 | i1<<2, kept element indices 0..3 of the group of 4)
 *            not touched for DENSE / KEEP(n) (dropped and outlier positions simply hold +0)
 *   in_scale [N][K/in_block] E8M0 code (SDQO_SCALE_UE4M3: unsigned E4M3 code, times 2^in_texp[n])
 *   in_texp  [N]           SDQO_SCALE_UE4M3: exponent t of the row's power-of-two factor (int32); else 0 (may be NULL)
 *   out_code [N][K/8][out_n] E4M3 codes; out_idx same shape, position 0..7 inside the group, ascending
 *   out_sexp [N]           e of the per-row outlier scale 2^e (int32); SDQO_OUT_INT8: out_code holds int8 codes and
 *                          out_sexp the bit pattern of the row's fp32 scale
 * returns 0, or -1 on a bad argument, -2 if W holds a non-finite value.
 */
/* Significance of element k of a row for the selections of Stage 2 (which values are outliers) and Stage 1 (which
   values survive pruning).  Without a channel weight it is the magnitude |w| (Section 5, Stage 1: "the most
   straightforward metric is magnitude").  With one it is the weight-activation product |w| * c[k], c[k] being a
   per-input-channel activation norm from calibration (Section 5, Stage 1 / Stage 2 and the decomposition-stage
   sensitivity study: product-based outlier extraction, outliers taken in descending order).  The product is ONE
   fp32 round-to-nearest multiply so that any implementation can reproduce the order exactly; with c == 1 it is |w|. */
static float significance(uint16_t w, const float* col_weight, int64_t k) {
  const float a = (float)fabs(sdqo_bf16_to_double(w));
  if (!col_weight) return a;
  volatile float p = a * col_weight[k];
  return p;
}

int sdqo_decompose_metric(const uint16_t* W, int64_t N, int64_t K, const sdqo_config* cfg, const float* col_weight,
                          uint8_t* in_code, uint8_t* in_meta, uint8_t* in_scale,
                          uint8_t* out_code, uint8_t* out_idx, int32_t* out_sexp, int32_t* in_texp) {
  if (!W || !cfg || N <= 0 || K <= 0 || K % 64 != 0) return -1;
  if (col_weight)
    for (int64_t k = 0; k < K; ++k)
      if (!(col_weight[k] >= 0.0f) || isinf(col_weight[k])) return -3;
  if (cfg->out_n < 0 || cfg->out_n > 2) return -1;
  if (cfg->out_order != SDQO_ORDER_LARGE && cfg->out_order != SDQO_ORDER_SMALL) return -1;
  if (cfg->out_fmt != SDQO_OUT_E4M3 && cfg->out_fmt != SDQO_OUT_INT8) return -1;
  if (cfg->in_block != 32 && cfg->in_block != 64) return -1;
  if (cfg->scale_rule < 0 || cfg->scale_rule > SDQO_SCALE_UE4M3 || (cfg->scale_rule == SDQO_SCALE_UE4M3 && !in_texp)) return -1;
  if (cfg->in_gran < 0 || cfg->in_gran > SDQO_GRAN_3OF4) return -1;
  /* S-Vector length, values that survive Stage 1 per S-Vector (meaningful from DENSE on), outliers per S-Vector */
  const int sv = cfg->in_gran == SDQO_GRAN_3OF4 ? 4 : 8;
  const int keep_n = cfg->in_gran == SDQO_GRAN_3OF4 ? 3 : 10 - cfg->in_gran;
  if (cfg->in_gran == SDQO_GRAN_3OF4 && cfg->out_n == 1) return -1;    /* one outlier per 4 is two per 8 */
  const int on_sv = cfg->out_n * sv / 8;
  if (cfg->in_gran >= SDQO_GRAN_DENSE && keep_n <= on_sv) return -1;
  const int on = cfg->out_n, Bs = cfg->in_block;
  const int64_t G8 = K / 8;
  const int64_t slots = cfg->in_gran >= SDQO_GRAN_DENSE ? K : K / 2;   /* inlier slots per row */
  for (int64_t i = 0; i < N * K; ++i)
    if (!is_finite_bf16(W[i])) return -2;

  uint8_t* is_out = (uint8_t*)malloc((size_t)K);   /* 1 where the element went to W_o            */
  uint8_t* kept = (uint8_t*)malloc((size_t)K);     /* 1 where the element is a kept inlier SLOT  */
  uint8_t* dropped = (uint8_t*)malloc((size_t)K);  /* KEEP(n): 1 where Stage 1 removed the value (its slot holds +0) */
  float* sig = (float*)malloc((size_t)K * sizeof(float));
  for (int64_t n = 0; n < N; ++n) {
    const uint16_t* w = W + n * K;
    memset(is_out, 0, (size_t)K);
    memset(kept, 0, (size_t)K);
    memset(dropped, 0, (size_t)K);
    for (int64_t k = 0; k < K; ++k) sig[k] = significance(w[k], col_weight, k);

    /* Stage 2, local outlier extraction: the most significant values of every S-Vector (out_n of 8; with S-Vectors of
       4, one of 4), largest first, ties to the lower index */
    double out_amax = 0.0;
    for (int64_t g = 0; g < G8; ++g) {
      int chosen[2] = {-1, -1};
      int nc = 0;
      for (int sub = 0; sub < 8 / sv; ++sub)
        for (int t = 0; t < on_sv; ++t) {
          int best = -1;
          for (int i = sub * sv; i < (sub + 1) * sv; ++i) {
            if (is_out[8 * g + i]) continue;
            if (best < 0 || (cfg->out_order == SDQO_ORDER_SMALL ? sig[8 * g + i] < sig[8 * g + best]
                                                                : sig[8 * g + i] > sig[8 * g + best])) best = i;
          }
          is_out[8 * g + best] = 1;
          chosen[nc++] = best;
        }
      if (nc == 2 && chosen[0] > chosen[1]) { int t = chosen[0]; chosen[0] = chosen[1]; chosen[1] = t; }
      for (int t = 0; t < on; ++t) {
        out_idx[(n * G8 + g) * on + t] = (uint8_t)chosen[t];
        double a = fabs(sdqo_bf16_to_double(w[8 * g + chosen[t]]));
        if (a > out_amax) out_amax = a;
      }
    }
    /* Stage 3 for outliers: per-row power-of-two scale, E4M3 codes of w / 2^e -- or int8 codes of w / s, s = amax / 127 */
    if (cfg->out_fmt == SDQO_OUT_INT8) {
      const float sw = sdqo_int8_scale(out_amax);
      out_sexp[n] = float_bits(sw);
      for (int64_t g = 0; g < G8; ++g)
        for (int t = 0; t < on; ++t) {
          int i = out_idx[(n * G8 + g) * on + t];
          out_code[(n * G8 + g) * on + t] = (uint8_t)sdqo_int8_encode(sdqo_bf16_to_double(w[8 * g + i]), sw);
        }
    } else {
      const int e = sdqo_fp8_scale_exp(out_amax);
      out_sexp[n] = e;
      for (int64_t g = 0; g < G8; ++g)
        for (int t = 0; t < on; ++t) {
          int i = out_idx[(n * G8 + g) * on + t];
          out_code[(n * G8 + g) * on + t] = sdqo_e4m3_encode(ldexp(sdqo_bf16_to_double(w[8 * g + i]), -e));
        }
    }

    /* Stage 1 on the remaining values: N:M pruning by significance.  The dense configuration
       (Section 5, decomposition-stage study: 8:8 split as 1:8 outliers + 7:8 inliers) skips it. */
    if (cfg->in_gran >= SDQO_GRAN_DENSE) {
      /* n:8 sparsification then out_n:8 outlier extraction with one metric: the outliers are the out_n most
         significant of the 8, the inliers the next n - out_n (largest first, ties to the lower index), the rest is
         dropped -- in whichever order the two stages run.  Every position is a slot. */
      memset(kept, 1, (size_t)K);
      for (int64_t g = 0; g < G8; ++g) {
        uint8_t chosen[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        for (int sub = 0; sub < 8 / sv; ++sub)
          for (int t = 0; t < keep_n - on_sv; ++t) {
            int best = -1;
            for (int i = sub * sv; i < (sub + 1) * sv; ++i) {
              if (is_out[8 * g + i] || chosen[i]) continue;
              if (best < 0 || sig[8 * g + i] > sig[8 * g + best]) best = i;
            }
            chosen[best] = 1;
          }
        for (int i = 0; i < 8; ++i) dropped[8 * g + i] = (uint8_t)(!is_out[8 * g + i] && !chosen[i]);
      }
    } else if (cfg->in_gran == SDQO_GRAN_PAIR) {
      for (int64_t g = 0; g < G8; ++g) {
        float score[4];
        for (int j = 0; j < 4; ++j) {
          float a0 = is_out[8 * g + 2 * j] ? 0.0f : sig[8 * g + 2 * j];
          float a1 = is_out[8 * g + 2 * j + 1] ? 0.0f : sig[8 * g + 2 * j + 1];
          volatile float s = a0 + a1;             /* one fp32 round-to-nearest add */
          score[j] = s;
        }
        int j0 = -1, j1 = -1;
        for (int j = 0; j < 4; ++j) if (j0 < 0 || score[j] > score[j0]) j0 = j;
        for (int j = 0; j < 4; ++j) if (j != j0 && (j1 < 0 || score[j] > score[j1])) j1 = j;
        if (j0 > j1) { int t = j0; j0 = j1; j1 = t; }
        in_meta[n * G8 + g] = (uint8_t)(j0 | (j1 << 2));
        kept[8 * g + 2 * j0] = kept[8 * g + 2 * j0 + 1] = 1;
        kept[8 * g + 2 * j1] = kept[8 * g + 2 * j1 + 1] = 1;
      }
    } else {
      for (int64_t h = 0; h < K / 4; ++h) {
        int i0 = -1, i1 = -1;
        for (int i = 0; i < 4; ++i) {
          if (is_out[4 * h + i]) continue;
          if (i0 < 0 || sig[4 * h + i] > sig[4 * h + i0]) i0 = i;
        }
        for (int i = 0; i < 4; ++i) {
          if (is_out[4 * h + i] || i == i0) continue;
          if (i1 < 0 || sig[4 * h + i] > sig[4 * h + i1]) i1 = i;
        }
        if (i0 > i1) { int t = i0; i0 = i1; i1 = t; }
        in_meta[n * (K / 4) + h] = (uint8_t)(i0 | (i1 << 2));
        kept[4 * h + i0] = kept[4 * h + i1] = 1;
      }
    }

    /* Stage 3 for inliers: per Q-Vector E8M0 scale over the kept inlier values, then E2M1 codes.
       A kept slot that holds an outlier position carries the value +0. */
    const int ue = cfg->scale_rule == SDQO_SCALE_UE4M3;
    int t = 0;                                   /* two-level scaling: the row's power-of-two factor */
    if (ue) {
      double row_amax = 0.0;
      for (int64_t k = 0; k < K; ++k)
        if (kept[k] && !is_out[k] && !dropped[k]) {
          double a = fabs(sdqo_bf16_to_double(w[k]));
          if (a > row_amax) row_amax = a;
        }
      t = sdqo_fp8_scale_exp(row_amax);
    }
    if (in_texp) in_texp[n] = t;
    for (int64_t b = 0; b < K / Bs; ++b) {
      double amax = 0.0;
      for (int64_t k = b * Bs; k < (b + 1) * Bs; ++k)
        if (kept[k] && !is_out[k] && !dropped[k]) {
          double a = fabs(sdqo_bf16_to_double(w[k]));
          if (a > amax) amax = a;
        }
      in_scale[n * (K / Bs) + b] = ue ? sdqo_ue4m3_scale_code(amax, t) : sdqo_e8m0_scale_code(amax, cfg->scale_rule);
    }
    int64_t slot = 0;
    for (int64_t k = 0; k < K; ++k) {
      if (!kept[k]) continue;
      uint8_t code = 0;
      if (!is_out[k] && !dropped[k]) {
        int c = in_scale[n * (K / Bs) + k / Bs];
        code = ue ? e2m1_of_quotient(sdqo_bf16_to_double(w[k]), (uint8_t)c, t)
                  : sdqo_e2m1_encode(ldexp(sdqo_bf16_to_double(w[k]), 127 - c));
      }
      in_code[n * slots + slot++] = code;
    }
  }
  free(is_out);
  free(kept);
  free(dropped);
  free(sig);
  return 0;
}

/* magnitude metric: the decomposition of Section 5 with |w| as the significance */
int sdqo_decompose(const uint16_t* W, int64_t N, int64_t K, const sdqo_config* cfg,
                   uint8_t* in_code, uint8_t* in_meta, uint8_t* in_scale,
                   uint8_t* out_code, uint8_t* out_idx, int32_t* out_sexp, int32_t* in_texp) {
  return sdqo_decompose_metric(W, N, K, cfg, (const float*)0, in_code, in_meta, in_scale, out_code, out_idx, out_sexp, in_texp);
}

/* value of a Q-Vector scale code: E8M0, or unsigned E4M3 times the vector's power-of-two factor 2^t */
static double scale_value(const sdqo_config* cfg, uint8_t code, int t) {
  return cfg->scale_rule == SDQO_SCALE_UE4M3 ? ldexp(sdqo_e4m3_decode(code), t) : sdqo_e8m0_decode(code);
}

/* Dequantize the canonical arrays of ONE weight matrix back to dense W_i and W_o (fp64, [N][K]).
   in_texp [N]: the rows' power-of-two factors (read under SDQO_SCALE_UE4M3 only). */
int sdqo_dequant_weights(int64_t N, int64_t K, const sdqo_config* cfg,
                         const uint8_t* in_code, const uint8_t* in_meta, const uint8_t* in_scale,
                         const uint8_t* out_code, const uint8_t* out_idx, const int32_t* out_sexp, const int32_t* in_texp,
                         double* W_in, double* W_out) {
  const int on = cfg->out_n, Bs = cfg->in_block;
  const int64_t G8 = K / 8;
  memset(W_in, 0, sizeof(double) * (size_t)(N * K));
  memset(W_out, 0, sizeof(double) * (size_t)(N * K));
  for (int64_t n = 0; n < N; ++n) {
    int64_t slot = 0;
    if (cfg->in_gran >= SDQO_GRAN_DENSE) {
      for (int64_t k = 0; k < K; ++k)
        W_in[n * K + k] = sdqo_e2m1_decode(in_code[n * K + k]) * scale_value(cfg, in_scale[n * (K / Bs) + k / Bs], in_texp ? in_texp[n] : 0);
    } else if (cfg->in_gran == SDQO_GRAN_PAIR) {
      for (int64_t g = 0; g < G8; ++g) {
        int nib = in_meta[n * G8 + g];
        int jj[2] = {nib & 3, (nib >> 2) & 3};
        for (int t = 0; t < 2; ++t)
          for (int u = 0; u < 2; ++u) {
            int64_t k = 8 * g + 2 * jj[t] + u;
            W_in[n * K + k] = sdqo_e2m1_decode(in_code[n * (K / 2) + slot++]) *
                              scale_value(cfg, in_scale[n * (K / Bs) + k / Bs], in_texp ? in_texp[n] : 0);
          }
      }
    } else {
      for (int64_t h = 0; h < K / 4; ++h) {
        int nib = in_meta[n * (K / 4) + h];
        int ii[2] = {nib & 3, (nib >> 2) & 3};
        for (int t = 0; t < 2; ++t) {
          int64_t k = 4 * h + ii[t];
          W_in[n * K + k] = sdqo_e2m1_decode(in_code[n * (K / 2) + slot++]) *
                            scale_value(cfg, in_scale[n * (K / Bs) + k / Bs], in_texp ? in_texp[n] : 0);
        }
      }
    }
    for (int64_t g = 0; g < G8; ++g)
      for (int t = 0; t < on; ++t) {
        int64_t k = 8 * g + out_idx[(n * G8 + g) * on + t];
        W_out[n * K + k] = out_value(cfg, out_code[(n * G8 + g) * on + t], out_sexp[n]);
      }
  }
  return 0;
}

/* ------------------------------------------------------------------ activations: A -> A_i (4-bit), A_o (8-bit)
 * X [M][K] bf16 patterns.  xq4_code [M][K] E2M1 codes, xq4_scale [M][K/in_block] E8M0 codes (SDQO_SCALE_UE4M3:
 * unsigned E4M3 codes; the Q-Vector scale is then that value times 2^xq8_sexp[m]),
 * xq8_code [M][K] E4M3 codes, xq8_sexp [M] exponent e of the per-token scale 2^e (SDQO_OUT_INT8: int8 codes and the bit
 * pattern of the token's fp32 scale amax / 127; not combined with SDQO_SCALE_UE4M3, whose 4-bit scales hang on e).
 * +-Inf saturates to the largest finite value; NaN is rejected (-2). */
int sdqo_quantize_act(const uint16_t* X, int64_t M, int64_t K, const sdqo_config* cfg,
                      uint8_t* xq4_code, uint8_t* xq4_scale, uint8_t* xq8_code, int32_t* xq8_sexp) {
  if (!X || !cfg || M <= 0 || K <= 0) return -1;
  if (cfg->in_block != 32 && cfg->in_block != 64) return -1;
  if (cfg->scale_rule < 0 || cfg->scale_rule > SDQO_SCALE_UE4M3) return -1;
  if (K % cfg->in_block != 0) return -1;
  if (cfg->out_fmt != SDQO_OUT_E4M3 && (cfg->out_fmt != SDQO_OUT_INT8 || cfg->scale_rule == SDQO_SCALE_UE4M3)) return -1;
  const int Bs = cfg->in_block;
  const double BF16_MAX = 3.3895313892515355e38;
  for (int64_t m = 0; m < M; ++m) {
    const uint16_t* x = X + m * K;
    double row_amax = 0.0;
    for (int64_t k = 0; k < K; ++k) {
      if ((x[k] & 0x7F80) == 0x7F80 && (x[k] & 0x007F)) return -2; /* NaN */
    }
    const int ue = cfg->scale_rule == SDQO_SCALE_UE4M3;
    for (int64_t k = 0; k < K; ++k) {
      double a = fabs(sdqo_bf16_to_double(x[k]));
      if (isinf(a)) a = BF16_MAX;
      if (a > row_amax) row_amax = a;
    }
    /* the token's 8-bit scale exponent; under two-level scaling also the power-of-two factor of its 4-bit Q-Vectors */
    const int e = sdqo_fp8_scale_exp(row_amax);
    const float sx = sdqo_int8_scale(row_amax);
    xq8_sexp[m] = cfg->out_fmt == SDQO_OUT_INT8 ? float_bits(sx) : e;
    for (int64_t b = 0; b < K / Bs; ++b) {
      double amax = 0.0;
      for (int64_t k = b * Bs; k < (b + 1) * Bs; ++k) {
        double a = fabs(sdqo_bf16_to_double(x[k]));
        if (isinf(a)) a = BF16_MAX;
        if (a > amax) amax = a;
      }
      uint8_t c = ue ? sdqo_ue4m3_scale_code(amax, e) : sdqo_e8m0_scale_code(amax, cfg->scale_rule);
      xq4_scale[m * (K / Bs) + b] = c;
      for (int64_t k = b * Bs; k < (b + 1) * Bs; ++k) {
        double v = sdqo_bf16_to_double(x[k]);
        if (isinf(v)) v = copysign(BF16_MAX, v);
        xq4_code[m * K + k] = ue ? e2m1_of_quotient(v, c, e) : sdqo_e2m1_encode(ldexp(v, 127 - (int)c));
      }
    }
    for (int64_t k = 0; k < K; ++k) {
      double v = sdqo_bf16_to_double(x[k]);
      if (isinf(v)) v = copysign(BF16_MAX, v);
      xq8_code[m * K + k] = cfg->out_fmt == SDQO_OUT_INT8 ? (uint8_t)sdqo_int8_encode(v, sx) : sdqo_e4m3_encode(ldexp(v, -e));
    }
  }
  return 0;
}

/* ------------------------------------------------------------------ the decomposed product, fp64
 * Y[m][n] = sum_k A_i[m][k] * W_i[n][k]  +  sum_k A_o[m][k] * W_o[n][k]        (O = O_i + O_o)
 * Rows n in [n_begin, n_end) and tokens m in [0, M) are produced into Y [M][n_end-n_begin].
 * Only the non-zero weights are visited; every term is formed and added in fp64. */
int sdqo_linear(int64_t M, int64_t N, int64_t K, const sdqo_config* cfg,
                const uint8_t* in_code, const uint8_t* in_meta, const uint8_t* in_scale,
                const uint8_t* out_code, const uint8_t* out_idx, const int32_t* out_sexp, const int32_t* in_texp,
                const uint8_t* xq4_code, const uint8_t* xq4_scale, const uint8_t* xq8_code, const int32_t* xq8_sexp,
                int64_t n_begin, int64_t n_end, double* Y, int n_threads) {
  if (n_begin < 0 || n_end > N || n_begin > n_end) return -1;
  const int on = cfg->out_n, Bs = cfg->in_block;
  const int64_t G8 = K / 8, NB = n_end - n_begin;
  double* A_i = (double*)malloc(sizeof(double) * (size_t)(M * K));
  double* A_o = (double*)malloc(sizeof(double) * (size_t)(M * K));
  for (int64_t m = 0; m < M; ++m)
    for (int64_t k = 0; k < K; ++k) {
      A_i[m * K + k] = sdqo_e2m1_decode(xq4_code[m * K + k]) * scale_value(cfg, xq4_scale[m * (K / Bs) + k / Bs], xq8_sexp[m]);
      A_o[m * K + k] = out_value(cfg, xq8_code[m * K + k], xq8_sexp[m]);
    }
#pragma omp parallel num_threads(n_threads > 0 ? n_threads : 1)
  {
    int32_t* ki = (int32_t*)malloc(sizeof(int32_t) * (size_t)K);
    double* wi = (double*)malloc(sizeof(double) * (size_t)K);
    int32_t* ko = (int32_t*)malloc(sizeof(int32_t) * (size_t)(G8 * 2));
    double* wo = (double*)malloc(sizeof(double) * (size_t)(G8 * 2));
#pragma omp for schedule(static)
    for (int64_t n = n_begin; n < n_end; ++n) {
      /* positions and values of the non-zeros of row n of W_i and W_o */
      int64_t ni = 0, no = 0, slot = 0;
      if (cfg->in_gran >= SDQO_GRAN_DENSE) {
        for (int64_t k = 0; k < K; ++k) {
          ki[ni] = (int32_t)k;
          wi[ni++] = sdqo_e2m1_decode(in_code[n * K + k]) * scale_value(cfg, in_scale[n * (K / Bs) + k / Bs], in_texp ? in_texp[n] : 0);
        }
      } else if (cfg->in_gran == SDQO_GRAN_PAIR) {
        for (int64_t g = 0; g < G8; ++g) {
          int nib = in_meta[n * G8 + g];
          int jj[2] = {nib & 3, (nib >> 2) & 3};
          for (int t = 0; t < 2; ++t)
            for (int u = 0; u < 2; ++u) {
              int64_t k = 8 * g + 2 * jj[t] + u;
              ki[ni] = (int32_t)k;
              wi[ni++] = sdqo_e2m1_decode(in_code[n * (K / 2) + slot++]) *
                         scale_value(cfg, in_scale[n * (K / Bs) + k / Bs], in_texp ? in_texp[n] : 0);
            }
        }
      } else {
        for (int64_t h = 0; h < K / 4; ++h) {
          int nib = in_meta[n * (K / 4) + h];
          int ii[2] = {nib & 3, (nib >> 2) & 3};
          for (int t = 0; t < 2; ++t) {
            int64_t k = 4 * h + ii[t];
            ki[ni] = (int32_t)k;
            wi[ni++] = sdqo_e2m1_decode(in_code[n * (K / 2) + slot++]) *
                       scale_value(cfg, in_scale[n * (K / Bs) + k / Bs], in_texp ? in_texp[n] : 0);
          }
        }
      }
      for (int64_t g = 0; g < G8; ++g)
        for (int t = 0; t < on; ++t) {
          ko[no] = (int32_t)(8 * g + out_idx[(n * G8 + g) * on + t]);
          wo[no++] = out_value(cfg, out_code[(n * G8 + g) * on + t], out_sexp[n]);
        }
      for (int64_t m = 0; m < M; ++m) {
        double acc = 0.0;
        for (int64_t t = 0; t < ni; ++t) acc += A_i[m * K + ki[t]] * wi[t];
        for (int64_t t = 0; t < no; ++t) acc += A_o[m * K + ko[t]] * wo[t];
        Y[m * NB + (n - n_begin)] = acc;
      }
    }
    free(ki); free(wi); free(ko); free(wo);
  }
  free(A_i);
  free(A_o);
  return 0;
}

/* ------------------------------------------------------------------ the paper's accounting (Section 3)
 * Average bits per weight element of the compressed format: data + index metadata + scale metadata.
 * An N:M part with b-bit values stores N*b data bits and N*ceil(log2 M) index bits per S-Vector of M
 * ("ELLPACK-like": one index per non-zero); a scale of s bits per Q-Vector of q logical elements
 * adds s/q. */
double sdqo_bits_per_weight_part(int n, int m, int value_bits, int scale_bits, int qvec) {
  int idx_bits = 0;
  while ((1 << idx_bits) < m) ++idx_bits;
  if (n == m) idx_bits = 0; /* dense: no index metadata */
  double bits = ((double)n * value_bits + (double)n * idx_bits) / (double)m;
  if (qvec > 0) bits += (double)scale_bits / (double)qvec;
  return bits;
}

/* Effective compute throughput model: an N:M part computed with b-bit operands costs
 * (N/M) * (b/16) of the fp16-dense time; the SDQ layer costs the sum of its two parts. */
double sdqo_relative_cost(int n, int m, int bits) { return ((double)n / m) * ((double)bits / 16.0); }
