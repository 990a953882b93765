"""ctypes/numpy front end of the SDQ oracle (sdq_oracle.c).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests, the smoke check and the CPU-baseline leg of the
benchmark may import this module.  It never imports the CUDA package.

All arrays are numpy; bf16 tensors are passed as uint16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sdq_oracle.c")
_LIB = os.path.join(_HERE, "libsdq_oracle.so")

GRAN_PAIR, GRAN_ELEM, GRAN_DENSE = 0, 1, 2
GRAN_3OF4 = 9      # S-Vectors of 4: 3:4 sparsification, one outlier per 4 (out_n = 2 per 8, or 0), two inliers per 4; stored dense


def gran_keep(n: int) -> int:
    """in_gran value of the pattern that keeps the n most significant of every 8 (out_n outliers + n - out_n inliers at
    any positions, stored like the dense pattern); gran_keep(8) == GRAN_DENSE."""
    assert 2 <= n <= 8
    return 2 + (8 - n)
SCALE_OCP_FLOOR, SCALE_CEIL_NOSAT, SCALE_UE4M3 = 0, 1, 2
ORDER_LARGE, ORDER_SMALL = 0, 1
OUT_E4M3, OUT_INT8 = 0, 1      # 8-bit format of W_o / A_o: E4M3 with power-of-two scales, or int8 with fp32 scales amax / 127


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (plain C11 + OpenMP); returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Cfg(ctypes.Structure):
    _fields_ = [("out_n", ctypes.c_int), ("in_gran", ctypes.c_int), ("in_block", ctypes.c_int),
                ("scale_rule", ctypes.c_int), ("out_order", ctypes.c_int), ("out_fmt", ctypes.c_int)]


@dataclass(frozen=True)
class Config:
    out_n: int = 1
    in_gran: int = GRAN_PAIR
    in_block: int = 64
    scale_rule: int = SCALE_OCP_FLOOR
    out_order: int = 0          # ORDER_LARGE; ORDER_SMALL takes the least significant values as outliers (study control)
    out_fmt: int = 0            # OUT_E4M3; OUT_INT8: int8 outlier operands (out_sexp / xq8_sexp then hold fp32 bit patterns)

    def c(self) -> _Cfg:
        return _Cfg(self.out_n, self.in_gran, self.in_block, self.scale_rule, self.out_order, self.out_fmt)


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.sdqo_bf16_to_double.restype = ctypes.c_double
        L.sdqo_bf16_to_double.argtypes = [ctypes.c_uint16]
        for name in ("sdqo_e2m1_decode", "sdqo_e4m3_decode", "sdqo_e8m0_decode"):
            getattr(L, name).restype = ctypes.c_double
            getattr(L, name).argtypes = [ctypes.c_uint8]
        for name in ("sdqo_e2m1_encode", "sdqo_e4m3_encode"):
            getattr(L, name).restype = ctypes.c_uint8
            getattr(L, name).argtypes = [ctypes.c_double]
        L.sdqo_e8m0_scale_code.restype = ctypes.c_uint8
        L.sdqo_e8m0_scale_code.argtypes = [ctypes.c_double, ctypes.c_int]
        L.sdqo_ue4m3_scale_code.restype = ctypes.c_uint8
        L.sdqo_ue4m3_scale_code.argtypes = [ctypes.c_double, ctypes.c_int]
        L.sdqo_fp8_scale_exp.restype = ctypes.c_int
        L.sdqo_fp8_scale_exp.argtypes = [ctypes.c_double]
        L.sdqo_int8_scale.restype = ctypes.c_float
        L.sdqo_int8_scale.argtypes = [ctypes.c_double]
        L.sdqo_int8_encode.restype = ctypes.c_int8
        L.sdqo_int8_encode.argtypes = [ctypes.c_double, ctypes.c_float]
        L.sdqo_bits_per_weight_part.restype = ctypes.c_double
        L.sdqo_bits_per_weight_part.argtypes = [ctypes.c_int] * 5
        L.sdqo_relative_cost.restype = ctypes.c_double
        L.sdqo_relative_cost.argtypes = [ctypes.c_int] * 3
        L.sdqo_decompose.restype = ctypes.c_int
        L.sdqo_decompose_metric.restype = ctypes.c_int
        L.sdqo_dequant_weights.restype = ctypes.c_int
        L.sdqo_quantize_act.restype = ctypes.c_int
        L.sdqo_linear.restype = ctypes.c_int
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


@dataclass
class Packed:
    """Canonical (layout-free) arrays of one decomposed weight matrix, one code per byte."""
    N: int
    K: int
    cfg: Config
    in_code: np.ndarray    # [N, K/2] u8 E2M1 codes of kept slots, ascending k ([N, K] from GRAN_DENSE on)
    in_meta: np.ndarray    # [N, K/8] (pair) or [N, K/4] (elem) u8 nibble values ([N, 0] from GRAN_DENSE on)
    in_scale: np.ndarray   # [N, K/in_block] u8 E8M0 codes
    out_code: np.ndarray   # [N, K/8, out_n] u8 E4M3 codes
    out_idx: np.ndarray    # [N, K/8, out_n] u8 positions 0..7
    out_sexp: np.ndarray   # [N] i32, outlier scale = 2^out_sexp
    in_texp: np.ndarray = None   # [N] i32, SCALE_UE4M3: inlier scale = E4M3(in_scale) * 2^in_texp (zeros otherwise)


@dataclass
class QAct:
    """Canonical arrays of one quantized activation matrix."""
    M: int
    K: int
    cfg: Config
    xq4_code: np.ndarray   # [M, K] u8 E2M1 codes
    xq4_scale: np.ndarray  # [M, K/in_block] u8 E8M0 codes
    xq8_code: np.ndarray   # [M, K] u8 E4M3 codes
    xq8_sexp: np.ndarray   # [M] i32, per-token scale = 2^xq8_sexp


def decompose(W_bits: np.ndarray, cfg: Config, col_weight=None) -> Packed:
    """Stage 2 / 1 / 3 of Section 5.  col_weight: optional per-input-channel activation norm c[k] >= 0 (fp32); the
    significance of an element is then the weight-activation product |w| * c[k] instead of the magnitude."""
    W_bits = np.ascontiguousarray(W_bits, dtype=np.uint16)
    N, K = W_bits.shape
    nmeta = 0 if cfg.in_gran >= GRAN_DENSE else (K // 8 if cfg.in_gran == GRAN_PAIR else K // 4)
    nslot = K if cfg.in_gran >= GRAN_DENSE else K // 2
    on = max(cfg.out_n, 0)
    p = Packed(N, K, cfg,
               np.zeros((N, nslot), np.uint8), np.zeros((N, nmeta), np.uint8),
               np.zeros((N, K // cfg.in_block), np.uint8),
               np.zeros((N, K // 8, on), np.uint8), np.zeros((N, K // 8, on), np.uint8),
               np.zeros((N,), np.int32), np.zeros((N,), np.int32))
    c = cfg.c()
    if col_weight is None:
        cw = None
    else:
        cw_arr = np.ascontiguousarray(col_weight, dtype=np.float32)
        assert cw_arr.shape == (K,)
        cw = _p(cw_arr)
    rc = lib().sdqo_decompose_metric(_p(W_bits), ctypes.c_int64(N), ctypes.c_int64(K), ctypes.byref(c), cw,
                                     _p(p.in_code), _p(p.in_meta), _p(p.in_scale), _p(p.out_code), _p(p.out_idx),
                                     _p(p.out_sexp), _p(p.in_texp))
    if rc != 0:
        raise ValueError("sdqo_decompose failed: %d" % rc)
    return p


def channel_norm(X_bits: np.ndarray) -> np.ndarray:
    """Euclidean norm of every input channel over the tokens, c[k] = sqrt(sum_m x[m][k]^2) (the activation statistic
    of the weight-activation product metric, Section 5 Stage 1), in fp64, returned as fp32."""
    X_bits = np.ascontiguousarray(X_bits, dtype=np.uint16)
    x = (X_bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return np.sqrt((x * x).sum(axis=0)).astype(np.float32)


def dequant_weights(p: Packed):
    """Dense fp64 (W_in, W_out), each [N, K]."""
    W_in = np.zeros((p.N, p.K), np.float64)
    W_out = np.zeros((p.N, p.K), np.float64)
    c = p.cfg.c()
    rc = lib().sdqo_dequant_weights(ctypes.c_int64(p.N), ctypes.c_int64(p.K), ctypes.byref(c),
                                    _p(p.in_code), _p(p.in_meta), _p(p.in_scale), _p(p.out_code), _p(p.out_idx),
                                    _p(p.out_sexp), _p(p.in_texp), _p(W_in), _p(W_out))
    assert rc == 0
    return W_in, W_out


def quantize_act(X_bits: np.ndarray, cfg: Config) -> QAct:
    X_bits = np.ascontiguousarray(X_bits, dtype=np.uint16)
    M, K = X_bits.shape
    q = QAct(M, K, cfg, np.zeros((M, K), np.uint8), np.zeros((M, K // cfg.in_block), np.uint8),
             np.zeros((M, K), np.uint8), np.zeros((M,), np.int32))
    c = cfg.c()
    rc = lib().sdqo_quantize_act(_p(X_bits), ctypes.c_int64(M), ctypes.c_int64(K), ctypes.byref(c),
                                 _p(q.xq4_code), _p(q.xq4_scale), _p(q.xq8_code), _p(q.xq8_sexp))
    if rc != 0:
        raise ValueError("sdqo_quantize_act failed: %d" % rc)
    return q


def dequant_act(q: QAct):
    """Dense fp64 (A_i, A_o), each [M, K]."""
    L = lib()
    e2m1 = np.array([L.sdqo_e2m1_decode(c) for c in range(16)])
    e4m3 = np.array([L.sdqo_e4m3_decode(c) for c in range(256)])
    if q.cfg.scale_rule == SCALE_UE4M3:
        sc = np.repeat(np.ldexp(e4m3[q.xq4_scale], q.xq8_sexp[:, None].astype(np.int64)), q.cfg.in_block, axis=1)
    else:
        sc = np.repeat(np.ldexp(1.0, q.xq4_scale.astype(np.int64) - 127), q.cfg.in_block, axis=1)
    A_i = e2m1[q.xq4_code] * sc
    if q.cfg.out_fmt == OUT_INT8:
        A_o = q.xq8_code.view(np.int8).astype(np.float64) * q.xq8_sexp.view(np.float32)[:, None].astype(np.float64)
    else:
        A_o = np.ldexp(e4m3[q.xq8_code], q.xq8_sexp[:, None].astype(np.int64))
    return A_i, A_o


def linear(q: QAct, p: Packed, n_begin: int = 0, n_end: int | None = None, threads: int | None = None) -> np.ndarray:
    """Y[:, n_begin:n_end] of the decomposed product in fp64."""
    assert q.K == p.K and q.cfg == p.cfg
    n_end = p.N if n_end is None else n_end
    threads = threads or (os.cpu_count() or 1)
    Y = np.zeros((q.M, n_end - n_begin), np.float64)
    c = p.cfg.c()
    rc = lib().sdqo_linear(ctypes.c_int64(q.M), ctypes.c_int64(p.N), ctypes.c_int64(p.K), ctypes.byref(c),
                           _p(p.in_code), _p(p.in_meta), _p(p.in_scale), _p(p.out_code), _p(p.out_idx),
                           _p(p.out_sexp), _p(p.in_texp), _p(q.xq4_code), _p(q.xq4_scale), _p(q.xq8_code), _p(q.xq8_sexp),
                           ctypes.c_int64(n_begin), ctypes.c_int64(n_end), _p(Y), ctypes.c_int(threads))
    assert rc == 0
    return Y


def bits_per_weight(cfg: Config, K: int | None = None) -> float:
    """Average bits per weight element of the packed SDQ format (data + index + scale metadata)."""
    L = lib()
    if cfg.in_gran >= GRAN_DENSE:
        # every position stored as a 4-bit value (outlier and dropped positions hold +0): no index metadata
        inl = L.sdqo_bits_per_weight_part(8, 8, 4, 8, cfg.in_block)
    elif cfg.in_gran == GRAN_PAIR:
        # 2 of 4 pairs: per 8 elements 4 stored 4-bit values + two 2-bit pair indices
        inl = (4 * 4 + 2 * 2) / 8.0 + 8.0 / cfg.in_block
    else:
        inl = L.sdqo_bits_per_weight_part(2, 4, 4, 8, cfg.in_block)
    out = L.sdqo_bits_per_weight_part(cfg.out_n, 8, 8, 0, 0) if cfg.out_n else 0.0
    row = (32.0 / K) if (K and cfg.out_n) else 0.0
    return inl + out + row
