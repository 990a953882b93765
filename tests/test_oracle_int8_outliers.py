"""Pins for the int8 outlier format of the oracle (Section 5.1: W_o and A_o in int8; the evaluation's "1:8int8"
configurations): closed forms at exactly representable points, the nearest-integer property in exact arithmetic, and a
product that must equal an exact integer matrix product times the two scales."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import sdq_synth
from oracle import sdq_oracle as so

CFG = so.Config(1, so.GRAN_PAIR, 64, so.SCALE_OCP_FLOOR, 0, so.OUT_INT8)


def bits_of(values):
    return sdq_synth.bf16_bits(torch.tensor(values, dtype=torch.float32).to(torch.bfloat16))


def f64_of(bits):
    return sdq_synth.bits_to_bf16(bits).to(torch.float64).numpy()


def test_scale_and_codes_at_exact_points():
    L = so.lib()
    # amax = 127 * 2^j: the scale is 2^j exactly and every integer multiple k * 2^j has code k
    for j in (-20, -3, 0, 5):
        s = L.sdqo_int8_scale(127.0 * 2.0 ** j)
        assert s == 2.0 ** j
        for k in range(-127, 128):
            assert L.sdqo_int8_encode(k * 2.0 ** j, s) == k
        # half-way points go to the even integer; beyond the range the code saturates at 127, never -128
        for k in range(-126, 126):
            want = k if k % 2 == 0 else k + 1
            assert L.sdqo_int8_encode((k + 0.5) * 2.0 ** j, s) == want
        assert L.sdqo_int8_encode(300.0 * 2.0 ** j, s) == 127 and L.sdqo_int8_encode(-300.0 * 2.0 ** j, s) == -127
    assert L.sdqo_int8_scale(0.0) == 1.0


def test_activation_codes_are_nearest_integers_of_x_over_s():
    """in exact rational arithmetic: |x / s - code| <= 1/2 up to the rounding of the fp32 quotient, the element of
    largest magnitude gets +-127, and the scale is the fp32 quotient amax / 127"""
    X = sdq_synth.make_act(6, 512, 11)
    Xb = sdq_synth.bf16_bits(X)
    q = so.quantize_act(Xb, CFG)
    x = f64_of(Xb)
    s = q.xq8_sexp.view(np.float32)
    codes = q.xq8_code.view(np.int8).astype(np.int64)
    assert (np.abs(codes) <= 127).all()
    for m in range(x.shape[0]):
        amax = np.abs(x[m]).max()
        assert s[m] == np.float32(np.float32(amax) / np.float32(127.0))
        assert abs(codes[m][np.abs(x[m]).argmax()]) == 127
        sm = Fraction(float(s[m]))
        for k in range(0, x.shape[1], 7):
            r = Fraction(float(x[m, k])) / sm
            assert abs(r - int(codes[m, k])) <= Fraction(1, 2) + abs(r) * Fraction(1, 2 ** 23)
    # the 4-bit side is untouched by the choice of the 8-bit format
    q0 = so.quantize_act(Xb, so.Config(1, so.GRAN_PAIR, 64, so.SCALE_OCP_FLOOR))
    assert np.array_equal(q.xq4_code, q0.xq4_code) and np.array_equal(q.xq4_scale, q0.xq4_scale)


def test_weight_outlier_codes_and_row_scales():
    Wb = sdq_synth.bf16_bits(sdq_synth.make_weight(32, 512, 3))
    p = so.decompose(Wb, CFG)
    p0 = so.decompose(Wb, so.Config(1, so.GRAN_PAIR, 64, so.SCALE_OCP_FLOOR))
    # which values are outliers and everything about the inliers does not depend on the 8-bit format
    assert np.array_equal(p.out_idx, p0.out_idx) and np.array_equal(p.in_code, p0.in_code)
    assert np.array_equal(p.in_meta, p0.in_meta) and np.array_equal(p.in_scale, p0.in_scale)
    w = f64_of(Wb).reshape(32, 64, 8)
    wo = np.take_along_axis(w, p.out_idx.astype(np.int64), axis=2)[..., 0]          # [N, K/8] the outlier values
    s = p.out_sexp.view(np.float32)
    codes = p.out_code.view(np.int8).astype(np.int64)[..., 0]
    for n in range(32):
        amax = np.abs(wo[n]).max()
        assert s[n] == np.float32(np.float32(amax) / np.float32(127.0))
        assert np.abs(codes[n]).max() == 127
        sn = Fraction(float(s[n]))
        for g in range(64):
            r = Fraction(float(wo[n, g])) / sn
            assert abs(r - int(codes[n, g])) <= Fraction(1, 2) + abs(r) * Fraction(1, 2 ** 23)
    # dequantized outliers: code * scale at the outlier positions, zero elsewhere; within half a step of the weights
    W_in, W_out = so.dequant_weights(p)
    got = np.take_along_axis(W_out.reshape(32, 64, 8), p.out_idx.astype(np.int64), axis=2)[..., 0]
    assert np.array_equal(got, codes * s.astype(np.float64)[:, None])
    assert (np.abs(got - wo) <= (0.5 + 127 * 2.0 ** -22) * s.astype(np.float64)[:, None]).all()     # (fp32 quotient)
    assert ((W_out != 0).reshape(32, 64, 8).sum(-1) <= 1).all()


def test_outlier_product_is_an_exact_integer_product_times_the_scales():
    """weights whose only non-zeros are the outliers (one per S-Vector): O = O_o, and O_o[m][n] must be
    s_x[m] * s_w[n] * (integer dot product of the codes) -- formed here with numpy's int64 matmul"""
    rng = np.random.default_rng(5)
    N, K, M = 24, 256, 5
    W = np.zeros((N, K), dtype=np.float32)
    pos = rng.integers(0, 8, size=(N, K // 8))
    vals = rng.standard_normal((N, K // 8)).astype(np.float32) * 0.05
    vals[vals == 0] = 0.01
    for n in range(N):
        W[n, np.arange(K // 8) * 8 + pos[n]] = vals[n]
    Wb = bits_of(W)
    Xb = sdq_synth.bf16_bits(sdq_synth.make_act(M, K, 8))
    p, q = so.decompose(Wb, CFG), so.quantize_act(Xb, CFG)
    assert np.array_equal(p.out_idx[..., 0], pos)
    Y = so.linear(q, p)
    qw = np.zeros((N, K), dtype=np.int64)
    cw = p.out_code.view(np.int8).astype(np.int64)[..., 0]
    for n in range(N):
        qw[n, np.arange(K // 8) * 8 + pos[n]] = cw[n]
    qx = q.xq8_code.view(np.int8).astype(np.int64)
    isum = qx @ qw.T                                                     # exact
    want = isum.astype(np.float64) * q.xq8_sexp.view(np.float32).astype(np.float64)[:, None] * p.out_sexp.view(np.float32).astype(np.float64)[None, :]
    assert np.allclose(Y, want, rtol=1e-12, atol=0)
    # and it is the product it approximates: error bounded by the two quantization steps
    x, w = f64_of(Xb), f64_of(Wb)
    sx, sw = q.xq8_sexp.view(np.float32).astype(np.float64), p.out_sexp.view(np.float32).astype(np.float64)
    bound = 0.5 * sx[:, None] * np.abs(w).sum(1)[None, :] + 0.5 * sw[None, :] * np.abs(x).sum(1)[:, None] + 0.25 * sx[:, None] * sw[None, :] * (K // 8)
    assert (np.abs(Y - x @ w.T) <= bound * 1.01).all()


def test_int8_with_e4m3_scale_codes_is_refused():
    Xb = sdq_synth.bf16_bits(sdq_synth.make_act(2, 128, 1))
    with pytest.raises(ValueError):
        so.quantize_act(Xb, so.Config(1, so.GRAN_PAIR, 32, so.SCALE_UE4M3, 0, so.OUT_INT8))
