"""Pins for the oracle's decomposed product O = A_i W_i^T + A_o W_o^T and the paper's accounting."""
import os

import numpy as np
import pytest
import torch

import sdq_synth
from oracle import sdq_oracle as so
from tests.indep_definition import decompose_dense, quantize_act_dense

CFG = so.Config(1, so.GRAN_PAIR, 64, so.SCALE_OCP_FLOOR)


def make(M, N, K, seed, cfg=CFG):
    Wb = sdq_synth.bf16_bits(sdq_synth.make_weight(N, K, seed))
    Xb = sdq_synth.bf16_bits(sdq_synth.make_act(M, K, seed, n_outlier_channels=2))
    return Wb, Xb, so.decompose(Wb, cfg), so.quantize_act(Xb, cfg)


@pytest.mark.parametrize("cfg", [CFG, so.Config(2, so.GRAN_ELEM, 32, so.SCALE_CEIL_NOSAT), so.Config(0, so.GRAN_PAIR, 64, 0),
                                 so.Config(1, so.GRAN_DENSE, 32, so.SCALE_OCP_FLOOR),
                                 so.Config(1, so.gran_keep(7), 32, so.SCALE_OCP_FLOOR),
                                 so.Config(1, so.GRAN_PAIR, 32, so.SCALE_UE4M3)])
def test_brute_force_triple_loop(cfg):
    Wb, Xb, p, q = make(3, 16, 128, 2, cfg)
    W_in, W_out = so.dequant_weights(p)
    A_i, A_o = so.dequant_act(q)
    Y = so.linear(q, p, threads=2)
    for m in range(3):
        for n in range(16):
            acc = 0.0
            for k in range(128):
                acc += A_i[m, k] * W_in[n, k]
            for k in range(128):
                acc += A_o[m, k] * W_out[n, k]
            assert abs(Y[m, n] - acc) <= 1e-12 * (abs(acc) + 1)


def test_matches_independent_definition_end_to_end():
    """product of the independently quantized dense operands (no oracle routine involved)"""
    Wb, Xb, p, q = make(8, 64, 256, 0)
    Win, Wout, _, _ = decompose_dense(Wb, 1, True, 64, True)
    Ai, Ao = quantize_act_dense(Xb, 64, True)
    ref = Ai @ Win.T + Ao @ Wout.T
    Y = so.linear(q, p)
    assert np.allclose(Y, ref, rtol=1e-12, atol=1e-12)


def test_no_outliers_reduces_to_plain_quantized_gemm():
    cfg = so.Config(0, so.GRAN_PAIR, 64, so.SCALE_OCP_FLOOR)
    Wb, Xb, p, q = make(4, 32, 256, 3, cfg)
    W_in, W_out = so.dequant_weights(p)
    assert not W_out.any()
    A_i, _ = so.dequant_act(q)
    assert np.allclose(so.linear(q, p), A_i @ W_in.T, rtol=1e-13, atol=1e-13)


def test_dense_inliers_match_independent_definition_end_to_end():
    cfg = so.Config(1, so.GRAN_DENSE, 32, so.SCALE_CEIL_NOSAT)
    Wb, Xb, p, q = make(8, 64, 256, 9, cfg)
    Win, Wout, _, _ = decompose_dense(Wb, 1, None, 32, False)
    Ai, Ao = quantize_act_dense(Xb, 32, False)
    assert np.allclose(so.linear(q, p), Ai @ Win.T + Ao @ Wout.T, rtol=1e-12, atol=1e-12)
    # and it is closer to the unquantized product than the pruned decomposition of the same weights
    W = torch.from_numpy(Wb.view(np.int16)).view(torch.bfloat16).double().numpy()
    X = torch.from_numpy(Xb.view(np.int16)).view(torch.bfloat16).double().numpy()
    cfg_p = so.Config(1, so.GRAN_PAIR, 32, so.SCALE_CEIL_NOSAT)
    err_dense = np.linalg.norm(so.linear(q, p) - X @ W.T)
    err_pruned = np.linalg.norm(so.linear(so.quantize_act(Xb, cfg_p), so.decompose(Wb, cfg_p)) - X @ W.T)
    assert err_dense < err_pruned


def test_ue4m3_scales_match_independent_definition_end_to_end():
    cfg = so.Config(1, so.GRAN_PAIR, 32, so.SCALE_UE4M3)
    Wb, Xb, p, q = make(8, 64, 256, 11, cfg)
    Win, Wout, _, _ = decompose_dense(Wb, 1, True, 32, "ue4m3")
    Ai, Ao = quantize_act_dense(Xb, 32, "ue4m3")
    assert np.allclose(so.linear(q, p), Ai @ Win.T + Ao @ Wout.T, rtol=1e-12, atol=1e-12)


def test_one_hot_readback_returns_columns_of_W_in_plus_W_out():
    Wb, _, p, _ = make(1, 32, 128, 4)
    W_in, W_out = so.dequant_weights(p)
    X = np.eye(128)                        # 1.0 is exact in both activation formats
    Xb = sdq_synth.bf16_bits(torch.from_numpy(X).to(torch.bfloat16))
    q = so.quantize_act(Xb, CFG)
    Y = so.linear(q, p)                    # [128, 32]
    assert np.array_equal(Y, (W_in + W_out).T)


def test_scaling_x_by_power_of_two_scales_y_exactly():
    Wb, Xb, p, q = make(4, 32, 256, 5)
    X = torch.from_numpy(Xb.view(np.int16)).view(torch.bfloat16)
    q8 = so.quantize_act(sdq_synth.bf16_bits(X * 8), CFG)
    assert np.array_equal(so.linear(q8, p), 8.0 * so.linear(q, p))


def test_row_permutation_of_W_permutes_columns_of_Y():
    Wb, Xb, p, q = make(4, 32, 256, 6)
    perm = np.random.default_rng(0).permutation(32)
    p2 = so.decompose(Wb[perm], CFG)
    assert np.array_equal(so.linear(q, p2), so.linear(q, p)[:, perm])


def test_row_slice_and_thread_count_do_not_change_results():
    Wb, Xb, p, q = make(5, 64, 256, 7)
    Y = so.linear(q, p, threads=1)
    assert np.array_equal(so.linear(q, p, threads=os.cpu_count()), Y)
    assert np.array_equal(so.linear(q, p, 16, 48), Y[:, 16:48])


def test_error_against_unquantized_product_is_small():
    """sanity of the whole scheme: the decomposed product tracks the bf16 product"""
    Wb, Xb, p, q = make(8, 64, 1024, 8)
    W = torch.from_numpy(Wb.view(np.int16)).view(torch.bfloat16).double().numpy()
    X = torch.from_numpy(Xb.view(np.int16)).view(torch.bfloat16).double().numpy()
    ref = X @ W.T
    Y = so.linear(q, p)
    rel = np.linalg.norm(Y - ref) / np.linalg.norm(ref)
    assert rel < 0.6   # 2:4 pruning + 4-bit: coarse, but correlated
    assert np.corrcoef(Y.ravel(), ref.ravel())[0, 1] > 0.8


def test_error_order_of_the_configurations():
    """the paper's qualitative findings on the synthetic layer: outlier extraction lowers the output error, dropping one
    of eight values costs little, 50 % sparsity costs most, and 1:8 outliers + 6:8 inliers beat plain dense 4-bit"""
    Wb = sdq_synth.bf16_bits(sdq_synth.make_weight(96, 2048, 21))
    Xb = sdq_synth.bf16_bits(sdq_synth.make_act(16, 2048, 22))
    W = torch.from_numpy(Wb.view(np.int16)).view(torch.bfloat16).double().numpy()
    X = torch.from_numpy(Xb.view(np.int16)).view(torch.bfloat16).double().numpy()
    ref = X @ W.T

    def err(cfg):
        return np.linalg.norm(so.linear(so.quantize_act(Xb, cfg), so.decompose(Wb, cfg)) - ref) / np.linalg.norm(ref)
    e48_0, e48_1, e48_2 = (err(so.Config(n, so.GRAN_PAIR, 32, 0)) for n in (0, 1, 2))
    e78, e88, e88_0 = err(so.Config(1, so.gran_keep(7), 32, 0)), err(so.Config(1, so.GRAN_DENSE, 32, 0)), err(so.Config(0, so.GRAN_DENSE, 32, 0))
    e34 = err(so.Config(2, so.GRAN_3OF4, 32, 0))
    e_ue = err(so.Config(1, so.GRAN_PAIR, 32, so.SCALE_UE4M3))
    assert e48_0 > e48_1 > e48_2
    assert e88 < e78 < e48_2
    assert e78 < e88_0                      # the headline claim: 7:8 = 1:8 + 6:8 beats dense 4-bit quantization
    assert e88 < e34 < e48_1
    assert e_ue < e48_1


def golden():
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_arithmetic.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split()
                vals[k] = float(v)
    return vals


def test_paper_accounting_arithmetic():
    g = golden()
    L = so.lib()
    # index metadata per S-Vector = N * ceil(log2 M)
    assert (L.sdqo_bits_per_weight_part(2, 4, 0, 0, 0) * 4) == g["index_bits_2of4_per_vector"]
    assert (L.sdqo_bits_per_weight_part(1, 8, 0, 0, 0) * 8) == g["index_bits_1of8_per_vector"]
    # 4-bit values, 16-bit scale, Q-Vector 4, dense
    assert L.sdqo_bits_per_weight_part(4, 4, 4, 16, 4) == g["bits_per_elt_4bit_16bitscale_qvec4"]
    # "a 3:4 sparse 4-bit model can have more bits per weight than a dense 4-bit one" (8-bit scale, Q-Vector 32)
    assert L.sdqo_bits_per_weight_part(3, 4, 4, 8, 32) > L.sdqo_bits_per_weight_part(4, 4, 4, 8, 32)
    assert L.sdqo_relative_cost(1, 8, 8) == g["cost_outlier_1of8_int8"]
    assert L.sdqo_relative_cost(6, 8, 4) == g["cost_inlier_6of8_fp4"]
    assert L.sdqo_relative_cost(1, 8, 8) + L.sdqo_relative_cost(6, 8, 4) == g["cost_total_1of8_6of8"]
    s = 1.0 / (L.sdqo_relative_cost(1, 8, 8) + L.sdqo_relative_cost(7, 8, 4))
    assert round(s, 1) == g["speedup_8of8_1of8_7of8"]


def test_bits_per_weight_of_the_formats_used_here():
    assert so.bits_per_weight(so.Config(1, so.GRAN_PAIR, 64, 0)) == 2 + 0.5 + 0.125 + 1.375
    assert so.bits_per_weight(so.Config(0, so.GRAN_PAIR, 64, 0)) == 2.625
    assert so.bits_per_weight(so.Config(2, so.GRAN_PAIR, 64, 0)) == 2.625 + 2.75
    assert so.bits_per_weight(so.Config(1, so.GRAN_ELEM, 32, 0)) == 2 + 1 + 0.25 + 1.375
    # no pruning: 4-bit value at every position, one 8-bit scale per 32, plus the 1:8 outliers (8-bit value + 3-bit index)
    assert so.bits_per_weight(so.Config(1, so.GRAN_DENSE, 32, 0)) == 4 + 0.25 + 1.375
    assert so.bits_per_weight(so.Config(0, so.GRAN_DENSE, 64, 0)) == 4.125
