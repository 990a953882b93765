"""Pins for the oracle's decomposition (Stages 1-3) and activation quantization."""
import itertools

import numpy as np
import pytest

import sdq_synth
from oracle import sdq_oracle as so
from tests.indep_definition import bf16_to_f64, decompose_dense, quantize_act_dense, two_level_quantize

CFGS = [so.Config(1, so.GRAN_PAIR, 64, so.SCALE_OCP_FLOOR),
        so.Config(1, so.GRAN_ELEM, 32, so.SCALE_OCP_FLOOR),
        so.Config(2, so.GRAN_PAIR, 64, so.SCALE_CEIL_NOSAT),
        so.Config(0, so.GRAN_PAIR, 64, so.SCALE_OCP_FLOOR),
        so.Config(2, so.GRAN_ELEM, 64, so.SCALE_OCP_FLOOR),
        so.Config(0, so.GRAN_ELEM, 32, so.SCALE_CEIL_NOSAT)]


def tiny_W(N=64, K=256, seed=0):
    return sdq_synth.bf16_bits(sdq_synth.make_weight(N, K, seed))


@pytest.mark.parametrize("cfg", CFGS)
def test_nm_invariants(cfg):
    """at most out_n outliers per 8; exactly 2 kept pairs per 8 / 2 kept per 4; disjoint supports"""
    Wb = tiny_W()
    p = so.decompose(Wb, cfg)
    W_in, W_out = so.dequant_weights(p)
    N, K = Wb.shape
    assert ((W_out != 0).reshape(N, K // 8, 8).sum(-1) <= cfg.out_n).all()
    assert not ((W_in != 0) & (W_out != 0)).any()
    if cfg.in_gran == so.GRAN_PAIR:
        j0, j1 = p.in_meta & 3, (p.in_meta >> 2) & 3
        assert (j0 < j1).all()
        pair_nz = (W_in != 0).reshape(N, K // 8, 4, 2).any(-1)
        assert (pair_nz.sum(-1) <= 2).all()
    else:
        i0, i1 = p.in_meta & 3, (p.in_meta >> 2) & 3
        assert (i0 < i1).all()
        assert ((W_in != 0).reshape(N, K // 4, 4).sum(-1) <= 2).all()
    if cfg.out_n:
        assert (np.diff(p.out_idx.astype(int), axis=-1) > 0).all()
        assert (p.out_idx < 8).all()


@pytest.mark.parametrize("cfg", CFGS)
def test_matches_independent_dense_definition(cfg):
    """W_in + W_out equals the pruned-quantized W computed by an independent routine"""
    for seed in (0, 1):
        Wb = tiny_W(48, 512, seed)
        p = so.decompose(Wb, cfg)
        W_in, W_out = so.dequant_weights(p)
        ref_in, ref_out, slots, mask_out = decompose_dense(Wb, cfg.out_n, cfg.in_gran == so.GRAN_PAIR, cfg.in_block,
                                                           cfg.scale_rule == so.SCALE_OCP_FLOOR)
        assert np.array_equal(W_out, ref_out)
        assert np.array_equal(W_in, ref_in)
        assert np.array_equal(W_in + W_out, ref_in + ref_out)


def test_selection_brute_force_all_choices():
    """chosen outlier set maximises kept magnitude and is lexicographically first among maximisers;
    same for the kept pair set (pair score) -- enumerated over all C(8,n) / C(4,2) choices"""
    rng = np.random.default_rng(5)
    # few distinct magnitudes -> many ties
    vals = np.array([0.0, 0.5, 1.0, 1.0, 2.0, -2.0, 3.0, -0.5])
    W = rng.choice(vals, size=(32, 64))
    import torch
    Wb = sdq_synth.bf16_bits(torch.from_numpy(W).to(torch.bfloat16))
    for out_n in (1, 2):
        cfg = so.Config(out_n, so.GRAN_PAIR, 64, so.SCALE_OCP_FLOOR)
        p = so.decompose(Wb, cfg)
        for n in range(W.shape[0]):
            for g in range(W.shape[1] // 8):
                a = np.abs(W[n, 8 * g:8 * g + 8])
                best, best_set = -1.0, None
                for comb in itertools.combinations(range(8), out_n):
                    s = a[list(comb)].sum()
                    if s > best:
                        best, best_set = s, comb
                # lexicographically first maximiser under "largest first, lower index on ties"
                order = sorted(range(8), key=lambda i: (-a[i], i))[:out_n]
                assert a[order].sum() == best
                assert tuple(p.out_idx[n, g]) == tuple(sorted(order))
                r = a.copy()
                r[order] = 0.0
                score = r.reshape(4, 2).sum(-1)
                bestp = max(itertools.combinations(range(4), 2), key=lambda c: (score[list(c)].sum(), ))
                porder = sorted(sorted(range(4), key=lambda j: (-score[j], j))[:2])
                assert score[porder].sum() == score[list(bestp)].sum()
                assert (int(p.in_meta[n, g]) & 3, int(p.in_meta[n, g]) >> 2) == tuple(porder)


def test_on_grid_weights_round_trip_exactly():
    """weights that already lie on the E2M1*2^E / E4M3*2^e grids with a valid pattern survive unchanged"""
    rng = np.random.default_rng(3)
    N, K = 16, 256
    W = np.zeros((N, K))
    e2m1 = np.array([0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
    for n in range(N):
        for g in range(K // 8):
            o = rng.integers(0, 8)
            W[n, 8 * g + o] = rng.choice([-1, 1]) * 16.0 * (1 + rng.integers(0, 8) / 8)   # E4M3-exact, dominates
            pairs = [j for j in range(4)]
            free = [j for j in pairs if j != o // 2]
            keep = rng.choice(free, size=2, replace=False)
            for j in keep:
                for u in range(2):
                    W[n, 8 * g + 2 * j + u] = rng.choice([-1, 1]) * rng.choice(e2m1) * 0.125
        # make sure every 64-block has amax = 6*0.125 so the shared scale is 2^-3 under both rules
        for b in range(K // 64):
            g = 8 * b
            o_pos = np.nonzero(np.abs(W[n, 8 * g:8 * g + 8]) >= 16)[0][0]
            j = [j for j in range(4) if j != o_pos // 2 and W[n, 8 * g + 2 * j] != 0][0]
            W[n, 8 * g + 2 * j] = 0.75
    import torch
    Wb = sdq_synth.bf16_bits(torch.from_numpy(W).to(torch.bfloat16))
    assert np.array_equal(bf16_to_f64(Wb), W)
    for rule in (so.SCALE_OCP_FLOOR, so.SCALE_CEIL_NOSAT):
        p = so.decompose(Wb, so.Config(1, so.GRAN_PAIR, 64, rule))
        W_in, W_out = so.dequant_weights(p)
        assert np.array_equal(W_in + W_out, W)


def test_ceil_rule_never_saturates_floor_rule_only_in_6_to_8():
    Wb = tiny_W(64, 512, 9)
    W = bf16_to_f64(Wb)
    for rule in (so.SCALE_OCP_FLOOR, so.SCALE_CEIL_NOSAT):
        cfg = so.Config(1, so.GRAN_PAIR, 64, rule)
        p = so.decompose(Wb, cfg)
        W_in, _ = so.dequant_weights(p)
        sc = np.repeat(np.ldexp(1.0, p.in_scale.astype(int) - 127), 64, axis=1)
        scaled = np.abs(np.where(W_in != 0, W, 0.0)) / sc
        if rule == so.SCALE_CEIL_NOSAT:
            assert scaled.max() <= 6.0
        else:
            assert scaled.max() < 8.0


def test_all_zero_and_ties_pick_lowest_indices():
    Wb = np.zeros((4, 128), np.uint16)
    p = so.decompose(Wb, so.Config(2, so.GRAN_PAIR, 64, so.SCALE_OCP_FLOOR))
    assert (p.out_idx[..., 0] == 0).all() and (p.out_idx[..., 1] == 1).all()
    assert (p.in_meta == (0 | (1 << 2))).all()
    assert (p.in_code == 0).all() and (p.in_scale == 0).all() and (p.out_sexp == 0).all()
    p = so.decompose(Wb, so.Config(1, so.GRAN_ELEM, 32, so.SCALE_OCP_FLOOR))
    # group of 4 that contains the outlier (position 0) keeps elements 1,2; the other keeps 0,1
    assert (p.in_meta[:, 0::2] == (1 | (2 << 2))).all()
    assert (p.in_meta[:, 1::2] == (0 | (1 << 2))).all()


def test_nonfinite_weight_rejected():
    Wb = tiny_W(8, 128, 0)
    Wb[3, 5] = 0x7F80
    with pytest.raises(ValueError):
        so.decompose(Wb, so.Config())


@pytest.mark.parametrize("cfg", CFGS[:3])
def test_activation_quantization_matches_independent_definition(cfg):
    Xb = sdq_synth.bf16_bits(sdq_synth.make_act(24, 512, 4, n_outlier_channels=5))
    q = so.quantize_act(Xb, cfg)
    A_i, A_o = so.dequant_act(q)
    ref_i, ref_o = quantize_act_dense(Xb, cfg.in_block, cfg.scale_rule == so.SCALE_OCP_FLOOR)
    assert np.array_equal(A_i, ref_i)
    assert np.array_equal(A_o, ref_o)
    # nothing saturates in the 8-bit copy; it is within half an E4M3 ulp (2^-4 relative) of x
    X = bf16_to_f64(Xb)
    assert (np.abs(A_o - X) <= np.abs(X) * 2.0 ** -4 + 2.0 ** (q.xq8_sexp[:, None].astype(float) - 10)).all()


def test_block64_scale_is_max_of_the_two_block32_scales():
    Xb = sdq_synth.bf16_bits(sdq_synth.make_act(16, 256, 11))
    q64 = so.quantize_act(Xb, so.Config(1, so.GRAN_PAIR, 64, so.SCALE_OCP_FLOOR))
    q32 = so.quantize_act(Xb, so.Config(1, so.GRAN_PAIR, 32, so.SCALE_OCP_FLOOR))
    assert np.array_equal(q64.xq4_scale, q32.xq4_scale.reshape(16, -1, 2).max(-1))


def test_activation_inf_saturates_nan_rejected():
    Xb = sdq_synth.bf16_bits(sdq_synth.make_act(2, 128, 1))
    Xb[0, 3] = 0x7F80   # +inf
    Xb[1, 9] = 0xFF80   # -inf
    q = so.quantize_act(Xb, so.Config())
    assert q.xq4_code[0, 3] == 7 and q.xq4_code[1, 9] == 15
    assert q.xq8_code[0, 3] in (0x7E, 0x7D, 0x7C, 0x7B, 0x7A, 0x79, 0x78)  # top binade, no NaN code
    Xb[0, 0] = 0x7FC0
    with pytest.raises(ValueError):
        so.quantize_act(Xb, so.Config())


# ---------------------------------------------------------------- weight-activation product metric
def lognormal_channel_weight(K, seed):
    rng = np.random.default_rng(seed)
    c = np.exp(rng.normal(0.0, 1.0, K)).astype(np.float32)
    c[rng.integers(0, K, max(1, K // 64))] *= 30.0        # a few heavy input channels, as in make_act
    return c


@pytest.mark.parametrize("cfg", CFGS)
def test_product_metric_with_unit_or_power_of_two_channel_weight_is_the_magnitude_metric(cfg):
    """|w| * 1 == |w| and |w| * 2^t preserves every order and every tie: the packed arrays must not change"""
    Wb = tiny_W(32, 512, 7)
    ref = so.decompose(Wb, cfg)
    for c in (np.ones(512, np.float32), np.full(512, 2.0 ** -9, np.float32), np.full(512, 64.0, np.float32)):
        p = so.decompose(Wb, cfg, col_weight=c)
        for name in ("in_code", "in_meta", "in_scale", "out_code", "out_idx", "out_sexp"):
            assert np.array_equal(getattr(p, name), getattr(ref, name)), name


def test_product_metric_hand_example():
    """Section 5 (Stage 1): a tiny weight whose activation is huge matters.  Row of one S-Vector of 8 (padded to 64
    with zeros): magnitudes pick position 0 (0.5) as the outlier, products with c[7] = 10 pick position 7 (0.09375*10)."""
    import torch
    w = np.zeros((1, 64))
    w[0, :8] = [0.5, 0.125, 0.125, 0.125, 0.125, 0.125, 0.125, 0.09375]
    Wb = sdq_synth.bf16_bits(torch.from_numpy(w).to(torch.bfloat16))
    cfg = so.Config(1, so.GRAN_PAIR, 64, so.SCALE_OCP_FLOOR)
    assert so.decompose(Wb, cfg).out_idx[0, 0, 0] == 0
    c = np.ones(64, np.float32)
    c[7] = 10.0
    p = so.decompose(Wb, cfg, col_weight=c)
    assert p.out_idx[0, 0, 0] == 7
    W_in, W_out = so.dequant_weights(p)
    assert W_out[0, 7] == 0.09375 and np.count_nonzero(W_out[0, :8]) == 1      # the VALUE is untouched by the metric
    # remaining products: 0.5, 0.125 x6 -> pair scores (0.625, 0.25, 0.25, 0.125): pairs 0 and 1 are kept
    assert p.in_meta[0, 0] == (0 | (1 << 2))
    assert W_in[0, 0] == 0.5 and W_in[0, 6] == 0.0 and W_in[0, 7] == 0.0


@pytest.mark.parametrize("cfg", CFGS)
def test_product_metric_matches_independent_dense_definition(cfg):
    for seed in (3, 4):
        Wb = tiny_W(40, 512, seed)
        c = lognormal_channel_weight(512, seed)
        p = so.decompose(Wb, cfg, col_weight=c)
        W_in, W_out = so.dequant_weights(p)
        ref_in, ref_out, slots, mask_out = decompose_dense(Wb, cfg.out_n, cfg.in_gran == so.GRAN_PAIR, cfg.in_block,
                                                           cfg.scale_rule == so.SCALE_OCP_FLOOR, col_weight=c)
        assert np.array_equal(W_out, ref_out)
        assert np.array_equal(W_in, ref_in)
        N, K = Wb.shape
        assert ((W_out != 0).reshape(N, K // 8, 8).sum(-1) <= cfg.out_n).all()
        assert not ((W_in != 0) & (W_out != 0)).any()


def test_product_metric_rejects_bad_channel_weight():
    Wb = tiny_W(4, 64, 0)
    cfg = CFGS[0]
    for bad in (-1.0, np.inf, np.nan):
        c = np.ones(64, np.float32)
        c[5] = bad
        with pytest.raises(ValueError):
            so.decompose(Wb, cfg, col_weight=c)


def test_channel_norm_closed_forms():
    """c[k] = sqrt(sum_m x[m][k]^2): a constant column of value v over M tokens gives |v| sqrt(M); a one-hot column gives
    the magnitude of its entry; a 3-4-12 column gives 13; zeros give 0"""
    import torch
    M, K = 16, 8
    x = np.zeros((M, K))
    x[:, 0] = -0.5                  # 0.5 * sqrt(16) = 2
    x[5, 1] = 3.0                   # one-hot
    x[0, 2], x[1, 2], x[2, 2] = 3.0, -4.0, 12.0
    x[:, 3] = np.arange(M)          # sqrt(sum i^2) = sqrt(1240)
    Xb = sdq_synth.bf16_bits(torch.from_numpy(x).to(torch.bfloat16))
    c = so.channel_norm(Xb)
    assert c.dtype == np.float32 and c.shape == (K,)
    assert c[0] == 2.0 and c[1] == 3.0 and c[2] == 13.0
    assert c[3] == np.float32(np.sqrt(1240.0))
    assert (c[4:] == 0).all()
    # invariance to the order of the tokens, scaling by a power of two
    perm = np.random.default_rng(0).permutation(M)
    assert np.array_equal(so.channel_norm(Xb[perm]), c)
    Xb4 = sdq_synth.bf16_bits(torch.from_numpy(x * 4).to(torch.bfloat16))
    assert np.array_equal(so.channel_norm(Xb4), c * 4)


# ---------------------------------------------------------------- no Stage 1: 8:8 split as out_n:8 outliers + dense inliers
DENSE_CFGS = [so.Config(1, so.GRAN_DENSE, 32, so.SCALE_OCP_FLOOR),
              so.Config(2, so.GRAN_DENSE, 32, so.SCALE_CEIL_NOSAT),
              so.Config(0, so.GRAN_DENSE, 64, so.SCALE_OCP_FLOOR),
              so.Config(1, so.GRAN_DENSE, 64, so.SCALE_CEIL_NOSAT)]


@pytest.mark.parametrize("cfg", DENSE_CFGS)
def test_dense_inliers_match_independent_dense_definition(cfg):
    """without pruning, W_in + W_out is the quantized W of an independent routine, with and without a channel weight"""
    for seed, cw in ((0, None), (1, lognormal_channel_weight(512, 7))):
        Wb = tiny_W(48, 512, seed)
        p = so.decompose(Wb, cfg, cw)
        assert p.in_code.shape == (48, 512) and p.in_meta.size == 0
        W_in, W_out = so.dequant_weights(p)
        ref_in, ref_out, slots, mask_out = decompose_dense(Wb, cfg.out_n, None, cfg.in_block,
                                                           cfg.scale_rule == so.SCALE_OCP_FLOOR, cw)
        assert slots.all()
        assert np.array_equal(W_out, ref_out)
        assert np.array_equal(W_in, ref_in)
        # every position that is not an outlier holds its own code; the outlier positions hold +0
        assert (p.in_code[mask_out] == 0).all()
        assert ((W_out != 0).reshape(48, 64, 8).sum(-1) <= cfg.out_n).all()
        assert not ((W_in != 0) & (W_out != 0)).any()


@pytest.mark.parametrize("out_n", [1, 2])
def test_dense_inliers_share_stage_2_with_the_pruned_patterns(out_n):
    """Stage 2 does not depend on Stage 1: the outlier arrays are those of the pair-wise and element-wise patterns"""
    Wb = tiny_W(32, 256, 11)
    d = so.decompose(Wb, so.Config(out_n, so.GRAN_DENSE, 64, so.SCALE_OCP_FLOOR))
    for gran in (so.GRAN_PAIR, so.GRAN_ELEM):
        p = so.decompose(Wb, so.Config(out_n, gran, 64, so.SCALE_OCP_FLOOR))
        assert np.array_equal(d.out_idx, p.out_idx) and np.array_equal(d.out_code, p.out_code)
        assert np.array_equal(d.out_sexp, p.out_sexp)
        # the pruned W_in is the dense W_in restricted to the kept slots whenever both use the same block scale
        Wd, _ = so.dequant_weights(d)
        Wp, _ = so.dequant_weights(p)
        same_scale = np.repeat(d.in_scale == p.in_scale, 64, axis=1)
        assert np.array_equal(np.where(same_scale & (Wp != 0), Wd, 0.0), np.where(same_scale, Wp, 0.0))


def test_dense_inliers_on_grid_weights_round_trip_exactly():
    """every element on the E2M1 * 2^E grid (one E4M3-exact dominant value per 8): nothing is lost, W_in + W_out == W"""
    rng = np.random.default_rng(13)
    N, K = 16, 256
    e2m1 = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
    W = rng.choice([-1.0, 1.0], size=(N, K)) * rng.choice(e2m1, size=(N, K)) * 0.125
    W[:, 1::32] = 0.75                                     # every block of 32 reaches 6 * 2^-3: one scale under both rules
    for g in range(K // 8):
        o = (3 * g) % 8
        if (8 * g + o) % 32 == 1:
            o += 1
        W[:, 8 * g + o] = rng.choice([-1, 1], size=N) * 16.0 * (1 + rng.integers(0, 8, size=N) / 8)
    import torch
    Wb = sdq_synth.bf16_bits(torch.from_numpy(W).to(torch.bfloat16))
    assert np.array_equal(bf16_to_f64(Wb), W)
    for rule in (so.SCALE_OCP_FLOOR, so.SCALE_CEIL_NOSAT):
        for block in (32, 64):
            p = so.decompose(Wb, so.Config(1, so.GRAN_DENSE, block, rule))
            W_in, W_out = so.dequant_weights(p)
            assert np.array_equal(W_in + W_out, W)
            assert (np.abs(W_out[W_out != 0]) >= 16).all() and (W_out != 0).sum() == N * K // 8


def test_dense_inliers_without_outliers_is_plain_block_scaled_4bit_quantization():
    """out_n = 0 and no pruning: the weight path is the activation path's 4-bit quantizer applied to W"""
    Wb = tiny_W(24, 512, 17)
    for block in (32, 64):
        for rule in (so.SCALE_OCP_FLOOR, so.SCALE_CEIL_NOSAT):
            cfg = so.Config(0, so.GRAN_DENSE, block, rule)
            p = so.decompose(Wb, cfg)
            q = so.quantize_act(Wb, cfg)
            assert np.array_equal(p.in_code, q.xq4_code) and np.array_equal(p.in_scale, q.xq4_scale)
            assert p.out_code.size == 0


def test_unknown_inlier_pattern_rejected():
    for out_n, gran in ((1, 9), (1, -1), (2, so.gran_keep(2))):      # the last: nothing would be left for the inliers
        with pytest.raises(ValueError):
            so.decompose(tiny_W(8, 128, 0), so.Config(out_n, gran, 64, so.SCALE_OCP_FLOOR))


# ---------------------------------------------------------------- n:8 sparsification + out_n:8 outliers + (n - out_n):8 inliers
KEEP_CFGS = [(7, 1, 32, so.SCALE_OCP_FLOOR), (6, 2, 32, so.SCALE_CEIL_NOSAT), (6, 1, 64, so.SCALE_OCP_FLOOR),
             (4, 0, 32, so.SCALE_OCP_FLOOR), (3, 2, 32, so.SCALE_OCP_FLOOR)]


@pytest.mark.parametrize("n,out_n,block,rule", KEEP_CFGS)
def test_keep_n_of_8_matches_independent_dense_definition(n, out_n, block, rule):
    cfg = so.Config(out_n, so.gran_keep(n), block, rule)
    for seed, cw in ((2, None), (3, lognormal_channel_weight(512, 9))):
        Wb = tiny_W(40, 512, seed)
        p = so.decompose(Wb, cfg, cw)
        W_in, W_out = so.dequant_weights(p)
        ref_in, ref_out, slots, mask_out = decompose_dense(Wb, out_n, n, block, rule == so.SCALE_OCP_FLOOR, cw)
        assert np.array_equal(W_out, ref_out) and np.array_equal(W_in, ref_in)
        assert ((slots & ~mask_out).reshape(40, 64, 8).sum(-1) == n - out_n).all()
        assert (((W_in != 0) | (W_out != 0)).reshape(40, 64, 8).sum(-1) <= n).all()
        assert (p.in_code[~(slots & ~mask_out)] == 0).all()


@pytest.mark.parametrize("n,out_n", [(7, 1), (6, 2), (5, 1)])
def test_keep_n_of_8_is_the_papers_stage_order(n, out_n):
    """sparsify to n:8 first, then take the out_n largest of the survivors (the paper's order), written out with numpy on
    magnitudes that are distinct inside every S-Vector: same outliers, same inliers, same dropped values"""
    rng = np.random.default_rng(21)
    N, K = 24, 256
    import torch
    mags = np.stack([rng.permutation(8) for _ in range(N * K // 8)]).reshape(N, K) + 1.0     # 1..8, distinct per group
    W = mags * rng.choice([-1.0, 1.0], size=(N, K)) * 0.03125
    Wb = sdq_synth.bf16_bits(torch.from_numpy(W).to(torch.bfloat16))
    assert np.array_equal(bf16_to_f64(Wb), W)
    p = so.decompose(Wb, so.Config(out_n, so.gran_keep(n), 32, so.SCALE_CEIL_NOSAT))
    W_in, W_out = so.dequant_weights(p)
    g = mags.reshape(N, K // 8, 8)
    survive = g > (8 - n)                       # Stage 1: the 8 - n smallest of every 8 go
    outl = g > (8 - out_n)                      # Stage 2: the out_n largest survivors
    inl = survive & ~outl
    assert np.array_equal((W_out != 0).reshape(g.shape), outl)
    # every surviving inlier is representable here (|w| * 32 in 1..8 with one scale per 32: at most one step of rounding,
    # never to zero), so the support of W_in is exactly the inlier set
    assert np.array_equal((W_in != 0).reshape(g.shape), inl)
    assert np.array_equal(W_out, np.where(outl.reshape(N, K), W, 0.0))


def test_keep_8_of_8_is_the_dense_pattern_and_keep_less_only_removes_values():
    Wb = tiny_W(16, 256, 23)
    d = so.decompose(Wb, so.Config(1, so.GRAN_DENSE, 32, so.SCALE_OCP_FLOOR))
    assert so.gran_keep(8) == so.GRAN_DENSE
    prev = so.dequant_weights(d)[0] != 0
    for n in (7, 6, 5, 4, 3, 2):
        p = so.decompose(Wb, so.Config(1, so.gran_keep(n), 32, so.SCALE_OCP_FLOOR))
        assert np.array_equal(p.out_idx, d.out_idx) and np.array_equal(p.out_code, d.out_code)
        nz = so.dequant_weights(p)[0] != 0
        assert not (nz & ~prev).any()            # supports are nested as n shrinks
        prev = nz


# ---------------------------------------------------------------- two-level scaling with fp8-e4m3 Q-Vector scales
def _e4m3_values():
    import torch
    return torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).double().numpy()


def test_ue4m3_scale_code_closed_forms():
    """amax = 6 * v * 2^t returns the code of v for every positive e4m3 value; just above / below a midpoint goes to the
    right neighbour, the midpoint itself to the even code; zero gives 0, anything tiny the smallest positive code"""
    L = so.lib()
    vals = _e4m3_values()
    for t in (-20, 0, 7):
        for c in range(1, 0x7F):
            assert L.sdqo_ue4m3_scale_code(6.0 * vals[c] * 2.0 ** t, t) == c
        for c in range(1, 0x7E):
            mid = 3.0 * (vals[c] + vals[c + 1]) * 2.0 ** t
            assert L.sdqo_ue4m3_scale_code(mid, t) == (c if c % 2 == 0 else c + 1)
            assert L.sdqo_ue4m3_scale_code(mid * (1 + 2.0 ** -30), t) == c + 1
            assert L.sdqo_ue4m3_scale_code(mid * (1 - 2.0 ** -30), t) == c
    assert L.sdqo_ue4m3_scale_code(0.0, 3) == 0
    assert L.sdqo_ue4m3_scale_code(1e-30, 0) == 1


@pytest.mark.parametrize("gran,block,out_n", [(so.GRAN_PAIR, 32, 1), (so.GRAN_PAIR, 64, 2), (so.GRAN_ELEM, 32, 0), (so.GRAN_DENSE, 32, 1)])
def test_ue4m3_weights_match_independent_definition(gran, block, out_n):
    cfg = so.Config(out_n, gran, block, so.SCALE_UE4M3)
    for seed in (0, 1):
        Wb = tiny_W(48, 512, seed)
        p = so.decompose(Wb, cfg)
        W_in, W_out = so.dequant_weights(p)
        pair = {so.GRAN_PAIR: True, so.GRAN_ELEM: False, so.GRAN_DENSE: None}[gran]
        ref_in, ref_out, slots, mask_out = decompose_dense(Wb, out_n, pair, block, "ue4m3")
        assert np.array_equal(W_out, ref_out)
        assert np.array_equal(W_in, ref_in)
        _, t = two_level_quantize(np.where(slots & ~mask_out, bf16_to_f64(Wb), 0.0), slots & ~mask_out, block)
        assert np.array_equal(p.in_texp, t)
        assert (p.in_scale <= 0x7E).all()
        # the selections do not depend on the scale format
        p0 = so.decompose(Wb, so.Config(out_n, gran, block, so.SCALE_OCP_FLOOR))
        assert np.array_equal(p.in_meta, p0.in_meta) and np.array_equal(p.out_idx, p0.out_idx)
        assert np.array_equal(p.out_code, p0.out_code)


def test_ue4m3_scales_on_power_of_two_blocks_equal_the_ceil_rule():
    """blocks whose largest kept magnitude is 6 * 2^j get the scale 2^j under both rules: identical W_in"""
    rng = np.random.default_rng(31)
    N, K = 16, 256
    import torch
    W = rng.choice([-1.0, 1.0], size=(N, K)) * rng.choice([0.5, 1.0, 1.5, 2.0, 3.0, 4.0], size=(N, K))
    j = rng.integers(-4, 3, size=(N, K // 32))
    W[:, ::32] = 6.0                                       # every block reaches 6 (kept: the pair (0,1) has the largest sum)
    W[:, 1::32] = 4.0
    W = W * np.repeat(2.0 ** j, 32, axis=1)
    Wb = sdq_synth.bf16_bits(torch.from_numpy(W).to(torch.bfloat16))
    a = so.dequant_weights(so.decompose(Wb, so.Config(0, so.GRAN_PAIR, 32, so.SCALE_UE4M3)))[0]
    b = so.dequant_weights(so.decompose(Wb, so.Config(0, so.GRAN_PAIR, 32, so.SCALE_CEIL_NOSAT)))[0]
    assert np.array_equal(a, b)
    assert np.array_equal(a != 0, b != 0) and (np.abs(a).reshape(N, K // 32, 32).max(-1) == 6.0 * 2.0 ** j).all()


def test_ue4m3_scales_lower_the_inlier_error():
    """the quantization-stage observation restated on synthetic weights: e4m3 Q-Vector scales give a smaller inlier
    error than power-of-two scales under either rule (same kept positions, same block)"""
    Wb = tiny_W(128, 1024, 41)
    W = bf16_to_f64(Wb)
    errs = {}
    for rule in (so.SCALE_OCP_FLOOR, so.SCALE_CEIL_NOSAT, so.SCALE_UE4M3):
        p = so.decompose(Wb, so.Config(1, so.GRAN_PAIR, 32, rule))
        W_in, W_out = so.dequant_weights(p)
        kept = np.repeat(np.zeros_like(p.in_meta, bool), 8, axis=1)
        j0, j1 = p.in_meta & 3, (p.in_meta >> 2) & 3
        for u in range(2):
            np.put_along_axis(kept.reshape(128, -1, 8), (2 * j0 + u)[..., None], True, axis=-1)
            np.put_along_axis(kept.reshape(128, -1, 8), (2 * j1 + u)[..., None], True, axis=-1)
        kept &= (W_out == 0)
        errs[rule] = np.sqrt((((W - W_in) * kept) ** 2).sum())
    assert errs[so.SCALE_UE4M3] < 0.9 * min(errs[so.SCALE_OCP_FLOOR], errs[so.SCALE_CEIL_NOSAT]), errs


@pytest.mark.parametrize("block", [32, 64])
def test_ue4m3_activations_match_independent_definition(block):
    Xb = sdq_synth.bf16_bits(sdq_synth.make_act(24, 512, 5, n_outlier_channels=5))
    Xb[3, :] = 0                                           # an all-zero token: factor 2^0, scale codes 0
    Xb[5, 64:128] = 0                                      # all-zero Q-Vectors inside a live token
    q = so.quantize_act(Xb, so.Config(1, so.GRAN_PAIR, block, so.SCALE_UE4M3))
    A_i, A_o = so.dequant_act(q)
    ref_i, ref_o = quantize_act_dense(Xb, block, "ue4m3")
    assert np.array_equal(A_i, ref_i) and np.array_equal(A_o, ref_o)
    assert (q.xq4_scale[3] == 0).all() and q.xq8_sexp[3] == 0 and (q.xq4_scale[5, 64 // block:128 // block] == 0).all()
    # the 8-bit part does not depend on the 4-bit scale format
    q0 = so.quantize_act(Xb, so.Config(1, so.GRAN_PAIR, block, so.SCALE_OCP_FLOOR))
    assert np.array_equal(q.xq8_code, q0.xq8_code) and np.array_equal(q.xq8_sexp, q0.xq8_sexp)
    # a Q-Vector 2^20 below the token's largest value still gets the smallest positive scale, not zero
    import torch
    X = torch.zeros((1, 256), dtype=torch.bfloat16)
    X[0, 0] = 256.0
    X[0, 40] = 2.0 ** -12
    q1 = so.quantize_act(sdq_synth.bf16_bits(X), so.Config(1, so.GRAN_PAIR, 32, so.SCALE_UE4M3))
    assert q1.xq8_sexp[0] == 0 and q1.xq4_scale[0, 1] == 1 and q1.xq4_scale[0, 0] == so.lib().sdqo_ue4m3_scale_code(256.0, 0)


@pytest.mark.parametrize("rule,block", [(so.SCALE_OCP_FLOOR, 32), (so.SCALE_CEIL_NOSAT, 64), (so.SCALE_UE4M3, 32), (so.SCALE_UE4M3, 64)])
def test_values_on_rounding_boundaries_match_the_independent_definition(rule, block):
    """inputs built from exact ties (element quotients on E2M1 midpoints, block maxima on E4M3 midpoints): the oracle and
    the independent definition must break every tie the same way, for activations and for un-pruned weights"""
    from tests.tie_cases import make_tie_matrix
    tag = {so.SCALE_OCP_FLOOR: True, so.SCALE_CEIL_NOSAT: False, so.SCALE_UE4M3: "ue4m3"}[rule]
    for seed in (0, 1, 2):
        Xb = sdq_synth.bf16_bits(make_tie_matrix(24, 512, seed))
        q = so.quantize_act(Xb, so.Config(1, so.GRAN_PAIR, block, rule))
        A_i, A_o = so.dequant_act(q)
        ref_i, ref_o = quantize_act_dense(Xb, block, tag)
        assert np.array_equal(A_i, ref_i) and np.array_equal(A_o, ref_o)
        p = so.decompose(Xb, so.Config(0, so.GRAN_DENSE, block, rule))
        W_in, _ = so.dequant_weights(p)
        assert np.array_equal(W_in, decompose_dense(Xb, 0, None, block, tag)[0])
        assert np.array_equal(W_in, A_i)          # un-pruned weights without outliers = the activation 4-bit quantizer


@pytest.mark.parametrize("out_n,block,rule", [(2, 32, so.SCALE_OCP_FLOOR), (0, 32, so.SCALE_CEIL_NOSAT), (2, 64, so.SCALE_OCP_FLOOR)])
def test_s_vectors_of_4_match_independent_definition(out_n, block, rule):
    """3:4 = 1:4 + 2:4: per 4 consecutive K the largest is the outlier, the next two are inliers, the smallest goes"""
    cfg = so.Config(out_n, so.GRAN_3OF4, block, rule)
    for seed, cw in ((4, None), (5, lognormal_channel_weight(512, 11))):
        Wb = tiny_W(40, 512, seed)
        p = so.decompose(Wb, cfg, cw)
        W_in, W_out = so.dequant_weights(p)
        ref_in, ref_out, slots, mask_out = decompose_dense(Wb, out_n, "3of4", block, rule == so.SCALE_OCP_FLOOR, cw)
        assert np.array_equal(W_out, ref_out) and np.array_equal(W_in, ref_in)
        assert ((W_out != 0).reshape(40, 128, 4).sum(-1) <= (1 if out_n else 0)).all()
        assert ((slots & ~mask_out).reshape(40, 128, 4).sum(-1) == 3 - (1 if out_n else 0)).all()
        if out_n:
            assert (p.out_idx[..., 0] < 4).all() and (p.out_idx[..., 1] >= 4).all()
    with pytest.raises(ValueError):
        so.decompose(tiny_W(8, 128, 0), so.Config(1, so.GRAN_3OF4, 32, so.SCALE_OCP_FLOOR))


def test_s_vectors_of_4_hand_example():
    """one row, magnitudes 1..8 in two groups of 4: (4, 1, 3, 2 | 5, 8, 6, 7) -> outliers 4 and 8, dropped 1 and 5"""
    import torch
    row = np.array([4.0, 1.0, 3.0, 2.0, 5.0, 8.0, 6.0, 7.0] * 8) * 0.0625
    W = np.tile(row, (2, 1))
    Wb = sdq_synth.bf16_bits(torch.from_numpy(W).to(torch.bfloat16))
    p = so.decompose(Wb, so.Config(2, so.GRAN_3OF4, 32, so.SCALE_CEIL_NOSAT))
    W_in, W_out = so.dequant_weights(p)
    assert (p.out_idx == np.array([0, 5])).all()
    assert np.array_equal(W_out[0, :8], np.array([4.0, 0, 0, 0, 0, 8.0, 0, 0]) * 0.0625)
    assert np.array_equal(W_in[0, :8] != 0, np.array([0, 0, 1, 1, 0, 0, 1, 1], bool))


@pytest.mark.parametrize("gran,block,out_n", [(so.GRAN_PAIR, 64, 1), (so.GRAN_PAIR, 32, 2), (so.gran_keep(7), 32, 1)])
def test_small_order_takes_the_least_significant_values(gran, block, out_n):
    """the decomposition-stage study's "Small" control: outliers in ascending order of the metric"""
    cfg = so.Config(out_n, gran, block, so.SCALE_OCP_FLOOR, so.ORDER_SMALL)
    pair = True if gran == so.GRAN_PAIR else 7
    for seed, cw in ((6, None), (7, lognormal_channel_weight(512, 13))):
        Wb = tiny_W(40, 512, seed)
        p = so.decompose(Wb, cfg, cw)
        W_in, W_out = so.dequant_weights(p)
        ref_in, ref_out, slots, mask_out = decompose_dense(Wb, out_n, pair, block, True, cw, small=True)
        assert np.array_equal(W_out, ref_out) and np.array_equal(W_in, ref_in)
    # magnitudes 1..8 in every group: "Small" picks 1 (and 2), "Large" 8 (and 7)
    import torch
    rng = np.random.default_rng(5)
    mags = np.stack([rng.permutation(8) for _ in range(4 * 64)]).reshape(4, 512) + 1.0
    Wb = sdq_synth.bf16_bits(torch.from_numpy(mags * 0.25).to(torch.bfloat16))
    ps = so.decompose(Wb, so.Config(out_n, so.GRAN_PAIR, 64, 0, so.ORDER_SMALL))
    pl = so.decompose(Wb, so.Config(out_n, so.GRAN_PAIR, 64, 0, so.ORDER_LARGE))
    g = mags.reshape(4, 64, 8)
    assert np.array_equal(np.sort(np.take_along_axis(g, ps.out_idx.astype(int), -1), -1), np.tile(np.arange(1, out_n + 1.0), (4, 64, 1)))
    assert np.array_equal(np.sort(np.take_along_axis(g, pl.out_idx.astype(int), -1), -1), np.tile(np.arange(9 - out_n, 9.0), (4, 64, 1)))
    with pytest.raises(ValueError):
        so.decompose(Wb, so.Config(1, so.GRAN_PAIR, 64, 0, 2))
