"""GPU parity: the CUDA path against the CPU oracle, element by element, through the C-ABI."""
import numpy as np
import pytest
import torch

import sdq_synth
from oracle import sdq_oracle as so

pytestmark = pytest.mark.gpu


def sdq():
    import paper_2406_13868_b200 as m
    return m


def ocfg(out_n=1, rule=0, block=64, gran=so.GRAN_PAIR):
    return so.Config(out_n, gran, block, rule)


def y_close(y_gpu, y_ref):
    """spec criterion on the fp32 accumulator: |d| <= 1e-3 * (|y| + 1e-2)"""
    d = np.abs(y_gpu.astype(np.float64) - y_ref)
    tol = 1e-3 * (np.abs(y_ref) + 1e-2)
    return d, tol


def run_case(M, N, K, seed, out_n=1, rule=0, n_out_ch=None, check_rows=None, block=64, gran=so.GRAN_PAIR):
    m = sdq()
    cfg = m.Config(out_n, gran, block, rule)
    W = sdq_synth.make_weight(N, K, seed)
    X = sdq_synth.make_act(M, K, seed, n_outlier_channels=n_out_ch)
    p = m.sdq_decompose(W.cuda(), cfg)
    xq = m.sdq_quantize_act(X.cuda(), cfg)
    y32 = m.sdq_linear(xq, p, f32=True)
    y16 = m.sdq_linear(xq, p)
    assert m.device_status() == 0
    op = so.decompose(sdq_synth.bf16_bits(W), ocfg(out_n, rule, block, gran))
    oq = so.quantize_act(sdq_synth.bf16_bits(X), ocfg(out_n, rule, block, gran))
    pe = {k: v.cpu().numpy() for k, v in m.packed_export(p).items()}
    ae = {k: v.cpu().numpy() for k, v in m.act_export(xq).items()}
    for name in ("in_code", "in_meta", "in_scale", "out_code", "out_idx", "out_sexp", "in_texp"):
        assert np.array_equal(pe[name], getattr(op, name)), name
    for name in ("xq4_code", "xq4_scale", "xq8_code", "xq8_sexp"):
        assert np.array_equal(ae[name], getattr(oq, name)), name
    if check_rows is None:
        yref = so.linear(oq, op)
        yg = y32.cpu().numpy()
        y16g = y16.float().cpu().numpy()
    else:
        n0, n1 = check_rows
        yref = so.linear(oq, op, n0, n1)
        yg = y32[:, n0:n1].cpu().numpy()
        y16g = y16[:, n0:n1].float().cpu().numpy()
    d, tol = y_close(yg, yref)
    assert (d <= tol).all(), (d.max(), (d / tol).max())
    # bf16 output is the round-to-nearest-even of the fp32 accumulator
    assert np.array_equal(y16g, torch.from_numpy(yg).to(torch.bfloat16).float().numpy())
    return float((d / tol).max())


def test_tiny_config_seed0():
    """C1: X 8x256 with 2 of 256 outlier channels x30, W 256x256"""
    run_case(8, 256, 256, 0, n_out_ch=2)


@pytest.mark.parametrize("out_n", [0, 1, 2])
@pytest.mark.parametrize("rule", [0, 1])
def test_patterns_and_scale_rules(out_n, rule):
    run_case(40, 256, 512, 3 + out_n, out_n=out_n, rule=rule)


@pytest.mark.parametrize("M", [1, 3, 16, 17, 33, 65, 128, 129, 300])
def test_ragged_token_counts(M):
    run_case(M, 128, 768, 10 + M)


def test_several_tiles_long_k():
    run_case(200, 384, 2816, 21)   # K = 11 x 256: more stages than the pipeline is deep


@pytest.mark.parametrize("M,N,K,out_n", [(129, 256, 512, 1), (256, 256, 768, 1), (300, 512, 1024, 2), (520, 256, 2816, 1),
                                         (384, 512, 512, 0), (1000, 1024, 256, 1)])
def test_more_than_128_tokens_few_tiles(M, N, K, out_n):
    """more than 128 tokens (256-token tiles, ragged token tails) against narrow matrices: few tiles, so the K range
    of a tile is split over a cluster"""
    run_case(M, N, K, 100 + M, out_n=out_n)


@pytest.mark.parametrize("M,N,K,out_n", [(300, 5120, 512, 1), (520, 6400, 256, 2), (257, 9600, 256, 0)])
def test_persistent_many_token_kernel(M, N, K, out_n):
    """enough 256-token tiles (80, 150, 150) for the persistent many-token instantiation: one and several tiles per
    CTA, fewer stages than ring slots, a ragged last token tile"""
    run_case(M, N, K, 200 + M, out_n=out_n)


@pytest.mark.parametrize("M,N,K,out_n,rule", [(600, 8192, 512, 1, 0), (161, 38400, 256, 1, 0), (481, 12800, 256, 2, 1), (640, 8192, 256, 0, 0),
                                              (1000, 5120, 768, 1, 0), (329, 19200, 256, 1, 1)])
def test_many_tokens_more_tiles_than_sms(M, N, K, out_n, rule):
    """many tokens and more 128 x 256 tiles than SMs, so that persistent CTAs run several tiles each; ragged last token
    tile, with and without a second 128-token record in it; sampled row tiles checked"""
    rows = (0, 256) if N <= 8192 else (N - 384, N - 128)
    run_case(M, N, K, 1700 + M, out_n=out_n, rule=rule, check_rows=rows)


def _random_shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        M = int(rng.choice([rng.integers(1, 17), rng.integers(17, 129), rng.integers(129, 700)]))
        N = 128 * int(rng.integers(1, 9))
        K = 256 * int(rng.integers(1, 13))
        out.append((M, N, K, int(rng.integers(0, 3)), int(rng.integers(0, 2))))
    return out


@pytest.mark.parametrize("M,N,K,out_n,rule", _random_shapes(24, 2024))
def test_seeded_random_shapes(M, N, K, out_n, rule):
    """seeded random token counts (few / up to 128 / several hundred), widths, depths, outlier counts and scale rules:
    every launch geometry the host logic can pick for small problems, full parity each"""
    run_case(M, N, K, 7 * M + N + K, out_n=out_n, rule=rule)


@pytest.mark.parametrize("M,N,K,out_n,rule", [(8, 256, 256, 1, 0), (1, 512, 2048, 1, 0), (16, 256, 4096, 2, 1), (33, 128, 768, 0, 0),
                                              (100, 256, 2816, 1, 0), (129, 256, 512, 1, 1), (300, 512, 1024, 2, 0),
                                              (520, 6400, 256, 1, 0)])
def test_block_32_scales_through_the_tensor_core(M, N, K, out_n, rule):
    """one E8M0 scale per 32 logical K for the inlier weights and the 4-bit activations (the literal block-32 MXFP4
    wording): executed by the sparse kind::mxf4nvf4 .block16 MMA; few tokens, cluster split K, several hundred tokens,
    and enough tiles for persistent CTAs"""
    run_case(M, N, K, 900 + M, out_n=out_n, rule=rule, block=32)


def test_block_32_one_hot_readback():
    m = sdq()
    cfg = m.Config(1, m.GRAN_PAIR, 32, 0)
    N, K = 256, 512
    W = sdq_synth.make_weight(N, K, 61)
    p = m.sdq_decompose(W.cuda(), cfg)
    X = torch.eye(K, dtype=torch.bfloat16)
    xq = m.sdq_quantize_act(X.cuda(), cfg)
    y = m.sdq_linear(xq, p, f32=True).cpu().numpy().astype(np.float64)
    W_in, W_out = so.dequant_weights(so.decompose(sdq_synth.bf16_bits(W), ocfg(block=32)))
    assert np.array_equal(y, (W_in + W_out).T)
    assert m.device_status() == 0


@pytest.mark.parametrize("M,N,K,out_n,rule", [(8, 256, 256, 1, 0), (1, 512, 2048, 1, 0), (16, 256, 4096, 2, 1), (33, 128, 768, 0, 0),
                                              (100, 256, 2816, 1, 0), (128, 1024, 4096, 1, 0), (129, 256, 512, 1, 1),
                                              (300, 512, 1024, 2, 0), (520, 6400, 256, 1, 0), (700, 2560, 1024, 1, 1)])
def test_dense_inliers_through_the_tensor_core(M, N, K, out_n, rule):
    """no Stage 1 (8:8 split as out_n:8 outliers + dense 4-bit inliers, one scale per 32 K): packed arrays bit-exact, the
    inlier product on the dense kind::mxf4 MMA; few tokens, cluster split K, several hundred tokens, persistent CTAs"""
    run_case(M, N, K, 1200 + M, out_n=out_n, rule=rule, block=32, gran=so.GRAN_DENSE)


@pytest.mark.parametrize("n,M,N,K,out_n,rule", [(7, 8, 256, 256, 1, 0), (7, 1, 512, 2048, 1, 0), (6, 16, 256, 4096, 2, 1), (4, 33, 128, 768, 0, 0),
                                                (7, 100, 256, 2816, 1, 0), (6, 129, 256, 512, 1, 1), (3, 300, 512, 1024, 2, 0),
                                                (7, 520, 6400, 256, 1, 0), (5, 64, 1024, 1024, 1, 0)])
def test_n_of_8_sparsification_with_outliers_and_inliers_at_any_position(n, M, N, K, out_n, rule):
    """SDQ_GRAN_KEEP(n): the n most significant of every 8 survive, out_n of them as FP8 outliers, the others as MXFP4
    inliers wherever they sit (7:8 = 1:8 + 6:8 is the evaluation's headline pattern): packed arrays bit-exact, product
    through the dense 4-bit MMA"""
    run_case(M, N, K, 1500 + 10 * n + M, out_n=out_n, rule=rule, block=32, gran=so.gran_keep(n))


@pytest.mark.parametrize("M,N,K,out_n,rule", [(8, 256, 256, 2, 0), (1, 512, 2048, 2, 0), (33, 128, 768, 0, 1), (129, 256, 512, 2, 1),
                                              (520, 6400, 256, 2, 0)])
def test_s_vectors_of_4(M, N, K, out_n, rule):
    """SDQ_GRAN_3OF4 (3:4 = 1:4 + 2:4): packed arrays bit-exact, product through the dense 4-bit MMA"""
    run_case(M, N, K, 2600 + M, out_n=out_n, rule=rule, block=32, gran=so.GRAN_3OF4)


@pytest.mark.parametrize("gran,block,out_n", [(0, 64, 1), (0, 32, 2), (1, 32, 1), (3, 32, 1), (9, 32, 2)])
def test_small_order_packer_and_product(gran, block, out_n):
    """SDQ_ORDER_SMALL (the decomposition-stage study's control): the least significant values become the outliers;
    packed arrays bit-exact for every layout, the product within the criterion where the GEMM runs the pattern"""
    m = sdq()
    N, K, M = 256, 1024, 24
    cfg = m.Config(out_n, gran, block, 0, m.ORDER_SMALL)
    oc = so.Config(out_n, gran, block, 0, so.ORDER_SMALL)
    W = sdq_synth.make_weight(N, K, 2800 + gran)
    p = m.sdq_decompose(W.cuda(), cfg)
    op = so.decompose(sdq_synth.bf16_bits(W), oc)
    pe = {k: v.cpu().numpy() for k, v in m.packed_export(p).items()}
    for name in ("in_code", "in_meta", "in_scale", "out_code", "out_idx", "out_sexp"):
        assert np.array_equal(pe[name], getattr(op, name)), name
    assert not np.array_equal(op.out_idx, so.decompose(sdq_synth.bf16_bits(W), so.Config(out_n, gran, block, 0)).out_idx)
    if gran != m.GRAN_ELEM:
        X = sdq_synth.make_act(M, K, 2801)
        xq = m.sdq_quantize_act(X.cuda(), cfg)
        d, tol = y_close(m.sdq_linear(xq, p, f32=True).cpu().numpy(), so.linear(so.quantize_act(sdq_synth.bf16_bits(X), oc), op))
        assert (d <= tol).all()
    with pytest.raises(m.SdqError) as e:
        m.sdq_decompose(W.cuda(), m.Config(out_n, gran, block, 0, 2))
    assert e.value.code == 1


@pytest.mark.parametrize("M,N,K,out_n,rule", [(8, 256, 256, 1, 0), (1, 512, 2048, 1, 0), (16, 256, 4096, 2, 1), (33, 128, 768, 0, 0),
                                              (129, 256, 512, 1, 1), (300, 512, 1024, 2, 0), (520, 6400, 256, 1, 0)])
def test_element_wise_2of4_block_32_through_the_tensor_core(M, N, K, out_n, rule):
    """the literal wording (element-wise 2:4 inliers, one scale per 32 K): packed arrays bit-exact in their own canonical
    form (two kept slots and their indices per 4), the product on the dense 4-bit MMA with the dropped positions at +0"""
    run_case(M, N, K, 2900 + M, out_n=out_n, rule=rule, block=32, gran=so.GRAN_ELEM)


def test_dense_inliers_one_hot_readback_and_workspace_split():
    m = sdq()
    cfg = m.Config(1, m.GRAN_DENSE, 32, 0)
    N, K = 256, 512
    W = sdq_synth.make_weight(N, K, 71)
    p = m.sdq_decompose(W.cuda(), cfg)
    X = torch.eye(K, dtype=torch.bfloat16)
    xq = m.sdq_quantize_act(X.cuda(), cfg)
    y = m.sdq_linear(xq, p, f32=True).cpu().numpy().astype(np.float64)
    op = so.decompose(sdq_synth.bf16_bits(W), ocfg(block=32, gran=so.GRAN_DENSE))
    W_in, W_out = so.dequant_weights(op)
    assert np.array_equal(y, (W_in + W_out).T)
    # K split through a caller workspace: same criterion, identical from call to call
    M = 7
    Xs = sdq_synth.make_act(M, K, 72)
    xs = m.sdq_quantize_act(Xs.cuda(), cfg)
    ws = m.make_workspace(M, N, K, cfg, "cuda")
    assert ws is not None
    y1 = m.sdq_linear(xs, p, f32=True, workspace=ws)
    y2 = m.sdq_linear(xs, p, f32=True, workspace=ws)
    assert torch.equal(y1, y2)
    d, tol = y_close(y1.cpu().numpy(), so.linear(so.quantize_act(sdq_synth.bf16_bits(Xs), op.cfg), op))
    assert (d <= tol).all()
    assert m.device_status() == 0
    # the dense 4-bit tensor-core kind has no scale per 64 K
    with pytest.raises(m.SdqError) as e:
        m.sdq_decompose(W.cuda(), m.Config(1, m.GRAN_DENSE, 64, 0))
    assert e.value.code == 4
    for out_n, gran in ((2, m.gran_keep(2)), (1, 9)):             # nothing left for the inliers; unknown pattern
        with pytest.raises(m.SdqError) as e:
            m.sdq_decompose(W.cuda(), m.Config(out_n, gran, 32, 0))
        assert e.value.code == 1


@pytest.mark.parametrize("M,N,K,out_n", [(8, 256, 256, 1), (1, 512, 2048, 1), (16, 256, 4096, 2), (33, 128, 768, 0), (100, 256, 2816, 1),
                                         (128, 1024, 4096, 1), (129, 256, 512, 1), (300, 512, 1024, 2), (520, 6400, 256, 1),
                                         (700, 2560, 1024, 1)])
def test_two_level_e4m3_scales_through_the_tensor_core(M, N, K, out_n):
    """SDQ_SCALE_UE4M3: E4M3 Q-Vector scale codes for inlier weights and 4-bit activations (kind::mxf4nvf4 .block16 with
    its scale format switched), accumulator in units of the row and token factors, multiplied back in by the epilogue:
    few tokens, cluster split K, several hundred tokens, persistent tiles"""
    run_case(M, N, K, 2300 + M, out_n=out_n, rule=2, block=32)


def test_two_level_e4m3_scales_one_hot_readback_and_workspace_split():
    m = sdq()
    cfg = m.Config(1, m.GRAN_PAIR, 32, m.SCALE_UE4M3)
    oc = so.Config(1, so.GRAN_PAIR, 32, so.SCALE_UE4M3)
    N, K = 256, 512
    W = sdq_synth.make_weight(N, K, 2401)
    W[9, :] = W[9, :] * 2.0 ** -14                     # a row with a very different factor
    p = m.sdq_decompose(W.cuda(), cfg)
    X = torch.eye(K, dtype=torch.bfloat16)            # 1.0 is exact in the 8-bit format, not with a 4-bit code times an E4M3 scale
    xq = m.sdq_quantize_act(X.cuda(), cfg)
    y = m.sdq_linear(xq, p, f32=True).cpu().numpy().astype(np.float64)
    op = so.decompose(sdq_synth.bf16_bits(W), oc)
    oq = so.quantize_act(sdq_synth.bf16_bits(X), oc)
    A_i, A_o = so.dequant_act(oq)
    W_in, W_out = so.dequant_weights(op)
    # one non-zero per token: every output is a single product pair, exact in fp32 up to the final sum of the two parts
    a_i, a_o = np.diag(A_i), np.diag(A_o)
    assert (a_o == 1.0).all()
    ref = (W_in * a_i[None, :] + W_out).T
    assert np.allclose(y, ref, rtol=2e-7, atol=0)
    M = 7
    Xs = sdq_synth.make_act(M, K, 2402)
    xs = m.sdq_quantize_act(Xs.cuda(), cfg)
    ws = m.make_workspace(M, N, K, cfg, "cuda")
    y1 = m.sdq_linear(xs, p, f32=True, workspace=ws)
    y2 = m.sdq_linear(xs, p, f32=True, workspace=ws)
    assert torch.equal(y1, y2)
    d, tol = y_close(y1.cpu().numpy(), so.linear(so.quantize_act(sdq_synth.bf16_bits(Xs), oc), op))
    assert (d <= tol).all()
    assert m.device_status() == 0


@pytest.mark.parametrize("M,K", [(13, 256), (21, 11008), (3, 16640)])
def test_two_level_e4m3_scales_quantizer(M, K):
    """SDQ_SCALE_UE4M3 activations (single-pass and two-pass quantizer): E4M3 scale codes and element codes bit-exact,
    including an all-zero token, all-zero Q-Vectors, an infinity and a Q-Vector far below the token's maximum"""
    m = sdq()
    cfg = m.Config(1, m.GRAN_PAIR, 32, m.SCALE_UE4M3)
    X = sdq_synth.make_act(M, K, 2100 + M)
    X[1, :] = 0
    X[2, 64:160] = 0
    X[0, 5] = float("inf")
    X[2, 200:232] = X[2, 200:232] * 2.0 ** -22
    xq = m.sdq_quantize_act(X.cuda(), cfg)
    oq = so.quantize_act(sdq_synth.bf16_bits(X), so.Config(1, so.GRAN_PAIR, 32, so.SCALE_UE4M3))
    ae = {k: v.cpu().numpy() for k, v in m.act_export(xq).items()}
    for name in ("xq4_scale", "xq4_code", "xq8_code", "xq8_sexp"):
        assert np.array_equal(ae[name], getattr(oq, name)), name
    with pytest.raises(m.SdqError) as e:
        m.sdq_quantize_act(X.cuda(), m.Config(1, m.GRAN_PAIR, 64, m.SCALE_UE4M3))
    assert e.value.code == 4


@pytest.mark.parametrize("out_n", [0, 1, 2])
def test_two_level_e4m3_scales_packer(out_n):
    m = sdq()
    N, K = 256, 1024
    W = sdq_synth.make_weight(N, K, 2200 + out_n)
    W[3, :] = 0
    W[5, 32:96] = 0
    W[7, :] = W[7, :] * 2.0 ** -30
    rng = np.random.default_rng(3)
    c = np.exp(rng.normal(0.0, 1.0, K)).astype(np.float32)
    for cw in (None, c):
        p = m.sdq_decompose(W.cuda(), m.Config(out_n, m.GRAN_PAIR, 32, m.SCALE_UE4M3), col_weight=None if cw is None else torch.from_numpy(cw).cuda())
        op = so.decompose(sdq_synth.bf16_bits(W), so.Config(out_n, so.GRAN_PAIR, 32, so.SCALE_UE4M3), col_weight=cw)
        pe = {k: v.cpu().numpy() for k, v in m.packed_export(p).items()}
        for name in ("in_texp", "in_scale", "in_code", "in_meta", "out_code", "out_idx", "out_sexp"):
            assert np.array_equal(pe[name], getattr(op, name)), name
    for gran, block in ((m.GRAN_ELEM, 32), (m.GRAN_PAIR, 64), (m.GRAN_DENSE, 32)):
        with pytest.raises(m.SdqError) as e:
            m.sdq_decompose(W.cuda(), m.Config(out_n, gran, block, m.SCALE_UE4M3))
        assert e.value.code == 4


@pytest.mark.parametrize("rule,block", [(0, 64), (1, 64), (0, 32), (1, 32), (2, 32)])
def test_values_on_rounding_boundaries(rule, block):
    """inputs built from exact ties (element quotients on E2M1 midpoints, block maxima on E4M3 midpoints, blocks far below
    the row maximum): quantizer and packer (pair-wise and un-pruned) bit-exact against the oracle, product within the
    criterion"""
    from tests.tie_cases import make_tie_matrix
    m = sdq()
    for seed in (0, 1):
        X = make_tie_matrix(40, 1024, 10 + seed)
        W = make_tie_matrix(128, 1024, 20 + seed)
        grans = [m.GRAN_PAIR] + ([m.GRAN_DENSE] if (block == 32 and rule != 2) else [])
        for gran in grans:
            for out_n in (0, 1):
                cfg, oc = m.Config(out_n, gran, block, rule), so.Config(out_n, gran, block, rule)
                xq = m.sdq_quantize_act(X.cuda(), cfg)
                p = m.sdq_decompose(W.cuda(), cfg)
                oq = so.quantize_act(sdq_synth.bf16_bits(X), oc)
                op = so.decompose(sdq_synth.bf16_bits(W), oc)
                ae = {k: v.cpu().numpy() for k, v in m.act_export(xq).items()}
                pe = {k: v.cpu().numpy() for k, v in m.packed_export(p).items()}
                for name in ("xq4_scale", "xq4_code", "xq8_code", "xq8_sexp"):
                    assert np.array_equal(ae[name], getattr(oq, name)), (name, gran, out_n)
                for name in ("in_texp", "in_scale", "in_code", "in_meta", "out_code", "out_idx", "out_sexp"):
                    assert np.array_equal(pe[name], getattr(op, name)), (name, gran, out_n)
                d, tol = y_close(m.sdq_linear(xq, p, f32=True).cpu().numpy(), so.linear(oq, op))
                assert (d <= tol).all(), (gran, out_n, d.max())
    assert m.device_status() == 0


def test_error_order_of_the_configurations_on_the_gpu():
    """the whole CUDA path against the unquantized product (fp64 on the GPU) on a synthetic layer: outliers lower the
    error, 7:8 = 1:8 + 6:8 beats dense 4-bit, 50 % sparsity costs most, E4M3 scales help"""
    m = sdq()
    M, N, K = 256, 1024, 4096
    X = sdq_synth.make_act(M, K, 2701).cuda()
    W = sdq_synth.make_weight(N, K, 2702).cuda()
    ref = X.double() @ W.double().T

    def err(cfg):
        y = m.sdq_linear(m.sdq_quantize_act(X, cfg), m.sdq_decompose(W, cfg), f32=True)
        return float((y.double() - ref).norm() / ref.norm())
    e48_0, e48_1, e48_2 = (err(m.Config(n, m.GRAN_PAIR, 32, 0)) for n in (0, 1, 2))
    e78, e88, e88_0 = err(m.Config(1, m.gran_keep(7), 32, 0)), err(m.Config(1, m.GRAN_DENSE, 32, 0)), err(m.Config(0, m.GRAN_DENSE, 32, 0))
    e34, e_ue = err(m.Config(2, m.GRAN_3OF4, 32, 0)), err(m.Config(1, m.GRAN_PAIR, 32, m.SCALE_UE4M3))
    assert m.device_status() == 0
    assert e48_0 > e48_1 > e48_2 and e88 < e78 < e48_2 and e78 < e88_0 and e88 < e34 < e48_1 and e_ue < e48_1, \
        (e48_0, e48_1, e48_2, e78, e88, e88_0, e34, e_ue)


def test_one_hot_readback_512_tokens():
    m = sdq()
    cfg = m.Config()
    N, K = 256, 512
    W = sdq_synth.make_weight(N, K, 6)
    p = m.sdq_decompose(W.cuda(), cfg)
    X = torch.eye(K, dtype=torch.bfloat16)
    xq = m.sdq_quantize_act(X.cuda(), cfg)
    y = m.sdq_linear(xq, p, f32=True).cpu().numpy().astype(np.float64)
    W_in, W_out = so.dequant_weights(so.decompose(sdq_synth.bf16_bits(W), ocfg()))
    assert np.array_equal(y, (W_in + W_out).T)
    assert m.device_status() == 0


@pytest.mark.parametrize("M,N,K,out_n", [(1, 512, 2048, 1), (16, 256, 4096, 1), (7, 1024, 1024, 2), (100, 256, 2816, 1),
                                         (16, 256, 512, 0), (3, 128, 4096, 1)])
def test_split_k_with_workspace(M, N, K, out_n):
    """few tokens + workspace: K split over several thread blocks, partial tiles added in split order;
    the result must meet the same criterion and be identical from call to call"""
    m = sdq()
    cfg = m.Config(out_n, m.GRAN_PAIR, 64, 0)
    W = sdq_synth.make_weight(N, K, 200 + M)
    X = sdq_synth.make_act(M, K, 200 + M)
    p = m.sdq_decompose(W.cuda(), cfg)
    xq = m.sdq_quantize_act(X.cuda(), cfg)
    ws = m.make_workspace(M, N, K, cfg, "cuda")
    assert ws is not None and m.workspace_size(M, N, K, cfg) == ws.numel()
    y1 = m.sdq_linear(xq, p, f32=True, workspace=ws)
    y2 = m.sdq_linear(xq, p, f32=True, workspace=ws)     # workspace is left ready for the next call
    y16 = m.sdq_linear(xq, p, workspace=ws)
    assert m.device_status() == 0
    assert torch.equal(y1, y2)
    assert torch.equal(y16, y1.to(torch.bfloat16))
    yref = so.linear(so.quantize_act(sdq_synth.bf16_bits(X), ocfg(out_n)), so.decompose(sdq_synth.bf16_bits(W), ocfg(out_n)))
    d, tol = y_close(y1.cpu().numpy(), yref)
    assert (d <= tol).all(), (d.max(), (d / tol).max())
    with pytest.raises(m.SdqError) as e:
        m.sdq_linear(xq, p, workspace=ws[:256])
    assert e.value.code == 5


@pytest.mark.parametrize("M,N,K,out_n", [(1, 512, 4096, 1), (16, 1024, 4096, 1), (32, 256, 2048, 2), (5, 4096, 1024, 1),
                                         (16, 256, 1024, 0), (2, 128, 11008, 1), (33, 512, 4096, 1), (128, 1024, 4096, 1),
                                         (100, 256, 11008, 2), (64, 4096, 2048, 1)])
def test_cluster_split_k_few_tokens(M, N, K, out_n):
    """up to 128 tokens without a workspace: the thread blocks of a row tile form a cluster and add their partial
    tiles through distributed shared memory in rank order -- same criterion, identical from call to call"""
    m = sdq()
    cfg = m.Config(out_n, m.GRAN_PAIR, 64, 0)
    W = sdq_synth.make_weight(N, K, 300 + M)
    X = sdq_synth.make_act(M, K, 300 + M)
    p = m.sdq_decompose(W.cuda(), cfg)
    xq = m.sdq_quantize_act(X.cuda(), cfg)
    y1 = m.sdq_linear(xq, p, f32=True)
    y2 = m.sdq_linear(xq, p, f32=True)
    y16 = m.sdq_linear(xq, p)
    assert m.device_status() == 0
    assert torch.equal(y1, y2)
    assert torch.equal(y16, y1.to(torch.bfloat16))
    yref = so.linear(so.quantize_act(sdq_synth.bf16_bits(X), ocfg(out_n)), so.decompose(sdq_synth.bf16_bits(W), ocfg(out_n)))
    d, tol = y_close(y1.cpu().numpy(), yref)
    assert (d <= tol).all(), (d.max(), (d / tol).max())


@pytest.mark.parametrize("M,N,K,out_n", [(5, 19200, 2048, 1), (64, 22016, 2304, 1), (100, 19200, 2048, 2), (16, 38400, 2048, 0), (7, 19200, 512, 1)])
def test_few_tokens_more_row_tiles_than_sms(M, N, K, out_n):
    """few tokens against a very wide matrix: more row tiles than SMs, K still split in two, the grid runs in waves"""
    m = sdq()
    cfg = m.Config(out_n, m.GRAN_PAIR, 64, 0)
    W = sdq_synth.make_weight(N, K, 2500 + M)
    X = sdq_synth.make_act(M, K, 2501 + M)
    p = m.sdq_decompose(W.cuda(), cfg)
    xq = m.sdq_quantize_act(X.cuda(), cfg)
    y1 = m.sdq_linear(xq, p, f32=True)
    y2 = m.sdq_linear(xq, p, f32=True)
    y16 = m.sdq_linear(xq, p)
    assert m.device_status() == 0
    assert torch.equal(y1, y2) and torch.equal(y16, y1.to(torch.bfloat16))
    oq = so.quantize_act(sdq_synth.bf16_bits(X), ocfg(out_n))
    RT = N // 128
    for t in (0, 1, RT // 2, RT - 2, RT - 1):
        op = so.decompose(sdq_synth.bf16_bits(W[128 * t:128 * t + 128]), ocfg(out_n))
        d, tol = y_close(y1[:, 128 * t:128 * t + 128].cpu().numpy(), so.linear(oq, op))
        assert (d <= tol).all(), (t, d.max())


def test_one_hot_readback_through_the_tensor_core():
    """X = identity rows (1.0 is exact in both activation formats): Y^T must equal W_in + W_out exactly"""
    m = sdq()
    cfg = m.Config()
    N, K = 128, 512
    W = sdq_synth.make_weight(N, K, 5)
    p = m.sdq_decompose(W.cuda(), cfg)
    X = torch.eye(K, dtype=torch.bfloat16)
    xq = m.sdq_quantize_act(X.cuda(), cfg)
    y = m.sdq_linear(xq, p, f32=True).cpu().numpy().astype(np.float64)
    W_in, W_out = so.dequant_weights(so.decompose(sdq_synth.bf16_bits(W), ocfg()))
    assert np.array_equal(y, (W_in + W_out).T)


def test_hardware_converters_match_oracle_exhaustively():
    """all 65536 bf16 patterns through the activation quantizer (finite ones), several magnitudes"""
    m = sdq()
    bits = np.arange(65536, dtype=np.uint16)
    finite = (bits & 0x7F80) != 0x7F80
    vals = bits[finite]
    K = 256
    pad = (-len(vals)) % K
    vals = np.concatenate([vals, np.zeros(pad, np.uint16)])
    rng = np.random.default_rng(0)
    rng.shuffle(vals)
    Xb = vals.reshape(-1, K)
    X = sdq_synth.bits_to_bf16(Xb)
    for rule in (0, 1):
        cfg = m.Config(1, m.GRAN_PAIR, 64, rule)
        ae = {k: v.cpu().numpy() for k, v in m.act_export(m.sdq_quantize_act(X.cuda(), cfg)).items()}
        oq = so.quantize_act(Xb, ocfg(1, rule))
        for name in ("xq4_code", "xq4_scale", "xq8_code", "xq8_sexp"):
            assert np.array_equal(ae[name], getattr(oq, name)), name
    # and sorted by magnitude so that blocks hold similar exponents (exercises every rounding boundary)
    order = np.argsort(vals & 0x7FFF, kind="stable")
    Xb2 = vals[order].reshape(-1, K)
    ae = {k: v.cpu().numpy() for k, v in m.act_export(m.sdq_quantize_act(sdq_synth.bits_to_bf16(Xb2).cuda(), m.Config())).items()}
    oq = so.quantize_act(Xb2, ocfg())
    for name in ("xq4_code", "xq4_scale", "xq8_code", "xq8_sexp"):
        assert np.array_equal(ae[name], getattr(oq, name)), name


@pytest.mark.parametrize("M,K", [(13, 256), (8, 2048), (21, 11008), (5, 16384), (3, 16640), (9, 20480)])
@pytest.mark.parametrize("rule,block", [(0, 64), (1, 64), (0, 32), (1, 32)])
def test_activation_quantizer_row_lengths(M, K, rule, block):
    """Rows up to 16384 take the single-launch cluster kernel (1..8 CTAs per group of 8 tokens), longer rows the
    two-launch path; both must give the oracle's codes and scales bit for bit, ragged token groups included."""
    m = sdq()
    cfg = m.Config(1, m.GRAN_PAIR, block, rule)
    X = sdq_synth.make_act(M, K, 100 + M, n_outlier_channels=max(1, K // 100))
    X[M // 2, K // 3] = float("inf")            # saturates, must not poison the row
    X[0, :64] = 0.0                             # an all-zero Q-Vector
    xq = m.sdq_quantize_act(X.cuda(), cfg)
    assert m.device_status() == 0
    oq = so.quantize_act(sdq_synth.bf16_bits(X), ocfg(1, rule, block))
    ae = {k: v.cpu().numpy() for k, v in m.act_export(xq).items()}
    for name in ("xq4_code", "xq4_scale", "xq8_code", "xq8_sexp"):
        assert np.array_equal(ae[name], getattr(oq, name)), name


@pytest.mark.parametrize("gran,block", [(1, 64), (0, 32), (0, 64), (2, 32), (3, 32), (9, 32)])
@pytest.mark.parametrize("out_n", [0, 1, 2])
def test_product_metric_packer(gran, block, out_n):
    """sdq_decompose_metric: selections by |w| * c[k]; packed arrays bit-exact against the oracle for the tensor-core
    layout and for the literal readings, the product-metric weights run through the GEMM, and bad channel weights are
    reported."""
    m = sdq()
    N, K, M = 256, 1024, 24
    cfg = m.Config(out_n, gran, block, 0)
    oc = so.Config(out_n, gran, block, 0)
    W = sdq_synth.make_weight(N, K, 40 + out_n)
    if gran == m.GRAN_3OF4 and out_n == 1:          # one outlier per 4 is two per 8: there is no such configuration
        with pytest.raises(m.SdqError) as ei:
            m.sdq_decompose(W.cuda(), cfg)
        assert ei.value.code == 1
        return
    rng = np.random.default_rng(17)
    c = np.exp(rng.normal(0.0, 1.0, K)).astype(np.float32)
    c[rng.integers(0, K, 12)] *= 30.0
    c[5] = 0.0                                    # a dead input channel never wins a selection
    p = m.sdq_decompose(W.cuda(), cfg, col_weight=torch.from_numpy(c).cuda())
    op = so.decompose(sdq_synth.bf16_bits(W), oc, col_weight=c)
    pe = {k: v.cpu().numpy() for k, v in m.packed_export(p).items()}
    for name in ("in_code", "in_meta", "in_scale", "out_code", "out_idx", "out_sexp"):
        assert np.array_equal(pe[name], getattr(op, name)), name
    # it does change the selection (otherwise the test would prove nothing)
    om = so.decompose(sdq_synth.bf16_bits(W), oc)
    if gran >= m.GRAN_DENSE:
        # no pattern metadata: the metric shows in the outlier positions, or (7:8 with no outliers) in what is dropped;
        # 8:8 with no outliers has no selection at all
        if out_n:
            assert not np.array_equal(op.out_idx, om.out_idx)
        elif gran > m.GRAN_DENSE:
            assert not np.array_equal(op.in_code, om.in_code)
    else:
        assert not np.array_equal(op.in_meta, om.in_meta)
    if gran != m.GRAN_ELEM:
        X = sdq_synth.make_act(M, K, 41)
        xq = m.sdq_quantize_act(X.cuda(), cfg)
        y = m.sdq_linear(xq, p, f32=True).cpu().numpy()
        oq = so.quantize_act(sdq_synth.bf16_bits(X), oc)
        d, tol = y_close(y, so.linear(oq, op))
        assert (d <= tol).all()
    for bad in (-1.0, float("inf"), float("nan")):
        cb = c.copy()
        cb[100] = bad
        with pytest.raises(m.SdqError) as ei:
            m.sdq_decompose(W.cuda(), cfg, col_weight=torch.from_numpy(cb).cuda())
        assert ei.value.code == 6


@pytest.mark.parametrize("M", [5, 200])
def test_leading_dimensions_larger_than_the_row(M):
    """W, X and Y are views into wider buffers (ldw > K, ldx > K, ldy > N); nothing outside the views may be written"""
    m = sdq()
    cfg = m.Config()
    N, K = 256, 512
    W = sdq_synth.make_weight(N, K, 71)
    X = sdq_synth.make_act(M, K, 72)
    Wbig = torch.full((N, K + 64), 7.0, dtype=torch.bfloat16, device="cuda")
    Xbig = torch.full((M, K + 24), -3.0, dtype=torch.bfloat16, device="cuda")
    Wbig[:, :K] = W.cuda()
    Xbig[:, :K] = X.cuda()
    p = m.sdq_decompose(Wbig[:, :K], cfg)
    xq = m.sdq_quantize_act(Xbig[:, :K], cfg)
    Ybig = torch.full((M, N + 40), 123.0, dtype=torch.bfloat16, device="cuda")
    Y32big = torch.full((M, N + 8), 123.0, dtype=torch.float32, device="cuda")
    m.sdq_linear(xq, p, Ybig[:, :N])
    m.sdq_linear(xq, p, Y32big[:, :N], f32=True)
    assert m.device_status() == 0
    op = so.decompose(sdq_synth.bf16_bits(W), ocfg())
    oq = so.quantize_act(sdq_synth.bf16_bits(X), ocfg())
    pe = {k: v.cpu().numpy() for k, v in m.packed_export(p).items()}
    ae = {k: v.cpu().numpy() for k, v in m.act_export(xq).items()}
    for name in ("in_code", "in_meta", "in_scale", "out_code", "out_idx", "out_sexp"):
        assert np.array_equal(pe[name], getattr(op, name)), name
    for name in ("xq4_code", "xq4_scale", "xq8_code", "xq8_sexp"):
        assert np.array_equal(ae[name], getattr(oq, name)), name
    y32 = Y32big[:, :N].cpu().numpy()
    d, tol = y_close(y32, so.linear(oq, op))
    assert (d <= tol).all()
    assert np.array_equal(Ybig[:, :N].float().cpu().numpy(), torch.from_numpy(y32).to(torch.bfloat16).float().numpy())
    assert (Ybig[:, N:] == 123.0).all() and (Y32big[:, N:] == 123.0).all()


def test_leading_dimension_of_y_in_the_many_token_kernel():
    """ldy > N where persistent thread blocks run several tiles each (the epilogue that stores under the next tile's K
    loop): sampled row tiles against the oracle, bf16 = rounded fp32, nothing written outside the view"""
    m = sdq()
    cfg = m.Config()
    M, N, K = 601, 6400, 256
    W = sdq_synth.make_weight(N, K, 73)
    X = sdq_synth.make_act(M, K, 74)
    p = m.sdq_decompose(W.cuda(), cfg)
    xq = m.sdq_quantize_act(X.cuda(), cfg)
    Ybig = torch.full((M + 3, N + 72), 123.0, dtype=torch.bfloat16, device="cuda")
    Y32big = torch.full((M + 3, N + 8), 123.0, dtype=torch.float32, device="cuda")
    m.sdq_linear(xq, p, Ybig[:M, :N])
    m.sdq_linear(xq, p, Y32big[:M, :N], f32=True)
    assert m.device_status() == 0
    assert (Ybig[:, N:] == 123.0).all() and (Ybig[M:] == 123.0).all()
    assert (Y32big[:, N:] == 123.0).all() and (Y32big[M:] == 123.0).all()
    assert torch.equal(Ybig[:M, :N], Y32big[:M, :N].to(torch.bfloat16))
    oq = so.quantize_act(sdq_synth.bf16_bits(X), ocfg())
    for t in (0, 24, 49):
        op = so.decompose(sdq_synth.bf16_bits(W[128 * t:128 * t + 128]), ocfg())
        d, tol = y_close(Y32big[:M, 128 * t:128 * t + 128].cpu().numpy(), so.linear(oq, op))
        assert (d <= tol).all(), (t, d.max())


@pytest.mark.parametrize("M,N,K", [(16, 1024, 2048), (700, 6400, 512)])
def test_streams_and_graph_replay_give_the_eager_result(M, N, K):
    """the quantizer + GEMM chain on two streams at once (separate buffers) and captured in a CUDA graph replayed
    twice: bit-identical to the eager result on the default stream"""
    m = sdq()
    cfg = m.Config()
    W = sdq_synth.make_weight(N, K, 81).cuda()
    X = sdq_synth.make_act(M, K, 82).cuda()
    p = m.sdq_decompose(W, cfg)
    y_eager = m.sdq_linear(m.sdq_quantize_act(X, cfg), p)
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in range(2)]
    bufs = [torch.empty(m.act_size(M, K, cfg), dtype=torch.uint8, device="cuda") for _ in range(2)]
    outs = [torch.zeros((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    for _ in range(3):
        for st, b, o in zip(streams, bufs, outs):
            with torch.cuda.stream(st):
                m.sdq_linear(m.sdq_quantize_act(X, cfg, b), p, o)
    torch.cuda.synchronize()
    assert torch.equal(outs[0], y_eager) and torch.equal(outs[1], y_eager)
    g = torch.cuda.CUDAGraph()
    yg = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        m.sdq_linear(m.sdq_quantize_act(X, cfg, bufs[0]), p, yg)     # warm-up outside the capture
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    with torch.cuda.graph(g):
        m.sdq_linear(m.sdq_quantize_act(X, cfg, bufs[0]), p, yg)
    for _ in range(2):
        yg.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(yg, y_eager)
    assert m.device_status() == 0


@pytest.mark.parametrize("M,N,K,out_n", [(8, 128, 32768, 1), (20001, 256, 256, 1), (3, 128, 16640, 2)])
def test_extreme_shapes_long_rows_and_many_tokens(M, N, K, out_n):
    """the longest rows (128 inlier + 256 outlier stages per tile; a row length only the two-pass quantizer takes) and
    tens of thousands of tokens with a ragged last tile; tokens sampled for the oracle"""
    m = sdq()
    cfg = m.Config(out_n, m.GRAN_PAIR, 64, 0)
    W = sdq_synth.make_weight(N, K, 91 + M % 7)
    X = sdq_synth.make_act(M, K, 92 + M % 7)
    p = m.sdq_decompose(W.cuda(), cfg)
    xq = m.sdq_quantize_act(X.cuda(), cfg)
    y = m.sdq_linear(xq, p, f32=True)
    y16 = m.sdq_linear(xq, p)
    assert m.device_status() == 0
    assert torch.equal(y16, y.to(torch.bfloat16))
    toks = np.unique(np.concatenate([[0, M - 1], np.random.default_rng(M).integers(0, M, size=min(M, 24))]))
    op = so.decompose(sdq_synth.bf16_bits(W), ocfg(out_n))
    oq = so.quantize_act(sdq_synth.bf16_bits(X[toks]), ocfg(out_n))
    ae = m.act_export(xq)
    for name in ("xq4_code", "xq4_scale", "xq8_code", "xq8_sexp"):
        assert np.array_equal(ae[name][torch.from_numpy(toks).cuda()].cpu().numpy(), getattr(oq, name)), name
    d, tol = y_close(y[torch.from_numpy(toks).cuda()].cpu().numpy(), so.linear(oq, op))
    assert (d <= tol).all(), (d.max(), (d / tol).max())


@pytest.mark.parametrize("M,K", [(1, 256), (77, 512), (2048, 4096)])
def test_channel_norm_and_calibrated_decomposition(M, K):
    """sdq_channel_norm against the fp64 definition (fp64 accumulation on both sides: equal after rounding to fp32, one
    ulp allowed), then the whole calibrate -> decompose path: the packer fed with the GPU's norms must reproduce the
    oracle fed with the same norms bit for bit"""
    m = sdq()
    X = sdq_synth.make_act(M, K, 300 + M)
    c = m.channel_norm(X.cuda())
    ref = so.channel_norm(sdq_synth.bf16_bits(X))
    cg = c.cpu().numpy()
    assert np.all(np.abs(cg.astype(np.float64) - ref.astype(np.float64)) <= np.spacing(ref).astype(np.float64))
    if K <= 512:
        cfg = m.Config()
        W = sdq_synth.make_weight(256, K, 301)
        p = m.sdq_decompose(W.cuda(), cfg, col_weight=c)
        op = so.decompose(sdq_synth.bf16_bits(W), ocfg(), col_weight=cg)
        pe = {k: v.cpu().numpy() for k, v in m.packed_export(p).items()}
        for name in ("in_code", "in_meta", "in_scale", "out_code", "out_idx", "out_sexp"):
            assert np.array_equal(pe[name], getattr(op, name)), name


def test_packer_ties_zeros_and_negative_zero():
    m = sdq()
    rng = np.random.default_rng(1)
    vals = np.array([0.0, -0.0, 0.5, -0.5, 1.0, 1.0, -2.0, 2.0, 3.0, 1e-30, -1e-30, 448.0, 6.0, -6.0, 7.0, 0.75])
    W = torch.from_numpy(rng.choice(vals, size=(128, 512))).to(torch.bfloat16)
    W[5] = 0
    for out_n in (0, 1, 2):
        for rule in (0, 1):
            cfg = m.Config(out_n, m.GRAN_PAIR, 64, rule)
            pe = {k: v.cpu().numpy() for k, v in m.packed_export(m.sdq_decompose(W.cuda(), cfg)).items()}
            op = so.decompose(sdq_synth.bf16_bits(W), ocfg(out_n, rule))
            for name in ("in_code", "in_meta", "in_scale", "out_code", "out_idx", "out_sexp"):
                assert np.array_equal(pe[name], getattr(op, name)), (name, out_n, rule)


@pytest.mark.parametrize("gran,block", [(1, 32), (1, 64), (0, 32)])
@pytest.mark.parametrize("out_n", [0, 1, 2])
def test_literal_readings_element_wise_2of4_and_block32(gran, block, out_n):
    """element-wise 2:4 inliers and / or one scale per 32 K (the literal '2:4, block-32 MXFP4' wording): packer and
    activation quantizer are bit-exact against the oracle; these readings are decompose / quantize / export only"""
    m = sdq()
    for rule in (0, 1):
        cfg = m.Config(out_n, gran, block, rule)
        oc = so.Config(out_n, gran, block, rule)
        W = sdq_synth.make_weight(256, 1024, 40 + out_n)
        X = sdq_synth.make_act(37, 1024, 41 + out_n)
        pe = {k: v.cpu().numpy() for k, v in m.packed_export(m.sdq_decompose(W.cuda(), cfg)).items()}
        op = so.decompose(sdq_synth.bf16_bits(W), oc)
        for name in ("in_code", "in_meta", "in_scale", "out_code", "out_idx", "out_sexp"):
            assert np.array_equal(pe[name], getattr(op, name)), (name, rule)
        ae = {k: v.cpu().numpy() for k, v in m.act_export(m.sdq_quantize_act(X.cuda(), cfg)).items()}
        oq = so.quantize_act(sdq_synth.bf16_bits(X), oc)
        for name in ("xq4_code", "xq4_scale", "xq8_code", "xq8_sexp"):
            assert np.array_equal(ae[name], getattr(oq, name)), (name, rule)
    # ties, zeros and -0 under the element-wise pattern
    rng = np.random.default_rng(2)
    vals = np.array([0.0, -0.0, 0.5, -0.5, 1.0, 1.0, -2.0, 2.0, 3.0, 1e-30, 448.0, 6.0, 7.0, 0.75])
    Wt = torch.from_numpy(rng.choice(vals, size=(128, 512))).to(torch.bfloat16)
    cfg, oc = m.Config(out_n, gran, block, 0), so.Config(out_n, gran, block, 0)
    pe = {k: v.cpu().numpy() for k, v in m.packed_export(m.sdq_decompose(Wt.cuda(), cfg)).items()}
    op = so.decompose(sdq_synth.bf16_bits(Wt), oc)
    for name in ("in_code", "in_meta", "in_scale", "out_code", "out_idx", "out_sexp"):
        assert np.array_equal(pe[name], getattr(op, name)), name


def test_l2_copy_diagnostic_runs_and_reports_bytes():
    m = sdq()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    src = torch.zeros(sms * (128 << 10), dtype=torch.uint8, device="cuda")
    for issuers, iters in ((1, 50), (3, 50), (4, 3), (2, 1)):
        moved = m.diag_l2_copy(src, 16384, 4, iters, issuers)
        torch.cuda.synchronize()
        assert moved == sms * iters * 16384 and m.device_status() == 0
    for args, code in (((1000, 4, 10), 2), ((16384, 17, 10), 2), ((1 << 20, 4, 10), 2), ((16384, 4, 10, 5), 2)):
        with pytest.raises(m.SdqError) as e:
            m.diag_l2_copy(src, *args)
        assert e.value.code == code


def test_errors_are_status_codes():
    m = sdq()
    W = sdq_synth.make_weight(128, 256, 0).cuda()
    with pytest.raises(m.SdqError) as e:
        m.sdq_decompose(W[:, :128].contiguous())           # K not a multiple of 256
    assert e.value.code == 2
    p_elem = m.sdq_decompose(W, m.Config(1, m.GRAN_ELEM, 64, 0))            # decompose-only reading ...
    xq32 = m.sdq_quantize_act(sdq_synth.make_act(4, 256, 0).cuda(), m.Config(1, m.GRAN_ELEM, 64, 0))
    with pytest.raises(m.SdqError) as e:
        m.sdq_linear(xq32, p_elem)                                          # ... which the tensor core cannot run
    assert e.value.code == 4
    Wbad = W.clone()
    Wbad[3, 7] = float("inf")
    with pytest.raises(m.SdqError) as e:
        m.sdq_decompose(Wbad)
    assert e.value.code == 6
    p = m.sdq_decompose(W)
    xq = m.sdq_quantize_act(sdq_synth.make_act(4, 512, 0).cuda())
    with pytest.raises(m.SdqError) as e:
        m.sdq_linear(xq, p)                                  # K mismatch
    assert e.value.code == 2
