"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration bench.py times.

The oracle cannot run these sizes end to end in seconds, so it is applied to a seeded sample that it can compute
exactly: whole 128-row weight tiles (first, middle, last) and a spread of token rows.  Weight rows, token rows and
outputs are independent of one another in the method, so the sampled rows of the packed arrays / activation codes must
match bit for bit and the sampled outputs must meet the Y criterion.
"""
import numpy as np
import pytest
import torch

import sdq_synth
from oracle import sdq_oracle as so

pytestmark = pytest.mark.gpu


def sdq():
    import paper_2406_13868_b200 as m
    return m


def check_sampled(M, N, K, seed, out_n=1, n_tok=12, use_ws=False, block=64, gran=so.GRAN_PAIR, rule=0):
    m = sdq()
    cfg = m.Config(out_n, gran, block, rule)
    ocfg = so.Config(out_n, gran, block, rule)
    W = sdq_synth.make_weight(N, K, seed, device="cuda")
    X = sdq_synth.make_act(M, K, seed + 1, device="cuda")
    p = m.sdq_decompose(W, cfg)
    xq = m.sdq_quantize_act(X, cfg)
    ws = m.make_workspace(M, N, K, cfg, "cuda") if use_ws else None
    y = m.sdq_linear(xq, p, f32=True, workspace=ws)
    y16 = m.sdq_linear(xq, p, workspace=ws)
    assert m.device_status() == 0
    assert torch.equal(y16, y.to(torch.bfloat16))

    RT = N // 128
    tiles = sorted({0, RT // 2, RT - 1})
    rows = np.concatenate([np.arange(128 * t, 128 * t + 128) for t in tiles])
    rng = np.random.default_rng(seed)
    toks = np.unique(np.concatenate([[0, M - 1], rng.integers(0, M, size=min(n_tok, M))]))
    rows_t, toks_t = torch.from_numpy(rows).cuda(), torch.from_numpy(toks).cuda()

    op = so.decompose(sdq_synth.bf16_bits(W[rows_t]), ocfg)
    pe = m.packed_export(p)
    for name in ("in_code", "in_meta", "in_scale", "out_code", "out_idx", "out_sexp", "in_texp"):
        assert np.array_equal(pe[name][rows_t].cpu().numpy(), getattr(op, name)), name
    oq = so.quantize_act(sdq_synth.bf16_bits(X[toks_t]), ocfg)
    ae = m.act_export(xq)
    for name in ("xq4_code", "xq4_scale", "xq8_code", "xq8_sexp"):
        assert np.array_equal(ae[name][toks_t].cpu().numpy(), getattr(oq, name)), name
    del pe, ae
    yref = so.linear(oq, op)
    yg = y[toks_t][:, rows_t].cpu().numpy().astype(np.float64)
    d = np.abs(yg - yref)
    tol = 1e-3 * (np.abs(yref) + 1e-2)
    assert (d <= tol).all(), (float(d.max()), float((d / tol).max()))
    return float((d / tol).max())


@pytest.mark.parametrize("M", [1, 16])
@pytest.mark.parametrize("use_ws", [False, True])
def test_llama7b_attention_projection_decode(M, use_ws):
    """config 2: X M x 4096, W 4096 x 4096"""
    check_sampled(M, 4096, 4096, 2000 + M, use_ws=use_ws)


@pytest.mark.parametrize("N,K", [(11008, 4096), (4096, 11008)])
def test_llama7b_mlp_prefill(N, K):
    """config 3: X 2048 x K; gate/up 4096 -> 11008 and down 11008 -> 4096"""
    check_sampled(2048, N, K, 3000 + N)


@pytest.mark.parametrize("M,N,K", [(16, 4096, 4096), (2048, 11008, 4096), (2048, 4096, 11008)])
def test_scale_block_32_at_full_size(M, N, K):
    """configs 2 and 3 with one scale per 32 K (the literal block-32 MXFP4 wording)"""
    check_sampled(M, N, K, 3500 + M, block=32)


@pytest.mark.parametrize("M,N,K,n", [(16, 4096, 4096, 7), (2048, 11008, 4096, 7), (2048, 4096, 11008, 8), (4096, 16384, 4096, 7)])
def test_n_of_8_patterns_at_full_size(M, N, K, n):
    """configs 2, 3 and 4 with the evaluation's patterns 7:8 = 1:8 + 6:8 and 8:8 = 1:8 + 7:8 (inliers stored dense)"""
    check_sampled(M, N, K, 3700 + M + n, block=32, gran=so.gran_keep(n))


@pytest.mark.parametrize("M,N,K", [(16, 4096, 4096), (2048, 11008, 4096), (2048, 4096, 11008)])
def test_two_level_e4m3_scales_at_full_size(M, N, K):
    """configs 2 and 3 with E4M3 Q-Vector scales and power-of-two row / token factors"""
    check_sampled(M, N, K, 3900 + M, block=32, rule=2)


@pytest.mark.parametrize("out_n", [1, 2, 0])
def test_opt67b_ffn_prefill_outlier_sweep(out_n):
    """config 4: X 4096 x 4096, fc1 4096 -> 16384; outlier pattern 1:8, 2:8, none"""
    check_sampled(4096, 16384, 4096, 4000 + out_n, out_n=out_n)


def test_opt67b_fc2_long_k():
    """config 4: fc2 16384 -> 4096 (the longest K: 64 inlier + 128 outlier stages per tile)"""
    check_sampled(4096, 4096, 16384, 4100)


@pytest.mark.parametrize("M", [1, 16, 128, 1024, 8192])
def test_llama7b_layer_shapes_token_sweep(M):
    """config 5: the three weight shapes of a LLaMA-7B decoder layer at every token count of the sweep"""
    for i, (N, K) in enumerate([(4096, 4096), (11008, 4096), (4096, 11008)]):
        check_sampled(M, N, K, 5000 + 10 * M + i, n_tok=8)


@pytest.mark.parametrize("M", [1, 16])
@pytest.mark.parametrize("out_fmt", [so.OUT_E4M3, so.OUT_INT8])
def test_llama7b_decode_32_layers_in_one_grouped_call_as_in_the_bench(M, out_fmt):
    """config 2 in the launch configuration bench.py times for decode: 32 distinct 4096 x 4096 layers, compact packed form,
    ONE grouped call; three layers (first, middle, last) are checked on sampled 128-row tiles, every token.  Also with the
    activation quantizer inside the kernel (bit-identical) and with int8 outlier operands."""
    m = sdq()
    cfg = m.Config(1, so.GRAN_PAIR, 64, 0, 0, out_fmt)
    ocfg = so.Config(1, so.GRAN_PAIR, 64, 0, 0, out_fmt)
    N = K = 4096
    layers = 32
    Ws, ps = {}, []
    for i in range(layers):
        W = sdq_synth.make_weight(N, K, 2000 + i, device="cuda")
        ps.append(m.packed_compact(m.sdq_decompose(W, cfg)))
        if i in (0, 15, 31):
            Ws[i] = W
        del W
    X = sdq_synth.make_act(M, K, 2100 + M, device="cuda")
    xq = m.sdq_quantize_act(X, cfg)
    ys = m.sdq_linear_group([xq] * layers, ps, f32=True)
    ys16 = m.sdq_linear_group([xq] * layers, ps)
    yx = m.sdq_linear_group_x(X, ps, f32=True)
    assert m.device_status() == 0
    oq = so.quantize_act(sdq_synth.bf16_bits(X), ocfg)
    rows = np.concatenate([np.arange(128 * t, 128 * t + 128) for t in (0, 16, 31)])
    rows_t = torch.from_numpy(rows).cuda()
    for i, W in Ws.items():
        op = so.decompose(sdq_synth.bf16_bits(W[rows_t]), ocfg)
        yref = so.linear(oq, op)
        d = np.abs(ys[i][:, rows_t].cpu().numpy().astype(np.float64) - yref)
        tol = 1e-3 * (np.abs(yref) + 1e-2)
        assert (d <= tol).all(), (i, float(d.max()), float((d / tol).max()))
    for a, b, c in zip(ys, ys16, yx):
        assert torch.equal(b, a.to(torch.bfloat16)) and torch.equal(a, c)
