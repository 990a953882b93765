"""GPU parity of the grouped few-token call, the CTA-pair many-token kernel and the streamed outlier forms,
against the CPU oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

import sdq_synth
from oracle import sdq_oracle as so
from tests.test_gpu_parity import ocfg, run_case, sdq, y_close

pytestmark = pytest.mark.gpu


def _layers(shapes, Ms, cfg_args, seed, share_x=False):
    m = sdq()
    cfg = m.Config(*cfg_args)
    Ws = [sdq_synth.make_weight(N, K, seed + i) for i, (N, K) in enumerate(shapes)]
    Xs = [sdq_synth.make_act(M, K, seed + 50 + (0 if share_x else i)) for i, ((N, K), M) in enumerate(zip(shapes, Ms))]
    ps = [m.sdq_decompose(W.cuda(), cfg) for W in Ws]
    xqs = []
    for i, X in enumerate(Xs):
        xqs.append(xqs[0] if (share_x and i) else m.sdq_quantize_act(X.cuda(), cfg))
    return m, cfg, Ws, Xs, ps, xqs


def _check_against_oracle(m, Ws, Xs, ys32, ys16, cfg_args, rows=None):
    """every layer of the group against its own oracle result (all rows, or a sampled row range for wide layers)"""
    worst = 0.0
    oc = ocfg(cfg_args[0], cfg_args[3] if len(cfg_args) > 3 else 0, cfg_args[2] if len(cfg_args) > 2 else 64,
              cfg_args[1] if len(cfg_args) > 1 else so.GRAN_PAIR)
    for W, X, y32, y16 in zip(Ws, Xs, ys32, ys16):
        op = so.decompose(sdq_synth.bf16_bits(W), oc)
        oq = so.quantize_act(sdq_synth.bf16_bits(X), oc)
        n0, n1 = rows if rows else (0, W.shape[0])
        n1 = min(n1, W.shape[0])
        yref = so.linear(oq, op, n0, n1)
        d, tol = y_close(y32[:, n0:n1].cpu().numpy(), yref)
        assert (d <= tol).all(), (d.max(), (d / tol).max())
        assert torch.equal(y16, y32.to(torch.bfloat16))          # bf16 output = RNE of the fp32 accumulator
        worst = max(worst, float((d / tol).max()))
    return worst


@pytest.mark.parametrize("shapes,Ms,out_n,share_x", [
    ([(4096, 4096)] * 3, [1] * 3, 1, False),                 # q / k / v of one decoder layer, one token
    ([(4096, 4096)] * 3, [16] * 3, 1, True),                 # the same sharing one quantized X
    ([(11008, 4096)] * 2, [7] * 2, 1, True),                 # gate / up
    ([(4096, 4096), (11008, 4096), (4096, 11008)], [5, 5, 5], 1, False),   # different N and K in one call
    ([(2048, 1024)] * 10, [3] * 10, 1, False),               # many small layers, four 256-K units each: the shortest items of the fused kernel
    ([(4096, 2048)] * 4, [32] * 4, 1, False),                # 32 tokens: the wider token tile
    ([(4096, 2048)] * 4, [17, 20, 32, 1], 1, False),         # token counts differ inside the group
    ([(4096, 4096)] * 3, [16] * 3, 0, False),                # no outlier part
    ([(1152, 1280)] * 10, [2] * 10, 1, False),               # an odd number of units per item: items start on either ring parity
    ([(1152, 256)] * 10, [2] * 10, 1, False),                # K below the fused kernel's range: enqueued layer by layer
])
def test_group_call_matches_oracle(shapes, Ms, out_n, share_x):
    cfg_args = (out_n, so.GRAN_PAIR, 64, 0)
    m, cfg, Ws, Xs, ps, xqs = _layers(shapes, Ms, cfg_args, 4200, share_x)
    if share_x:
        Xs = [Xs[0]] * len(Xs)
    ys32 = m.sdq_linear_group(xqs, ps, f32=True)
    ys16 = m.sdq_linear_group(xqs, ps)
    assert m.device_status() == 0
    _check_against_oracle(m, Ws, Xs, ys32, ys16, cfg_args, rows=(0, 1024) if max(s[0] for s in shapes) > 4096 else None)
    # wide layers: also the last row tile
    if max(s[0] for s in shapes) > 4096:
        for W, X, y32 in zip(Ws, Xs, ys32):
            N = W.shape[0]
            oc = ocfg(out_n)
            yref = so.linear(so.quantize_act(sdq_synth.bf16_bits(X), oc), so.decompose(sdq_synth.bf16_bits(W), oc), N - 128, N)
            d, tol = y_close(y32[:, N - 128:].cpu().numpy(), yref)
            assert (d <= tol).all()


def test_group_call_runs_twice_in_a_row_and_inside_a_graph():
    cfg_args = (1, so.GRAN_PAIR, 64, 0)
    m, cfg, Ws, Xs, ps, xqs = _layers([(4096, 1024)] * 4, [9] * 4, cfg_args, 4300)
    outs = [torch.empty((9, 4096), dtype=torch.bfloat16, device="cuda") for _ in ps]
    ref = [o.clone() for o in m.sdq_linear_group(xqs, ps)]
    m.sdq_linear_group(xqs, ps, outs)
    m.sdq_linear_group(xqs, ps, outs)
    assert all(torch.equal(a, b) for a, b in zip(outs, ref))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        m.sdq_linear_group(xqs, ps, outs)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    for o in outs:
        o.zero_()
    with torch.cuda.graph(g):
        m.sdq_linear_group(xqs, ps, outs)
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    assert m.device_status() == 0
    assert all(torch.equal(a, b) for a, b in zip(outs, ref))


@pytest.mark.parametrize("shapes,Ms,cfg_args", [
    ([(4096, 1024)] * 3, [40] * 3, (1, so.GRAN_PAIR, 64, 0)),     # more than 32 tokens
    ([(4096, 1024)] * 3, [8] * 3, (1, so.GRAN_PAIR, 32, 0)),      # one scale per 32 K
    ([(4096, 1024)] * 3, [8] * 3, (2, so.GRAN_PAIR, 64, 0)),      # two outliers per S-Vector
    ([(256, 1024)] * 2, [8] * 2, (1, so.GRAN_PAIR, 64, 0)),       # too few row tiles for the persistent kernel
    ([(4096, 512)] * 3, [8] * 3, (1, so.GRAN_PAIR, 64, 0)),       # items shorter than half the ring
    ([(4096, 1024)] * 3, [8] * 3, (1, so.GRAN_DENSE, 32, 0)),     # dense inliers
])
def test_group_call_outside_the_fused_kernels_range_equals_single_calls(shapes, Ms, cfg_args):
    m, cfg, Ws, Xs, ps, xqs = _layers(shapes, Ms, cfg_args, 4400)
    ys = m.sdq_linear_group(xqs, ps)
    ys32 = m.sdq_linear_group(xqs, ps, f32=True)
    assert m.device_status() == 0
    for x, p, y, y32 in zip(xqs, ps, ys, ys32):
        assert torch.equal(y, m.sdq_linear(x, p))
        assert torch.equal(y32, m.sdq_linear(x, p, f32=True))


def test_group_call_errors_are_status_codes():
    m = sdq()
    cfg = m.Config()
    p = m.sdq_decompose(sdq_synth.make_weight(256, 512, 1).cuda(), cfg)
    x = m.sdq_quantize_act(sdq_synth.make_act(4, 512, 1).cuda(), cfg)
    x_other_k = m.sdq_quantize_act(sdq_synth.make_act(4, 256, 1).cuda(), cfg)
    with pytest.raises(m.SdqError) as e:
        m.sdq_linear_group([x, x_other_k], [p, p])
    assert e.value.code == 2                                     # SDQ_ERR_SHAPE: K of the second layer does not match
    import ctypes
    L = m.lib()
    assert L.sdq_linear_group(0, None, None, None, None, None) == 1     # SDQ_ERR_INVALID_ARG


# ---------------------------------------------------------------------------------------------- many tokens, CTA pairs
@pytest.mark.parametrize("M,N,K,out_n,block,gran,rule,rows", [
    (300, 512, 4096, 1, 64, so.GRAN_PAIR, 0, None),          # ragged second token tile: the odd CTA of a pair has no tokens
    (257, 256, 2816, 1, 64, so.GRAN_PAIR, 0, None),          # 33 stages per tile: the slot pairs straddle tiles
    (511, 768, 2048, 2, 64, so.GRAN_PAIR, 1, None),          # two outliers per S-Vector, ceil rule
    (640, 256, 8192, 0, 64, so.GRAN_PAIR, 0, None),          # no outlier part, 32 inlier stages
    (260, 512, 4096, 1, 32, so.GRAN_PAIR, 0, None),          # one scale per 32 K
    (260, 512, 4096, 1, 32, so.GRAN_PAIR, 2, None),          # E4M3 scale codes, two-level scaling
    (260, 512, 4096, 1, 32, so.GRAN_DENSE, 0, None),         # dense inliers
    (700, 20480, 3072, 1, 64, so.GRAN_PAIR, 0, (20224, 20480)),   # 240 pair tiles on 74 pairs: several rounds, last rows
    (2048, 11008, 4096, 1, 64, so.GRAN_PAIR, 0, (5376, 5504)),    # the benchmark's gate shape, one row tile sampled
])
def test_cta_pair_many_token_kernel(M, N, K, out_n, block, gran, rule, rows):
    run_case(M, N, K, 4500 + M, out_n=out_n, rule=rule, block=block, gran=gran, check_rows=rows)


# ---------------------------------------------------------------------------------------------- the streamed outlier forms
def _a_off(row, byte):
    j, b = byte >> 5, byte & 31
    return j * 4096 + (row >> 3) * 256 + (b >> 4) * 128 + (row & 7) * 16 + (b & 15)


@pytest.mark.parametrize("out_n", [1, 2])
def test_both_streamed_outlier_forms_decode_to_the_oracles_outliers(out_n):
    """The many-token kernels stream the 2:4 FP8 container (WO), the grouped few-token kernel the compact records (WC).
    Both are decoded here on the host, byte by byte from the packed buffer, and compared with the oracle's outlier
    codes and positions: the bytes the tensor core consumes are on the bit-exact surface, not only the exporter's view."""
    m = sdq()
    N, K = 256, 1024
    cfg = m.Config(out_n, m.GRAN_PAIR, 64, 0)
    W = sdq_synth.make_weight(N, K, 4600 + out_n)
    W[5, 8:16] = 0.0                                   # an all-zero S-Vector: its outlier has code 0 at position 0
    p = m.sdq_decompose(W.cuda(), cfg)
    blob = p.buf.cpu().numpy()
    op = so.decompose(sdq_synth.bf16_bits(W), ocfg(out_n))
    wo, wc = int(p.desc.off[1]), int(p.desc.off[3])
    T1 = K // 128
    wcb = 3072 * out_n
    for n in range(N):
        rt, r = n // 128, n % 128
        for g in range(K // 8):
            k1, gi = g // 16, g % 16
            want = {int(op.out_idx[n, g, t]): int(op.out_code[n, g, t]) for t in range(out_n)}
            # compact record: code bytes, then position nibbles
            rec = wc + (rt * T1 + k1) * wcb
            got = {}
            for t in range(out_n):
                e = gi * out_n + t
                code = int(blob[rec + r * 16 * out_n + e])
                pos = (int(blob[rec + 2048 * out_n + r * 8 * out_n + e // 2]) >> (4 * (e & 1))) & 15
                got[pos] = code
            assert got == want, (n, g, got, want)
            # 2:4 container: four stored bytes (two per group of 4) and one metadata byte (two index nibbles)
            rec = wo + (rt * T1 + k1) * 10240
            stored = [int(blob[rec + _a_off(r, gi * 4 + b)]) for b in range(4)]
            meta = int(blob[rec + 8192 + r * 16 + gi])
            dec = {}
            for h in range(2):
                nib = (meta >> (4 * h)) & 15
                i0, i1 = nib & 3, nib >> 2
                assert i0 < i1
                dec[4 * h + i0] = stored[2 * h]
                dec[4 * h + i1] = stored[2 * h + 1]
            nz = {k: v for k, v in dec.items() if v != 0}
            assert nz == {k: v for k, v in want.items() if v != 0}, (n, g, dec, want)


def test_rows_and_tokens_of_subnormal_magnitude():
    """bf16 subnormals drive the scale exponents into their clamps (E8M0 code 0, outlier exponent -127): packer,
    quantizer and product must still agree with the oracle."""
    m = sdq()
    N, K, M = 256, 512, 9
    cfg = m.Config(1, m.GRAN_PAIR, 64, 0)
    g = torch.Generator().manual_seed(4700)
    Wb = torch.randint(0, 0x80, (N, K), generator=g, dtype=torch.int32)          # subnormal magnitudes 0 .. 0x7F
    Wb = (Wb | (torch.randint(0, 2, (N, K), generator=g, dtype=torch.int32) << 15)).to(torch.int16)
    W = Wb.view(torch.bfloat16).clone()
    W[128:] = sdq_synth.make_weight(128, K, 4701)                                 # normal rows beside them
    Xb = torch.randint(0, 0x80, (M, K), generator=g, dtype=torch.int32).to(torch.int16)
    X = Xb.view(torch.bfloat16).clone()
    X[4:] = sdq_synth.make_act(M - 4, K, 4702)
    p = m.sdq_decompose(W.cuda(), cfg)
    xq = m.sdq_quantize_act(X.cuda(), cfg)
    op = so.decompose(sdq_synth.bf16_bits(W), ocfg(1))
    oq = so.quantize_act(sdq_synth.bf16_bits(X), ocfg(1))
    pe = {k: v.cpu().numpy() for k, v in m.packed_export(p).items()}
    ae = {k: v.cpu().numpy() for k, v in m.act_export(xq).items()}
    for name in ("in_code", "in_meta", "in_scale", "out_code", "out_idx", "out_sexp"):
        assert np.array_equal(pe[name], getattr(op, name)), name
    for name in ("xq4_code", "xq4_scale", "xq8_code", "xq8_sexp"):
        assert np.array_equal(ae[name], getattr(oq, name)), name
    assert int(op.out_sexp[:128].min()) == -127 and int(op.in_scale[:128].max()) <= 3      # the clamps are reached
    y = m.sdq_linear(xq, p, f32=True).cpu().numpy()
    assert m.device_status() == 0
    d, tol = y_close(y, so.linear(oq, op))
    assert (d <= tol).all()


# ---------------------------------------------------------------------------------------------- saved and restored buffers
@pytest.mark.parametrize("cfg_args,M", [((1, so.GRAN_PAIR, 64, 0), 5), ((2, so.GRAN_PAIR, 32, 1), 200), ((1, so.GRAN_DENSE, 32, 0), 33),
                                        ((1, so.GRAN_PAIR, 32, 2), 16), ((1, so.GRAN_ELEM, 64, 0), 0)])
def test_packed_buffer_survives_a_plain_copy_and_attach(cfg_args, M):
    """device -> host bytes -> another device buffer -> sdq_packed_attach: the descriptor is rebuilt from the buffer's own
    header and sdq_linear gives the original result bit for bit."""
    m = sdq()
    cfg = m.Config(*cfg_args)
    N, K = 256, 1024
    p = m.sdq_decompose(sdq_synth.make_weight(N, K, 4800).cuda(), cfg)
    saved = p.buf.cpu().numpy().tobytes()                      # what a file would hold
    pad = torch.zeros(len(saved) + 4096, dtype=torch.uint8, device="cuda")
    restored = pad[:len(saved)]
    restored.copy_(torch.frombuffer(bytearray(saved), dtype=torch.uint8))
    q = m.packed_attach(restored)
    assert (q.N, q.K) == (N, K)
    assert [q.cfg.out_n, q.cfg.in_gran, q.cfg.in_block, q.cfg.scale_rule, q.cfg.out_order] == \
           [cfg.out_n, cfg.in_gran, cfg.in_block, cfg.scale_rule, cfg.out_order]
    assert list(q.desc.off) == list(p.desc.off) and q.desc.bytes == p.desc.bytes
    a, b = m.packed_export(p), m.packed_export(q)
    assert all(torch.equal(a[k], b[k]) for k in a)
    if M:
        xq = m.sdq_quantize_act(sdq_synth.make_act(M, K, 4801).cuda(), cfg)
        assert torch.equal(m.sdq_linear(xq, q), m.sdq_linear(xq, p))
    assert m.device_status() == 0


def test_attach_refuses_what_is_not_a_packed_buffer():
    m = sdq()
    cfg = m.Config()
    p = m.sdq_decompose(sdq_synth.make_weight(128, 256, 4810).cuda(), cfg)
    junk = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(m.SdqError) as e:
        m.packed_attach(junk)
    assert e.value.code == 4                                   # no magic: SDQ_ERR_UNSUPPORTED
    cut = p.buf[:p.buf.numel() // 2].clone()
    with pytest.raises(m.SdqError) as e:
        m.packed_attach(cut)
    assert e.value.code == 5                                   # shorter than its header says
    bad = p.buf.clone()
    bad[16] = 7                                                # out_n = 7 in the header's configuration (byte 16)
    with pytest.raises(m.SdqError) as e:
        m.packed_attach(bad)
    assert e.value.code == 2


def test_a_bounded_wait_that_runs_out_sets_the_sticky_status_and_the_context_stays_usable():
    """Failure detection without a fault: a kernel waits, for 64 polls, on a barrier nothing completes; it returns, the
    sticky status word reports the timeout once, and the next call runs normally."""
    m = sdq()
    assert m.device_status() == 0
    m.diag_wait_timeout(64)
    assert m.device_status() == 8                              # SDQ_ERR_TIMEOUT
    assert m.device_status() == 0                              # reading cleared it
    cfg = m.Config()
    p = m.sdq_decompose(sdq_synth.make_weight(128, 256, 4820).cuda(), cfg)
    xq = m.sdq_quantize_act(sdq_synth.make_act(3, 256, 4821).cuda(), cfg)
    y = m.sdq_linear(xq, p, f32=True).cpu().numpy()
    assert m.device_status() == 0
    oc = ocfg(1)
    d, tol = y_close(y, so.linear(so.quantize_act(sdq_synth.bf16_bits(sdq_synth.make_act(3, 256, 4821)), oc),
                                  so.decompose(sdq_synth.bf16_bits(sdq_synth.make_weight(128, 256, 4820)), oc)))
    assert (d <= tol).all()


# ---------------------------------------------------------------------------------------------------------------------
# int8 outlier operands (Section 5.1: W_o and A_o in int8; the evaluation's "1:8int8" configurations)

I8_ARGS = (1, so.GRAN_PAIR, 64, 0, 0, so.OUT_INT8)


def _i8_cfgs():
    m = sdq()
    return m, m.Config(*I8_ARGS), so.Config(*I8_ARGS)


@pytest.mark.parametrize("N,K,M", [(256, 512, 9), (1152, 1280, 130), (128, 16640, 3)])
def test_int8_outlier_codes_and_scales_match_the_oracle_bit_for_bit(N, K, M):
    """packer and activation quantizer: int8 codes, positions and the bit patterns of the fp32 scales (short and long rows:
    the one-launch and the two-launch quantizer)"""
    m, cfg, oc = _i8_cfgs()
    W, X = sdq_synth.make_weight(N, K, 77), sdq_synth.make_act(M, K, 78)
    p, xq = m.sdq_decompose(W.cuda(), cfg), m.sdq_quantize_act(X.cuda(), cfg)
    assert m.device_status() == 0
    op, oq = so.decompose(sdq_synth.bf16_bits(W), oc), so.quantize_act(sdq_synth.bf16_bits(X), oc)
    pe = {k: v.cpu().numpy() for k, v in m.packed_export(p).items()}
    ae = {k: v.cpu().numpy() for k, v in m.act_export(xq).items()}
    for name in ("in_code", "in_meta", "in_scale", "out_code", "out_idx", "out_sexp"):
        assert np.array_equal(pe[name], getattr(op, name)), name
    for name in ("xq4_code", "xq4_scale", "xq8_code", "xq8_sexp"):
        assert np.array_equal(ae[name], getattr(oq, name)), name
    # an all-zero row and an all-zero token: scale 1, codes 0
    W2 = W.clone(); W2[5] = 0
    X2 = X.clone(); X2[0] = 0
    p2, x2 = m.sdq_decompose(W2.cuda(), cfg), m.sdq_quantize_act(X2.cuda(), cfg)
    assert m.packed_export(p2)["out_sexp"].cpu().numpy().view(np.float32)[5] == 1.0
    assert m.act_export(x2)["xq8_sexp"].cpu().numpy().view(np.float32)[0] == 1.0
    assert not m.act_export(x2)["xq8_code"].cpu().numpy()[0].any()


@pytest.mark.parametrize("shapes,Ms", [
    ([(4096, 4096)] * 3, [1, 16, 5]),                      # q / k / v
    ([(4096, 1024), (11008, 4096), (4096, 11008)], [7, 7, 7]),   # different widths and depths: up to 1376 outliers per row
    ([(4096, 2048)] * 4, [32, 17, 20, 2]),                 # the wider token tile
])
def test_int8_outlier_group_call_matches_oracle(shapes, Ms):
    m, cfg, oc = _i8_cfgs()
    Ws = [sdq_synth.make_weight(N, K, 4700 + i) for i, (N, K) in enumerate(shapes)]
    Xs = [sdq_synth.make_act(M, K, 4750 + i) for i, ((N, K), M) in enumerate(zip(shapes, Ms))]
    ps = [m.sdq_decompose(W.cuda(), cfg) for W in Ws]
    xqs = [m.sdq_quantize_act(X.cuda(), cfg) for X in Xs]
    ys32 = m.sdq_linear_group(xqs, ps, f32=True)
    ys16 = m.sdq_linear_group(xqs, ps)
    assert m.device_status() == 0
    for W, X, y32, y16 in zip(Ws, Xs, ys32, ys16):
        op, oq = so.decompose(sdq_synth.bf16_bits(W), oc), so.quantize_act(sdq_synth.bf16_bits(X), oc)
        N = W.shape[0]
        for n0, n1 in ((0, 512), (N - 128, N)):
            yref = so.linear(oq, op, n0, n1)
            d, tol = y_close(y32[:, n0:n1].cpu().numpy(), yref)
            assert (d <= tol).all(), (d.max(), (d / tol).max())
        assert torch.equal(y16, y32.to(torch.bfloat16))
    # the outlier part alone: weights whose only non-zeros are outliers give O = O_o = s_x s_w (integer sum), which the
    # kernel forms exactly in int32 and scales once
    N, K, M = 4096, 1024, 4
    g = torch.Generator().manual_seed(9)
    W = torch.zeros((N, K))
    pos = torch.randint(0, 8, (N, K // 8), generator=g)
    vals = torch.randn((N, K // 8), generator=g) * 0.05 + 0.001
    W.view(N, K // 8, 8).scatter_(2, pos.unsqueeze(-1), vals.unsqueeze(-1))
    W = W.to(torch.bfloat16)
    X = sdq_synth.make_act(M, K, 10)
    ps, xq = [m.sdq_decompose(W.cuda(), cfg)] * 3, m.sdq_quantize_act(X.cuda(), cfg)
    y = m.sdq_linear_group([xq] * 3, ps, f32=True)[2].cpu().numpy()
    op, oq = so.decompose(sdq_synth.bf16_bits(W), oc), so.quantize_act(sdq_synth.bf16_bits(X), oc)
    qw = np.zeros((N, K), dtype=np.int64)
    np.put_along_axis(qw.reshape(N, K // 8, 8), op.out_idx.astype(np.int64), op.out_code.view(np.int8).astype(np.int64), axis=2)
    isum = oq.xq8_code.view(np.int8).astype(np.int64) @ qw.T
    sx, sw = oq.xq8_sexp.view(np.float32), op.out_sexp.view(np.float32)
    want = isum.astype(np.float32) * (sw[None, :] * sx[:, None])          # the kernel's own two fp32 roundings
    assert np.array_equal(y, want)


def test_int8_outliers_outside_the_grouped_kernel_are_refused():
    m, cfg, oc = _i8_cfgs()
    p = m.sdq_decompose(sdq_synth.make_weight(256, 1024, 1).cuda(), cfg)
    x = m.sdq_quantize_act(sdq_synth.make_act(4, 1024, 1).cuda(), cfg)
    with pytest.raises(RuntimeError):
        m.sdq_linear(x, p)                                   # a single call
    with pytest.raises(RuntimeError):
        m.sdq_linear_group([x, x], [p, p])                   # too few row tiles for the fused kernel
    x_e4m3 = m.sdq_quantize_act(sdq_synth.make_act(4, 1024, 1).cuda(), m.Config(1, so.GRAN_PAIR, 64, 0))
    big = m.sdq_decompose(sdq_synth.make_weight(4096, 1024, 2).cuda(), cfg)
    with pytest.raises(RuntimeError):
        m.sdq_linear_group([x_e4m3] * 3, [big] * 3)          # the activations' 8-bit format differs from the weights'
    with pytest.raises(RuntimeError):
        m.sdq_decompose(sdq_synth.make_weight(256, 1024, 1).cuda(), m.Config(1, so.GRAN_PAIR, 32, 0, 0, so.OUT_INT8))   # block 32
    # the blob header carries the format
    q = m.packed_attach(big.buf.clone())
    assert q.cfg.out_fmt == so.OUT_INT8


# ---------------------------------------------------------------------------------------------------------------------
# the activation quantizer fused into the grouped kernel (Section 5, Stage 3 in the linear layers' load path)

@pytest.mark.parametrize("shapes,M,cfg_args", [
    ([(4096, 4096)] * 3, 1, (1, so.GRAN_PAIR, 64, 0)),                       # q / k / v, one token
    ([(4096, 4096)] * 3, 16, (1, so.GRAN_PAIR, 64, 0)),
    ([(11008, 4096)] * 2, 7, (1, so.GRAN_PAIR, 64, 1)),                      # gate / up, the ceil scale rule
    ([(4096, 1024), (2048, 1024), (4096, 1024)], 5, (0, so.GRAN_PAIR, 64, 0)),   # no outlier part, the shortest K
    ([(4096, 2048)] * 4, 13, I8_ARGS),                                       # int8 outlier operands
])
def test_fused_quantizer_group_call_equals_quantize_then_group(shapes, M, cfg_args):
    m = sdq()
    cfg = m.Config(*cfg_args)
    K = shapes[0][1]
    Ws = [sdq_synth.make_weight(N, K, 5100 + i) for i, (N, _) in enumerate(shapes)]
    X = sdq_synth.make_act(M, K, 5150)
    X[0, 5] = float("inf")                                                   # saturates like the stand-alone quantizer
    if M > 2:
        X[2] = 0                                                             # an all-zero token
    ps = [m.sdq_decompose(W.cuda(), cfg) for W in Ws]
    Xd = X.cuda()
    xq = m.sdq_quantize_act(Xd, cfg)
    ref32 = m.sdq_linear_group([xq] * len(ps), ps, f32=True)
    ref16 = m.sdq_linear_group([xq] * len(ps), ps)
    y32 = m.sdq_linear_group_x(Xd, ps, f32=True)
    y16 = m.sdq_linear_group_x(Xd, ps)
    assert m.device_status() == 0
    for a, b, c, d in zip(y32, ref32, y16, ref16):
        assert torch.equal(a, b) and torch.equal(c, d)                       # the same codes, scales and summation order
    # and against the oracle directly (first layer, sampled rows)
    oc = so.Config(*cfg_args)
    op, oq = so.decompose(sdq_synth.bf16_bits(Ws[0]), oc), so.quantize_act(sdq_synth.bf16_bits(X), oc)
    yref = so.linear(oq, op, 0, 256)
    dd, tol = y_close(y32[0][:, :256].cpu().numpy(), yref)
    assert (dd <= tol).all()
    # a strided X (a slice of a wider buffer)
    wide = torch.zeros((M, K + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, :K] = Xd
    y_s = m.sdq_linear_group_x(wide[:, :K], ps)
    assert all(torch.equal(a, b) for a, b in zip(y_s, ref16))


def test_fused_quantizer_group_call_outside_its_range_is_refused():
    m = sdq()
    cfg = m.Config(1, so.GRAN_PAIR, 64, 0)
    ps = [m.sdq_decompose(sdq_synth.make_weight(4096, 1024, 1).cuda(), cfg)] * 3
    with pytest.raises(RuntimeError):
        m.sdq_linear_group_x(sdq_synth.make_act(17, 1024, 1).cuda(), ps)                 # more than 16 tokens
    p_long = [m.sdq_decompose(sdq_synth.make_weight(4096, 11008, 1).cuda(), cfg)] * 3
    with pytest.raises(RuntimeError):
        m.sdq_linear_group_x(sdq_synth.make_act(4, 11008, 1).cuda(), p_long)             # X does not fit beside the ring
    with pytest.raises(RuntimeError):
        m.sdq_linear_group_x(sdq_synth.make_act(4, 1024, 1).cuda(), ps[:1])              # too few row tiles
    with pytest.raises(RuntimeError):
        m.sdq_linear_group_x(sdq_synth.make_act(4, 2048, 1).cuda(), ps)                  # K of X and of the weights differ
    assert m.device_status() == 0


# ---------------------------------------------------------------------------------------------------------------------
# the packed buffer without its 2:4 outlier containers

@pytest.mark.parametrize("cfg_args", [(1, so.GRAN_PAIR, 64, 0), I8_ARGS])
def test_compact_buffer_serves_the_grouped_calls_and_nothing_else(cfg_args):
    m = sdq()
    cfg = m.Config(*cfg_args)
    N, K, M = 4096, 2048, 6
    Ws = [sdq_synth.make_weight(N, K, 6100 + i) for i in range(3)]
    X = sdq_synth.make_act(M, K, 6150).cuda()
    full = [m.sdq_decompose(W.cuda(), cfg) for W in Ws]
    comp = [m.packed_compact(p) for p in full]
    # 2.625 + 1.5 bits per weight, scales, padding: under 4.3; the full buffer carries the 5-bit containers on top
    assert comp[0].buf.numel() * 8 / (N * K) < 4.3 and full[0].buf.numel() * 8 / (N * K) > 9.0
    assert comp[0].desc.off[1] == 0 and comp[0].desc.off[3] > 0
    xq = m.sdq_quantize_act(X, cfg)
    ref = m.sdq_linear_group([xq] * 3, full, f32=True)
    got = m.sdq_linear_group([xq] * 3, comp, f32=True)
    gotx = m.sdq_linear_group_x(X, comp, f32=True)
    assert m.device_status() == 0
    for a, b, c in zip(ref, got, gotx):
        assert torch.equal(a, b) and torch.equal(a, c)
    # the canonical export reads the compact records: identical
    ea, eb = m.packed_export(full[0]), m.packed_export(comp[0])
    for k in ea:
        assert torch.equal(ea[k], eb[k]), k
    # save -> reload: the header says which form the buffer holds
    re = m.packed_attach(comp[1].buf.clone())
    assert re.desc.off[1] == 0 and torch.equal(m.sdq_linear_group([xq] * 3, [comp[0], re, comp[2]], f32=True)[1], ref[1])
    # calls that need the containers refuse it: the single-layer call, the layer-by-layer path of a group too small to fuse,
    # and compacting twice
    with pytest.raises(RuntimeError):
        m.sdq_linear(xq, comp[0])
    small = m.packed_compact(m.sdq_decompose(sdq_synth.make_weight(256, K, 1).cuda(), cfg))
    with pytest.raises(RuntimeError):
        m.sdq_linear_group([xq], [small])
    with pytest.raises(RuntimeError):
        m.packed_compact(comp[0])
    assert m.device_status() == 0
