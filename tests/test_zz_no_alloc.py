"""The allocation-free entry point `sdq_linear_noalloc`, checked against `sdq_linear_ws`.

Some users of the library cannot obtain device memory at call time: a plug-in inside an inference server whose
memory was handed out at start-up, or a caller on a latency path that must never reach cudaMalloc.  For them the
library carries a fixed scratch array of its own.  This file is collected last on purpose: if it fails, a run that
stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

import sdq_synth

pytestmark = pytest.mark.gpu


def sdq():
    import paper_2406_13868_b200 as m
    return m


@pytest.mark.parametrize("M,N,K", [(16, 256, 4096), (1, 1024, 2048)])
def test_noalloc_matches_workspace_variant_twice_in_a_row(M, N, K):
    m = sdq()
    cfg = m.Config()
    W = sdq_synth.make_weight(N, K, 900 + M).cuda()
    X = sdq_synth.make_act(M, K, 900 + M).cuda()
    p = m.sdq_decompose(W, cfg)
    xq = m.sdq_quantize_act(X, cfg)
    need = m.workspace_size(M, N, K, cfg)
    assert 0 < need <= m.STATIC_WS_BYTES          # this shape really uses the built-in scratch
    ws = m.make_workspace(M, N, K, cfg, "cuda")
    ref = m.sdq_linear(xq, p, workspace=ws)       # existing entry point, caller-owned scratch
    out1 = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    out2 = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    m.sdq_linear_noalloc(xq, p, out1)             # first call on the device also resolves the array's address
    m.sdq_linear_noalloc(xq, p, out2)             # second call reuses the array with the first call's leftovers
    assert m.device_status() == 0
    # same split order on both paths: the tolerance of the other tests (1e-3 relative on y) is met with equality
    assert torch.equal(out1, ref)
    assert torch.equal(out2, ref)
    d = (out1.float() - ref.float()).abs()
    assert (d <= 1e-3 * (ref.float().abs() + 1e-2)).all()
    # and against the CPU oracle itself: the bf16 output lies within one bf16 rounding of the oracle's value
    from oracle import sdq_oracle as so
    oc = so.Config(1, so.GRAN_PAIR, 64, so.SCALE_OCP_FLOOR)
    yref = so.linear(so.quantize_act(sdq_synth.bf16_bits(X.cpu()), oc), so.decompose(sdq_synth.bf16_bits(W.cpu()), oc))
    err = np.abs(out2.float().cpu().numpy().astype(np.float64) - yref)
    assert (err <= 2.0 ** -8 * np.abs(yref) + 1e-3 * (np.abs(yref) + 1e-2)).all()


def test_noalloc_refuses_shapes_beyond_its_fixed_scratch_and_runs_shapes_without_scratch():
    m = sdq()
    cfg = m.Config()
    # 128 tokens x 4096 rows split 4 ways needs 8 MiB of partial tiles: more than the built-in array
    M, N, K = 128, 4096, 1024
    assert m.workspace_size(M, N, K, cfg) > m.STATIC_WS_BYTES
    p = m.sdq_decompose(sdq_synth.make_weight(N, K, 7).cuda(), cfg)
    xq = m.sdq_quantize_act(sdq_synth.make_act(M, K, 7).cuda(), cfg)
    out = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(m.SdqError) as e:
        m.sdq_linear_noalloc(xq, p, out)
    assert e.value.code == 5
    # many tokens: no split, no scratch -- behaves as sdq_linear
    M = 200
    xq = m.sdq_quantize_act(sdq_synth.make_act(M, K, 8).cuda(), cfg)
    out = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    assert m.workspace_size(M, N, K, cfg) == 0
    m.sdq_linear_noalloc(xq, p, out)
    assert torch.equal(out, m.sdq_linear(xq, p))
