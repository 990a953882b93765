"""CPU-side checks: the C-ABI library loads and exports every symbol include/sdq.h declares, host-only entry points
validate their arguments, and the multi-rank aggregation of bench.py works over gloo with two ranks."""
import ctypes
import os
import re
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def m():
    import paper_2406_13868_b200 as mod
    mod.build()
    return mod


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in sorted(os.listdir(inc)):                    # every header of the boundary: sdq.h and sdq_diag.h
        if f.endswith(".h"):
            src = re.sub(r"/\*.*?\*/", "", open(os.path.join(inc, f)).read(), flags=re.S)
            names |= set(re.findall(r"\b(sdq_[a-z0-9_]+)\s*\(", src))
    return sorted(names)


def test_library_exports_every_declared_symbol(m):
    names = declared_symbols()
    assert "sdq_decompose" in names and "sdq_quantize_act" in names and "sdq_linear" in names
    L = m.lib()
    for n in names:
        assert hasattr(L, n), n
    assert sorted(m.EXPORTS) == names


def test_size_queries_and_argument_errors_without_a_gpu(m):
    L = m.lib()
    cfg = m.Config()
    b, a = ctypes.c_size_t(), ctypes.c_size_t()
    assert L.sdq_packed_size(4096, 4096, ctypes.byref(cfg), ctypes.byref(b), ctypes.byref(a)) == 0
    assert a.value == 4096 * 4096 // 2 + 4096 * 4      # 4.0 bits per weight + one fp32 scale per row
    assert b.value >= a.value
    assert L.sdq_packed_size(4096, 4000, ctypes.byref(cfg), ctypes.byref(b), ctypes.byref(a)) == 2   # K % 256
    assert L.sdq_packed_size(100, 4096, ctypes.byref(cfg), ctypes.byref(b), ctypes.byref(a)) == 2    # N % 128
    bad = m.Config(3, 0, 64, 0)
    assert L.sdq_packed_size(128, 256, ctypes.byref(bad), ctypes.byref(b), ctypes.byref(a)) == 1
    elem = m.Config(1, m.GRAN_ELEM, 32, 0)      # literal "2:4, block-32" reading: 2 + 1 + 0.25 + 1.375 bits per weight
    assert L.sdq_packed_size(128, 256, ctypes.byref(elem), ctypes.byref(b), ctypes.byref(a)) == 0
    assert a.value == int(128 * 256 * 4.625 / 8) + 128 * 4
    assert L.sdq_act_size(1, 4096, ctypes.byref(cfg), ctypes.byref(b)) == 0 and b.value > 4096 * 3 // 2
    assert L.sdq_act_size(0, 4096, ctypes.byref(cfg), ctypes.byref(b)) == 2
    # null pointers are rejected before anything is launched
    assert L.sdq_decompose(None, 128, 256, 256, ctypes.byref(cfg), None, 0, None, None) == 1
    assert L.sdq_linear(None, None, None, 0, None) == 1
    assert L.sdq_linear_noalloc(None, None, None, 0, None) == 1
    assert L.sdq_status_string(8) == b"device-side bounded wait timed out"
    assert L.sdq_status_string(0) == b"ok"


def test_compute_calls_refuse_cpu_tensors(m):
    W = torch.zeros((128, 256), dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        m.sdq_decompose(W)
    with pytest.raises(ValueError):
        m.sdq_quantize_act(W)


_WORKER = r"""
import os, sys, torch, torch.distributed as dist
sys.path.insert(0, sys.argv[1])
import bench
rank, world = int(sys.argv[2]), int(sys.argv[3])
os.environ["MASTER_ADDR"] = "127.0.0.1"; os.environ["MASTER_PORT"] = sys.argv[4]
dist.init_process_group("gloo", rank=rank, world_size=world)
ms_local = 10.0 if rank == 0 else 12.5          # the slower rank sets the job time
rate, ms = bench.aggregate_over_ranks(ms_local, 1000.0, world)
assert ms == 12.5, ms
assert abs(rate - world * 1000.0 / 12.5e-3) < 1e-6, rate
dist.barrier()
dist.destroy_process_group()
print("ok", rank)
"""


def test_weak_scaling_aggregation_two_ranks_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    port = str(29500 + os.getpid() % 2000)
    procs = [subprocess.Popen([sys.executable, str(script), ROOT, str(r), "2", port], stdout=subprocess.PIPE, stderr=subprocess.STDOUT)
             for r in range(2)]
    outs = [p.communicate(timeout=120)[0].decode() for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o
        assert "ok" in o


def test_attach_group_and_selftest_argument_errors_without_a_gpu(m):
    L = m.lib()
    d = m._Packed()
    assert L.sdq_packed_attach(None, 1 << 20, ctypes.byref(d), None) == 1          # null buffer
    assert L.sdq_packed_attach(ctypes.c_void_p(0x1008), 1 << 20, ctypes.byref(d), None) == 3   # not 16-byte aligned
    assert L.sdq_packed_attach(ctypes.c_void_p(0x1000), 100, ctypes.byref(d), None) == 5       # smaller than a header
    assert L.sdq_linear_group(0, None, None, None, None, None) == 1
    assert L.sdq_linear_group(2, None, None, None, None, None) == 1
    assert L.sdq_diag_wait_timeout(0, None) == 2 and L.sdq_diag_wait_timeout(5000, None) == 2  # polls outside 1 .. 4096
    i64 = ctypes.c_int64
    assert L.sdq_linear_group_x(1, None, i64(4), i64(1024), i64(1024), None, None, None, None) == 1                    # null X
    pp, yy, ld = (ctypes.c_void_p * 1)(), (ctypes.c_void_p * 1)(), (ctypes.c_int64 * 1)(1024)
    x = ctypes.c_void_p(0x1000)
    assert L.sdq_linear_group_x(1, x, i64(4), i64(1000), i64(1024), pp, yy, ld, None) == 2                             # K % 256
    assert L.sdq_linear_group_x(1, ctypes.c_void_p(0x1008), i64(4), i64(1024), i64(1024), pp, yy, ld, None) == 3       # X not 16-byte aligned
    assert L.sdq_linear_group_x(1, x, i64(4), i64(1024), i64(1020), pp, yy, ld, None) == 2                             # row stride shorter than K
    # the sixth configuration word: int8 outlier operands only with the primary inlier format and power-of-two inlier scales
    b = ctypes.c_size_t()
    assert L.sdq_packed_size(128, 256, ctypes.byref(m.Config(1, m.GRAN_PAIR, 64, 0, 0, m.OUT_INT8)), ctypes.byref(b), None) == 0
    assert L.sdq_packed_size(128, 256, ctypes.byref(m.Config(1, m.GRAN_PAIR, 32, 0, 0, m.OUT_INT8)), ctypes.byref(b), None) == 4
    assert L.sdq_packed_size(128, 256, ctypes.byref(m.Config(1, m.GRAN_PAIR, 32, m.SCALE_UE4M3, 0, m.OUT_INT8)), ctypes.byref(b), None) == 1
    assert L.sdq_packed_size(128, 256, ctypes.byref(m.Config(1, m.GRAN_PAIR, 64, 0, 0, 7)), ctypes.byref(b), None) == 1
    assert L.sdq_act_size(4, 256, ctypes.byref(m.Config(1, m.GRAN_PAIR, 64, 0, 0, 7)), ctypes.byref(b)) == 1
    # the compact form: 2.625 + 1.5 bits per weight plus scales and the header; only where there are outliers to compact
    c, full = ctypes.c_size_t(), ctypes.c_size_t()
    cfg = m.Config()
    assert L.sdq_packed_compact_size(i64(4096), i64(4096), ctypes.byref(cfg), ctypes.byref(c)) == 0
    assert L.sdq_packed_size(4096, 4096, ctypes.byref(cfg), ctypes.byref(full), None) == 0
    assert c.value * 8 / 4096 ** 2 < 4.2 and full.value - c.value == 4096 * 4096 * 5 // 8
    assert L.sdq_packed_compact_size(i64(4096), i64(4096), ctypes.byref(m.Config(0)), ctypes.byref(c)) == 4
    assert L.sdq_packed_compact_size(i64(4096), i64(4000), ctypes.byref(cfg), ctypes.byref(c)) == 2
    assert L.sdq_packed_compact(None, None, 0, None, None) == 1


def test_bench_starts_its_own_ranks_when_run_without_a_launcher():
    """`python bench.py --gpus 2` with no WORLD_SIZE around it must become two ranks: here with the timed body stubbed
    (CPU, gloo), through the same spawn path, rendezvous on 127.0.0.1, max-over-ranks timing, one JSON line from rank 0."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "4", "--stub-body"], env=env,
                       stdout=subprocess.PIPE, stderr=subprocess.PIPE, timeout=300)
    assert r.returncode == 0, r.stderr.decode()[-2000:]
    lines = [l for l in r.stdout.decode().splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout.decode()
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["stub"] is True
    # rank 1 "took" 20 ms for its 400 units, rank 0 10 ms: the job took the max, and processed both batches
    assert abs(d["ms_per_step"] - 20.0 / 4) < 1e-9
    assert abs(d["value"] - 2 * 400.0 / 20e-3) < 1e-6
