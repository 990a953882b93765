#!/usr/bin/env python
"""Benchmark of the SDQ decomposed linear layer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass of the hot path over one batch of synthetic input shaped like the MLP of a
LLaMA-7B decoder layer at prefill: quantize X [2048, 4096] -> gate and up projections (4096 -> 11008,
sharing the quantized X) -> quantize H [2048, 11008] -> down projection (11008 -> 4096).  Weights are
decomposed and packed offline (untimed).  The headline value is dense-equivalent TFLOP/s of the whole
step (2*M*N*K per projection).  A second, separately timed region measures the decode shape
(M in {1, 16}, 4096 x 4096 attention projection, rotating over 32 distinct layers) in GB/s of
algorithmic compressed-weight bytes and is reported under "decode".

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import sdq_synth  # noqa: E402

METRIC = "sdq_linear_dense_equiv_tflops_prefill"
UNIT = "TFLOP/s"
WORKLOAD = "llama7b_mlp_prefill_M2048 (gate,up 4096->11008; down 11008->4096; 1:8 FP8 outlier + pair-wise 4:8 MXFP4 inlier, block 64)"
M_PREFILL, D_MODEL, D_FF = 2048, 4096, 11008
# Mixed-instruction tensor roofline: per dense-equivalent flop the layer issues one sparse-FP4 flop
# (nominally 8x the bf16 rate) and one sparse-FP8 flop (4x): peak = bf16_peak / (1/8 + 1/4).
MIXED_PEAK_OVER_BF16 = 1.0 / (1.0 / 8.0 + 1.0 / 4.0)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm=d["hbm_gbs"], bf16=d["bf16_tflops"], bf16_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                    source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """samples nvidia-smi clocks / throttle reasons while the timed region runs"""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                                       "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        # median over the upper half of the samples = clocks under load (the sampler also sees idle edges)
        hi = sorted(sm)[len(sm) // 2:]
        return {"sm_mhz": statistics.median(hi), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------------------------- oracle arm
class OracleSample:
    """The CPU oracle (as it stands) on a bounded sample of the prefill workload: `rows_x` tokens through
    the first `n_rows_w` output features of the gate projection; activation quantization is inside the
    timed region, the weight decomposition is offline (untimed), exactly as on the GPU arm."""

    def __init__(self, rows_x: int, n_rows_w: int = D_FF, seed: int = 3000):
        from oracle import sdq_oracle as so
        self.so = so
        self.cfg = so.Config(1, so.GRAN_PAIR, 64, so.SCALE_OCP_FLOOR)
        W = sdq_synth.bf16_bits(sdq_synth.make_weight(n_rows_w, D_MODEL, seed + 1))
        self.X = sdq_synth.bf16_bits(sdq_synth.make_act(rows_x, D_MODEL, seed + 4))
        self.p = so.decompose(W, self.cfg)
        self.threads = os.cpu_count() or 1
        self.flops = 2.0 * rows_x * n_rows_w * D_MODEL
        self.desc = "%d of 2048 tokens x %d of 11008 gate rows x K=4096 (quantize_act + product, fp64 accumulate)" % (rows_x, n_rows_w)

    def run(self):
        t0 = time.perf_counter()
        q = self.so.quantize_act(self.X, self.cfg)
        self.so.linear(q, self.p, threads=self.threads)
        dt = time.perf_counter() - t0
        return self.flops / dt / 1e12, dt


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # each step is a bounded sample; sized so that a 20+3 step run still ends within a few minutes
    sample = OracleSample(rows_x=256)
    vals, secs = [], []
    for i in range(args.warmup + args.steps):
        v, dt = sample.run()
        if i >= args.warmup:
            vals.append(v); secs.append(dt)
    v = sum(vals) / len(vals)
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * sum(secs) / len(secs), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": sample.desc},
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": sample.threads, "kind": "oracle", "sample": sample.desc},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def aggregate_over_ranks(ms_local: float, units_per_rank: float, world: int, device="cpu"):
    """Whole-job throughput under weak scaling: every rank processed `units_per_rank` in `ms_local`; the job took
    the MAX over ranks (all-reduce), and processed world * units_per_rank.  Returns (units per second, max ms)."""
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms = float(t.item())
    return world * units_per_rank / (ms * 1e-3), ms


# ----------------------------------------------------------------------------------------------- CUDA arm
def spawn_ranks(args) -> int:
    """`python bench.py --gpus N` without a launcher: start the N ranks (one process per GPU, NCCL rendezvous on the
    loopback address) through torch.distributed.run and pass their exit code on."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus), "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__), "--gpus", str(args.gpus), "--steps", str(args.steps), "--warmup",
           str(args.warmup), "--impl", args.impl] + (["--stub-body"] if args.stub_body else [])
    return subprocess.call(cmd)


def run_stub(args):
    """The rank plumbing of the CUDA arm with the timed body replaced by a fixed duration (CPU, gloo): what the
    multi-process test drives to check rendezvous, barrier, max-over-ranks and the one JSON line of rank 0."""
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    ms_local = 10.0 * (1 + rank)                       # rank r "took" 10 (r + 1) ms for its batch
    units_per_s, ms_max = aggregate_over_ranks(ms_local, 100.0 * args.steps, world, "cpu")
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "stub": True, "n_gpus": world, "steps": args.steps, "ms_per_step": ms_max / args.steps,
                          "value": units_per_s, "scaling": "weak"}))


def run_ours(args):
    import paper_2406_13868_b200 as sdq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    cfg = sdq.Config(1, sdq.GRAN_PAIR, 64, sdq.SCALE_OCP_FLOOR)
    peaks = measured_peaks()

    # ---- synthetic layer (seed = config index * 1000 + rank; weak scaling: every rank has its own batch)
    seed = 3000 + rank
    Wg = sdq_synth.make_weight(D_FF, D_MODEL, seed + 1, device=str(dev))
    Wu = sdq_synth.make_weight(D_FF, D_MODEL, seed + 2, device=str(dev))
    Wd = sdq_synth.make_weight(D_MODEL, D_FF, seed + 3, device=str(dev))
    X = sdq_synth.make_act(M_PREFILL, D_MODEL, seed + 4, device=str(dev))
    H = sdq_synth.make_act(M_PREFILL, D_FF, seed + 5, device=str(dev))
    Pg, Pu, Pd = (sdq.sdq_decompose(w, cfg) for w in (Wg, Wu, Wd))
    del Wg, Wu, Wd
    bx = torch.empty(sdq.act_size(M_PREFILL, D_MODEL, cfg), dtype=torch.uint8, device=dev)
    bh = torch.empty(sdq.act_size(M_PREFILL, D_FF, cfg), dtype=torch.uint8, device=dev)
    Yg = torch.empty((M_PREFILL, D_FF), dtype=torch.bfloat16, device=dev)
    Yu = torch.empty_like(Yg)
    Yd = torch.empty((M_PREFILL, D_MODEL), dtype=torch.bfloat16, device=dev)
    flops_step = 3 * 2.0 * M_PREFILL * D_MODEL * D_FF
    launches_per_step = 5   # 2 x quant_act_fused + 3 x sdq_linear

    ev = []   # (kind, start, end) per launch in the timed region

    def step(which=-1):
        """one pass of the hot path.  `which` selects what is bracketed by a CUDA event pair in this step: 0 the first
        quantizer, 1 the gate and up GEMMs together (two launches, one pair), 2 the second quantizer, 3 the down GEMM.
        Only one bracket per step: an event pair around every launch costs ~10 % of the step (gaps between dependent
        kernels), and a pair around two launches halves the share of its own overhead (~4 us) in the duration."""
        def timed(i, kind, n, fn):
            if i == which:
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); r = fn(); b.record(); ev.append((kind, n, a, b))
                return r
            return fn()
        xq = timed(0, "quant", 1, lambda: sdq.sdq_quantize_act(X, cfg, bx))
        timed(1, "gemm", 2, lambda: (sdq.sdq_linear(xq, Pg, Yg), sdq.sdq_linear(xq, Pu, Yu)))
        hq = timed(2, "quant", 1, lambda: sdq.sdq_quantize_act(H, cfg, bh))
        timed(3, "gemm", 1, lambda: sdq.sdq_linear(hq, Pd, Yd))

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    assert sdq.device_status() == 0, "device-side timeout flag set"
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.1)
    barrier(); torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        step(which=(1, 3, 1, 0, 2)[i % 5])      # GEMMs first, so that a short run still samples each of them
    e1.record()
    torch.cuda.synchronize(); barrier()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    assert sdq.device_status() == 0, "device-side timeout flag set"
    flops_per_s, ms_max = aggregate_over_ranks(ms_total, flops_step * args.steps, world, dev)
    ms_step = ms_max / args.steps
    value = flops_per_s / 1e12

    gemm_ms = sum(a.elapsed_time(b) for k, n, a, b in ev if k == "gemm")
    gemm_n = sum(n for k, n, a, b in ev if k == "gemm")
    quant_ms = [a.elapsed_time(b) for k, n, a, b in ev if k == "quant"]
    # the three projections have the same flop count, so the mean duration of the sampled launches gives the rate
    gemm_tf = (flops_step / 3) / (gemm_ms / gemm_n * 1e-3) / 1e12
    mixed_peak = peaks["bf16"] * MIXED_PEAK_OVER_BF16
    roofline = {"kernel": "sdq_linear_pair_kernel", "bound": "tensor", "achieved": gemm_tf, "peak": mixed_peak, "unit": "TFLOP/s",
                "frac": gemm_tf / mixed_peak,
                # dram__bytes_read.sum + dram__bytes_write.sum of one captured launch of the gate / up shape
                # (profiles/sdq_linear_pair_kernel_prefill_M2048_N11008_K4096.md); the down shape was not captured
                "traffic": 84.1e6, "traffic_unit": "bytes per launch (gate/up shape)",
                "peak_basis": "%s bf16 burst %.1f TF/s x 8/3 (sparse FP4 at 8x + sparse FP8 at 4x per dense-equivalent flop)" % (peaks["source"], peaks["bf16"]),
                "avg_launch_ms": gemm_ms / gemm_n, "launches": gemm_n,
                # what actually bounds the kernel: bytes staged from L2 into shared memory per launch against the rate that
                # all SMs pulling together reach in a copy-only kernel, measured in this run
                "l2_to_sm": l2_to_sm(sdq, dev, gemm_ms / gemm_n),
                "frac_of_sparse_fp4_peak": gemm_tf / (8 * peaks["bf16"])}
    # activation quantizer alone (quant_act_fused_kernel), back to back on the larger input so that
    # host launch overhead does not count: bytes = bf16 read + 4-bit codes + 8-bit codes + one scale byte per 64
    qa, qb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    qreps = 20
    sdq.sdq_quantize_act(H, cfg, bh)
    qa.record()
    for _ in range(qreps):
        sdq.sdq_quantize_act(H, cfg, bh)
    qb.record()
    torch.cuda.synchronize()
    quant_bytes = M_PREFILL * D_FF * (2 + 0.5 + 1.0 + 1.0 / 64)
    quant = {"kernel": "quant_act_fused_kernel", "bound": "hbm", "achieved": quant_bytes * qreps / (qa.elapsed_time(qb) * 1e-3) / 1e9,
             "peak": peaks["hbm"], "unit": "GB/s", "workload": "X 2048 x 11008 bf16, %d back-to-back calls" % qreps,
             "in_step_ms": sum(quant_ms) / max(1, len(quant_ms))}
    quant["frac"] = quant["achieved"] / quant["peak"]

    if rank != 0:
        return
    # ---- decode shape (C2): 4096x4096, M in {1,16}, rotating over 32 distinct packed layers (> L2)
    decode = measure_decode(sdq, cfg, dev, peaks)
    # ---- the same step with one scale per 32 K (the literal block-32 MXFP4 wording), timed the same way
    cfg32 = sdq.Config(1, sdq.GRAN_PAIR, 32, sdq.SCALE_OCP_FLOOR)
    b32 = measure_variant_step(sdq, cfg32, dev, rank, X, H, (Yg, Yu, Yd), flops_step, args.steps,
                               "the same step with one E8M0 scale per 32 K for inlier weights and 4-bit activations")
    # ---- and without Stage 1: 8:8 split as 1:8 FP8 outliers + dense MXFP4 inliers (dense kind::mxf4, one scale per 32 K)
    cfgd = sdq.Config(1, sdq.GRAN_DENSE, 32, sdq.SCALE_OCP_FLOOR)
    dns = measure_variant_step(sdq, cfgd, dev, rank, X, H, (Yg, Yu, Yd), flops_step, args.steps,
                               "the same step without pruning: 1:8 FP8 outliers + dense MXFP4 inliers, one scale per 32 K")
    # ---- the configuration as the benchmark spec words it: element-wise 2:4 inliers, one E8M0 scale per 32 K (stored and run as a
    # dense 4-bit operand: the sparse FP4 tensor core takes pairs only)
    cfgl = sdq.Config(1, sdq.GRAN_ELEM, 32, sdq.SCALE_OCP_FLOOR)
    lit = measure_variant_step(sdq, cfgl, dev, rank, X, H, (Yg, Yu, Yd), flops_step, args.steps,
                               "the same step with the literal wording: element-wise 2:4 MXFP4 inliers, block 32, 1:8 FP8 outliers")
    # ---- the headline step repeated for >= 1 s: clocks settle under the power cap; against the sustained bf16 peak
    sustained = measure_sustained(sdq, step, flops_step, local, peaks)
    # ---- end to end through the public API with host buffers (pinned), copies inside the timed region
    e2e = measure_e2e(sdq, cfg, dev, X, H, (Pg, Pu, Pd), (bx, bh), (Yg, Yu, Yd), flops_step, max(3, args.steps // 2))
    sample = OracleSample(rows_x=1024)
    v, dt = sample.run()
    threads, desc = sample.threads, sample.desc
    # ---- and with E4M3 Q-Vector scales under power-of-two row / token factors (the scale-factor format the paper prefers)
    cfge = sdq.Config(1, sdq.GRAN_PAIR, 32, sdq.SCALE_UE4M3)
    e4 = measure_variant_step(sdq, cfge, dev, rank, X, H, (Yg, Yu, Yd), flops_step, args.steps,
                              "the same step with E4M3 scale codes per 32 K and power-of-two row / token factors (two-level scaling)")
    packer = measure_packer(sdq, cfg, dev, peaks)
    del Pg, Pu, Pd
    torch.cuda.empty_cache()
    opt_ffn, keep = measure_opt_ffn(sdq, dev, peaks)
    del keep
    torch.cuda.empty_cache()
    model, keep = measure_model(sdq, dev, peaks)
    del keep
    torch.cuda.empty_cache()
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp4+fp8 (E2M1/E4M3 products, fp32 accumulate)",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "tokens_per_gpu": M_PREFILL, "l2": "packed weights + activations of one step exceed L2 (150 MB > 126 MB)",
                       "parallelism": "dp%d (independent batches, no collective)" % world},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "quantizer_roofline": quant, "sustained": sustained, "scale_block_32": b32, "literal_elem_2of4_block_32": lit, "dense_inliers": dns, "e4m3_scales": e4,
            "decode": decode, "packer_roofline": packer, "opt67b_ffn_M4096": opt_ffn, "llama7b_224_linears": model,
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc, "seconds": dt}}
    print(json.dumps(line))


def l2_to_sm(sdq, dev, gemm_launch_ms):
    """The ceiling of the L2 -> shared-memory path measured live with the library's copy-only kernel (every SM keeps 128 to
    220 KB of bulk copies in flight from a 37 MB, L2-resident source; best of four copy shapes, each the best of five
    launches of ~2 GB), and the fraction of it that the GEMM's staged operand bytes reach.  Staged bytes per launch of the
    CTA-pair kernel: per CTA and 256 x 256 tile, 16 inlier stages of 28160 B (weight record + own 128 tokens' codes + two
    scale atoms) + 32 outlier stages of 26624 B + 1536 B of outlier scale atoms = 1.304 MB; x 2 CTAs x 344 tiles = 0.897 GB
    for the gate / up shape (0.897 GB for the down shape too: 128 tiles of 43 + 86 stages)."""
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    src = torch.empty(sms * (256 << 10), dtype=torch.uint8, device=dev).fill_(1)
    best = 0.0
    for slot, nslot, issuers in ((65536, 3, 1), (32768, 6, 3), (16384, 13, 3), (14336, 15, 3)):
        for rep in range(7):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            moved = sdq.diag_l2_copy(src, slot, nslot, (12 << 20) // slot, issuers)
            b.record()
            torch.cuda.synchronize()
            if rep >= 2:
                best = max(best, moved / (a.elapsed_time(b) * 1e-3) / 1e12)
    staged = 0.897e9
    ach = staged / (gemm_launch_ms * 1e-3) / 1e12
    return {"bytes_per_launch": staged, "achieved_TBps": ach, "measured_ceiling_TBps": best, "frac": ach / best,
            "ceiling_basis": "copy-only kernel of this library (sdq_diag_l2_copy), all SMs, best of 3 x 64 KB, 6 x 32 KB, 13 x 16 KB and 15 x 14 KB bulk copies in flight per SM, L2-resident source"}


def measure_decode(sdq, cfg, dev, peaks, layers: int = 32, reps: int = 20):
    """Decode shape (configs[1]): 4096 x 4096, M in {1, 16}, rotating over 32 distinct packed layers (> L2).  Two ways
    of enqueuing the same 32 independent products, each captured once in a CUDA graph and replayed: ONE
    sdq_linear_group call (one persistent launch streaming the compact outlier records), and 32 sdq_linear calls
    (cluster split-K, consecutive launches overlapped by programmatic dependent launch)."""
    N = K = 4096
    packs = []
    for i in range(layers):
        W = sdq_synth.make_weight(N, K, 2000 + i, device=str(dev))
        packs.append(sdq.sdq_decompose(W, cfg))
        del W
    algo = packs[0].algorithmic_bytes
    # the grouped call runs from the compact form of the same layers (no 2:4 outlier containers: what it streams is all that is resident)
    cpacks = [sdq.packed_compact(p) for p in packs]
    out = {}
    for M in (1, 16):
        X = sdq_synth.make_act(M, K, 2100 + M, device=str(dev))
        Ys = [torch.empty((M, N), dtype=torch.bfloat16, device=dev) for _ in packs]
        xb = torch.empty(sdq.act_size(M, K, cfg), dtype=torch.uint8, device=dev)
        xq = sdq.sdq_quantize_act(X, cfg, xb)

        def grouped():
            sdq.sdq_linear_group([xq] * layers, cpacks, Ys)

        def chain():
            for p, y in zip(packs, Ys):
                sdq.sdq_linear(xq, p, y)
        res = {}
        for name, fn in (("group", grouped), ("chain", chain)):
            us = time_graph(fn, reps=reps) * 1e3 / layers
            assert sdq.device_status() == 0
            gbs = algo / (us * 1e-6) / 1e9
            res[name] = {"us_per_layer": us, "weight_GBps_algorithmic": gbs, "frac_of_hbm_peak": gbs / peaks["hbm"]}
        # four grouped calls per graph replay: the replay's own fixed cost (~4 us) spread over 128 layers
        us4 = time_graph(lambda: [grouped() for _ in range(4)], reps=max(reps // 2, 5)) * 1e3 / (4 * layers)
        gbs4 = algo / (us4 * 1e-6) / 1e9
        out["M%d" % M] = dict(res["group"], call="sdq_linear_group, 32 layers in one launch",
                              four_calls_per_graph={"us_per_layer": us4, "weight_GBps_algorithmic": gbs4, "frac_of_hbm_peak": gbs4 / peaks["hbm"]},
                              per_call_chain=dict(res["chain"], call="32 x sdq_linear"))
    # the evaluation's outlier format (int8 with fp32 scales, Section 5.1) through the same grouped call
    cfg8 = sdq.Config(cfg.out_n, cfg.in_gran, cfg.in_block, cfg.scale_rule, cfg.out_order, sdq.OUT_INT8)
    packs8 = []
    for i in range(layers):
        W = sdq_synth.make_weight(N, K, 2000 + i, device=str(dev))
        packs8.append(sdq.sdq_decompose(W, cfg8))
        del W
    out["int8_outliers"] = {}
    for M in (1, 16):
        X = sdq_synth.make_act(M, K, 2100 + M, device=str(dev))
        Ys = [torch.empty((M, N), dtype=torch.bfloat16, device=dev) for _ in packs8]
        xq = sdq.sdq_quantize_act(X, cfg8)
        us = time_graph(lambda: sdq.sdq_linear_group([xq] * layers, packs8, Ys), reps=reps) * 1e3 / layers
        assert sdq.device_status() == 0
        gbs = algo / (us * 1e-6) / 1e9
        out["int8_outliers"]["M%d" % M] = {"us_per_layer": us, "weight_GBps_algorithmic": gbs, "frac_of_hbm_peak": gbs / peaks["hbm"],
                                           "call": "sdq_linear_group, 32 layers in one launch, SDQ_OUT_INT8"}
    del packs8
    out["workload"] = ("llama7b_attn_proj_decode 4096x4096, %d distinct layers in rotation (%.0f MB packed > L2), products only, "
                       "one CUDA graph per variant replayed %d times" % (layers, layers * packs[0].buf.numel() / 1e6, reps))
    out["algorithmic_bytes_per_layer"] = algo
    out["streamed_bytes_per_layer"] = {"group": int(N * K * 4.125 / 8), "chain": int(N * K * 7.625 / 8)}
    out["stored_bytes_per_layer"] = {"group (compact form, sdq_packed_compact)": int(cpacks[0].buf.numel()), "chain (full form)": int(packs[0].buf.numel())}
    out["stored_bits_per_weight"] = {"group": cpacks[0].buf.numel() * 8.0 / (N * K), "chain": packs[0].buf.numel() * 8.0 / (N * K)}
    out["hbm_peak_GBps"] = peaks["hbm"]
    return out


def measure_variant_step(sdq, cfg, dev, rank, X, H, outs, flops_step, steps, workload):
    """The benchmark step under another configuration (in_block = 32 on kind::mxf4nvf4 .block16; dense inliers on the
    dense kind::mxf4): fresh packed weights of the same shapes, the same inputs and output buffers; whole-step
    throughput from one event pair around `steps` steps."""
    seed = 3000 + rank
    packs = []
    for i, (n, k) in enumerate(((D_FF, D_MODEL), (D_FF, D_MODEL), (D_MODEL, D_FF))):
        W = sdq_synth.make_weight(n, k, seed + 1 + i, device=str(dev))
        packs.append(sdq.sdq_decompose(W, cfg))
        del W
    bx = torch.empty(sdq.act_size(M_PREFILL, D_MODEL, cfg), dtype=torch.uint8, device=dev)
    bh = torch.empty(sdq.act_size(M_PREFILL, D_FF, cfg), dtype=torch.uint8, device=dev)

    def step():
        xq = sdq.sdq_quantize_act(X, cfg, bx)
        sdq.sdq_linear(xq, packs[0], outs[0])
        sdq.sdq_linear(xq, packs[1], outs[1])
        hq = sdq.sdq_quantize_act(H, cfg, bh)
        sdq.sdq_linear(hq, packs[2], outs[2])
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        step()
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / steps
    assert sdq.device_status() == 0
    return {"value": flops_step / (ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms, "workload": workload}


def measure_sustained(sdq, step, flops_step, gpu_index, peaks, seconds: float = 1.2):
    """The benchmark step back to back for at least `seconds`, clocks sampled meanwhile: the number a long-running job
    sees once the part sits at its power cap, set against the sustained bf16 peak (x 8/3 for the instruction mix)."""
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(); step(); b.record(); torch.cuda.synchronize()
    n = max(50, int(seconds * 1e3 / a.elapsed_time(b)) + 1)
    sampler = ClockSampler(gpu_index)
    sampler.start()
    time.sleep(0.1)
    a.record()
    for _ in range(n):
        step()
    b.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = a.elapsed_time(b)
    tf = flops_step * n / (ms * 1e-3) / 1e12
    peak = peaks["bf16_sustained"] * MIXED_PEAK_OVER_BF16
    return {"value": tf, "unit": UNIT, "steps": n, "seconds": ms * 1e-3, "ms_per_step": ms / n, "clocks": clocks,
            "frac_of_sustained_mixed_peak": tf / peak, "peak": peak,
            "peak_basis": "%s bf16 sustained %.1f TF/s x 8/3" % (peaks["source"], peaks["bf16_sustained"])}


def measure_packer(sdq, cfg, dev, peaks, N: int = D_FF, K: int = D_MODEL, reps: int = 10):
    """Offline weight packing (pack_kernel) on the gate shape: bytes = the bf16 weights read once + the algorithmic packed
    bytes written, against the HBM peak.  (sdq_decompose synchronises its stream to read back the non-finite flag, so
    the launches are timed one by one with events around each call.)"""
    W = sdq_synth.make_weight(N, K, 9001, device=str(dev))
    nbytes, algo = sdq.packed_size(N, K, cfg)
    buf = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    best = 1e9
    for i in range(reps + 2):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        sdq.sdq_decompose(W, cfg, buf)
        b.record()
        torch.cuda.synchronize()
        if i >= 2:
            best = min(best, a.elapsed_time(b))
    moved = N * K * 2 + algo
    gbs = moved / (best * 1e-3) / 1e9
    return {"kernel": "pack_kernel", "bound": "hbm", "achieved": gbs, "peak": peaks["hbm"], "unit": "GB/s", "frac": gbs / peaks["hbm"],
            "ms": best, "workload": "W %d x %d bf16 -> packed (best of %d calls, includes the call's flag read-back)" % (N, K, reps),
            "bytes_counted": moved, "bytes_written_all_sections": nbytes}


def measure_e2e(sdq, cfg, dev, X, H, packs, bufs, outs, flops_step, steps):
    """The same step through the public API from HOST buffers: every step copies its inputs in from pinned memory and
    its three outputs back.  The copies run on their own streams with two sets of device buffers, so that step i+1's
    inputs go in and step i-1's outputs come out while step i computes (PCIe is full duplex); the timed region covers
    all of it."""
    Xh, Hh = X.cpu().pin_memory(), H.cpu().pin_memory()
    Yh = [[torch.empty(o.shape, dtype=o.dtype).pin_memory() for o in outs] for _ in range(2)]
    Xd, Hd = [torch.empty_like(X) for _ in range(2)], [torch.empty_like(H) for _ in range(2)]
    Yd = [list(outs), [torch.empty_like(o) for o in outs]]
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]       # inputs of buffer set b are on the device
    ev_done = [torch.cuda.Event() for _ in range(2)]     # the step on buffer set b has finished
    ev_out = [torch.cuda.Event() for _ in range(2)]      # outputs of buffer set b are back on the host
    for e in ev_done + ev_out:
        e.record(main)

    def step(i):
        b = i & 1
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_done[b])                  # the step that last read these input buffers is over
            Xd[b].copy_(Xh, non_blocking=True)
            Hd[b].copy_(Hh, non_blocking=True)
            ev_in[b].record(s_in)
        main.wait_event(ev_in[b])
        main.wait_event(ev_out[b])                       # the outputs written two steps ago have been read back
        xq = sdq.sdq_quantize_act(Xd[b], cfg, bufs[0])
        sdq.sdq_linear(xq, packs[0], Yd[b][0])
        sdq.sdq_linear(xq, packs[1], Yd[b][1])
        hq = sdq.sdq_quantize_act(Hd[b], cfg, bufs[1])
        sdq.sdq_linear(hq, packs[2], Yd[b][2])
        ev_done[b].record(main)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_done[b])
            for yh, yd in zip(Yh[b], Yd[b]):
                yh.copy_(yd, non_blocking=True)
            ev_out[b].record(s_out)

    for i in range(4):
        step(i)
    torch.cuda.synchronize()
    a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(main)
    for i in range(steps):
        step(i)
    main.wait_stream(s_in)
    main.wait_stream(s_out)
    e.record(main)
    torch.cuda.synchronize()
    ms = a.elapsed_time(e) / steps
    return {"value": flops_step / (ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms,
            "h2d_bytes_per_step": int(Xh.numel() * 2 + Hh.numel() * 2), "d2h_bytes_per_step": int(sum(y.numel() * 2 for y in Yh[0])),
            "pipelining": "copies on their own streams, two buffer sets"}


def run_case(args):
    """Small single-kernel cases for profiler captures (few launches, a few hundred MB on the device)."""
    import paper_2406_13868_b200 as sdq
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    cfg = sdq.Config(1, sdq.GRAN_PAIR, 64, sdq.SCALE_OCP_FLOOR)
    if args.case == "gemm_prefill_b32":          # one scale per 32 K
        cfg = sdq.Config(1, sdq.GRAN_PAIR, 32, sdq.SCALE_OCP_FLOOR)
    elif args.case == "gemm_prefill_e4m3":       # E4M3 scale codes per 32 K, power-of-two row / token factors
        cfg = sdq.Config(1, sdq.GRAN_PAIR, 32, sdq.SCALE_UE4M3)
    elif args.case == "gemm_prefill_dense":      # 8:8 = 1:8 FP8 outliers + dense MXFP4 inliers
        cfg = sdq.Config(1, sdq.GRAN_DENSE, 32, sdq.SCALE_OCP_FLOOR)
    elif args.case == "gemm_prefill_mxfp4":      # no outliers, no pruning: a plain block-scaled 4-bit GEMM
        cfg = sdq.Config(0, sdq.GRAN_DENSE, 32, sdq.SCALE_OCP_FLOOR)
    if args.case == "pack":                      # the offline packer alone, on the gate shape
        W = sdq_synth.make_weight(D_FF, D_MODEL, 1, device=str(dev))
        for _ in range(args.steps):
            sdq.sdq_decompose(W, cfg)
        torch.cuda.synchronize()
        print(json.dumps({"case": args.case, "N": D_FF, "K": D_MODEL, "launches": args.steps}))
        return
    if args.case == "group_decode":              # 16 layers of 4096 x 4096 at 16 tokens in one grouped launch (139 MB > L2)
        packs = [sdq.sdq_decompose(sdq_synth.make_weight(4096, 4096, 10 + i, device=str(dev)), cfg) for i in range(16)]
        xq = sdq.sdq_quantize_act(sdq_synth.make_act(16, 4096, 2, device=str(dev)), cfg)
        Ys = [torch.empty((16, 4096), dtype=torch.bfloat16, device=dev) for _ in packs]
        for _ in range(args.steps):
            sdq.sdq_linear_group([xq] * 16, packs, Ys)
        torch.cuda.synchronize()
        assert sdq.device_status() == 0
        print(json.dumps({"case": args.case, "layers": 16, "M": 16, "launches": args.steps}))
        return
    if args.case.startswith("gemm_prefill"):
        M, K, N = M_PREFILL, D_MODEL, D_FF
    elif args.case == "gemm_decode":
        M, K, N = 16, 4096, 4096
    else:
        M, K, N = M_PREFILL, D_FF, 128
    W = sdq_synth.make_weight(N, K, 1, device=str(dev))
    X = sdq_synth.make_act(M, K, 2, device=str(dev))
    P = sdq.sdq_decompose(W, cfg)
    Y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
    for _ in range(args.steps):
        xq = sdq.sdq_quantize_act(X, cfg)
        sdq.sdq_linear(xq, P, Y)
    torch.cuda.synchronize()
    assert sdq.device_status() == 0
    print(json.dumps({"case": args.case, "M": M, "N": N, "K": K, "launches": args.steps}))


def time_graph(fn, reps=10):
    """captures fn() once in a CUDA graph and returns the mean replay time in ms"""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        fn()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    g.replay()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        g.replay()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


def measure_opt_ffn(sdq, dev, peaks):
    """configs[3]: OPT-6.7B-shaped FFN at prefill, M = 4096: fc1 4096 -> 16384 and fc2 16384 -> 4096 with the outlier pattern
    swept over 1:8, 2:8 and none (products only, one CUDA graph per GEMM)."""
    M = 4096
    X = sdq_synth.make_act(M, 4096, 4001, device=str(dev))
    H = sdq_synth.make_act(M, 16384, 4002, device=str(dev))
    W1 = sdq_synth.make_weight(16384, 4096, 4003, device=str(dev))
    W2 = sdq_synth.make_weight(4096, 16384, 4004, device=str(dev))
    Y1 = torch.empty((M, 16384), dtype=torch.bfloat16, device=dev)
    Y2 = torch.empty((M, 4096), dtype=torch.bfloat16, device=dev)
    fl = 2.0 * M * 4096 * 16384
    c4 = {"workload": "opt6.7b_ffn_prefill_M4096 (fc1 4096->16384, fc2 16384->4096), products only"}
    for on, name in ((1, "1:8"), (2, "2:8"), (0, "none")):
        cfg = sdq.Config(on, sdq.GRAN_PAIR, 64, 0)
        P1, P2 = sdq.sdq_decompose(W1, cfg), sdq.sdq_decompose(W2, cfg)
        xq, hq = sdq.sdq_quantize_act(X, cfg), sdq.sdq_quantize_act(H, cfg)
        t1 = time_graph(lambda: sdq.sdq_linear(xq, P1, Y1))
        t2 = time_graph(lambda: sdq.sdq_linear(hq, P2, Y2))
        # roofline of the pattern: sparse FP4 for the inliers (8x the bf16 peak) + sparse FP8 for the outlier part (4x), if any
        peak = peaks["bf16"] / (1.0 / 8.0 + (1.0 / 4.0 if on else 0.0))
        c4[name] = {"fc1_ms": t1, "fc1_TFLOPs": fl / t1 / 1e9, "fc2_ms": t2, "fc2_TFLOPs": fl / t2 / 1e9,
                    "frac_of_tensor_roofline": (fl / t1 / 1e9 + fl / t2 / 1e9) / 2 / peak, "roofline_TFLOPs": peak}
        del P1, P2, xq, hq
    return c4, (X, H, W1, W2, Y1, Y2)


def measure_model(sdq, dev, peaks, token_counts=(1, 16, 128, 1024, 8192)):
    """configs[4]: all 224 linear layers of a 32-layer LLaMA-7B-shaped decoder back to back on one stream, as one CUDA
    graph per token count (activation quantization where a new activation enters + the products).  For M <= 16 also with
    the independent projections of a layer issued as grouped calls (q, k, v together; gate, up together)."""
    cfg = sdq.Config(1, sdq.GRAN_PAIR, 64, 0)
    shapes = [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)]
    layers = []
    algo = 0
    for l in range(32):
        ps = []
        for i, (N, K) in enumerate(shapes):
            W = sdq_synth.make_weight(N, K, 5000 + 10 * l + i, device=str(dev))
            ps.append(sdq.sdq_decompose(W, cfg))
            algo += ps[-1].algorithmic_bytes
            del W
        layers.append(ps)
    mixed_peak = peaks["bf16"] * MIXED_PEAK_OVER_BF16
    c5 = {"workload": "llama7b_32_layers_224_linears (q,k,v,o 4096x4096; gate,up 4096->11008; down 11008->4096), 1%% outlier channels x30",
          "algorithmic_weight_bytes": algo}
    for M in token_counts:
        X = sdq_synth.make_act(M, 4096, 5500 + M, n_outlier_channels=41, device=str(dev))
        Hh = sdq_synth.make_act(M, 11008, 5600 + M, n_outlier_channels=110, device=str(dev))
        bx = torch.empty(sdq.act_size(M, 4096, cfg), dtype=torch.uint8, device=dev)
        bh = torch.empty(sdq.act_size(M, 11008, cfg), dtype=torch.uint8, device=dev)
        Ya = [torch.empty((M, 4096), dtype=torch.bfloat16, device=dev) for _ in range(3)]
        Yb = [torch.empty((M, 11008), dtype=torch.bfloat16, device=dev) for _ in range(2)]

        def model(grouped=False, fused=False):
            for ps in layers:
                if fused:                                      # quantizer inside the grouped kernel: no quantized buffer, no launch
                    sdq.sdq_linear_group_x(X, ps[0:3], Ya)
                    xq = sdq.sdq_quantize_act(X, cfg, bx)      # input of o
                    sdq.sdq_linear(xq, ps[3], Ya[0])
                    sdq.sdq_linear_group_x(X, ps[4:6], Yb)
                    hq = sdq.sdq_quantize_act(Hh, cfg, bh)     # input of down
                    sdq.sdq_linear(hq, ps[6], Ya[0])
                    continue
                xq = sdq.sdq_quantize_act(X, cfg, bx)          # input of q, k, v
                if grouped:
                    sdq.sdq_linear_group([xq] * 3, ps[0:3], Ya)
                else:
                    for j in range(3):
                        sdq.sdq_linear(xq, ps[j], Ya[j])
                xq = sdq.sdq_quantize_act(X, cfg, bx)          # input of o
                sdq.sdq_linear(xq, ps[3], Ya[0])
                xq = sdq.sdq_quantize_act(X, cfg, bx)          # input of gate, up
                if grouped:
                    sdq.sdq_linear_group([xq] * 2, ps[4:6], Yb)
                else:
                    sdq.sdq_linear(xq, ps[4], Yb[0])
                    sdq.sdq_linear(xq, ps[5], Yb[1])
                hq = sdq.sdq_quantize_act(Hh, cfg, bh)         # input of down
                sdq.sdq_linear(hq, ps[6], Ya[0])
        flops = 2.0 * M * sum(n * k for n, k in shapes) * 32

        def entry(ms):
            return {"ms_per_model_pass": ms, "dense_equiv_TFLOPs": flops / ms / 1e9, "weight_GBps_algorithmic": algo / ms / 1e6,
                    "frac_of_hbm_peak": algo / ms / 1e6 / peaks["hbm"], "frac_of_mixed_tensor_peak": flops / ms / 1e9 / mixed_peak}
        e = entry(time_graph(lambda: model(False), reps=3 if M >= 1024 else 10))
        if M <= 16:
            e["grouped_qkv_and_gate_up"] = entry(time_graph(lambda: model(True), reps=10))
            e["grouped_with_fused_quantizer"] = entry(time_graph(lambda: model(True, True), reps=10))
        c5["M%d" % M] = e
        assert sdq.device_status() == 0
    return c5, layers


def run_sweep(args):
    """Extra measurements for the other configurations (not the contract line): the OPT-6.7B FFN with the outlier
    pattern swept, and all 224 linear layers of a 32-layer LLaMA-7B-shaped decoder back to back for a sweep of
    token counts (quantize_act where a new activation enters + sdq_linear, one CUDA graph per token count)."""
    import paper_2406_13868_b200 as sdq
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    peaks = measured_peaks()
    out = {"peaks": peaks}
    c4, (X, H, W1, W2, Y1, Y2) = measure_opt_ffn(sdq, dev, peaks)
    M = 4096
    # the same layers with one scale per 32 K (the literal block-32 MXFP4 wording), and without pruning (dense MXFP4
    # inliers, with 1:8 outliers and with none = a plain block-scaled 4-bit GEMM)
    for name, cfg in (("1:8, scale block 32", sdq.Config(1, sdq.GRAN_PAIR, 32, 0)),
                      ("1:8, dense inliers", sdq.Config(1, sdq.GRAN_DENSE, 32, 0)),
                      ("none, dense inliers", sdq.Config(0, sdq.GRAN_DENSE, 32, 0))):
        P1, P2 = sdq.sdq_decompose(W1, cfg), sdq.sdq_decompose(W2, cfg)
        xq, hq = sdq.sdq_quantize_act(X, cfg), sdq.sdq_quantize_act(H, cfg)
        t1 = time_graph(lambda: sdq.sdq_linear(xq, P1, Y1))
        t2 = time_graph(lambda: sdq.sdq_linear(hq, P2, Y2))
        fl = 2.0 * M * 4096 * 16384
        c4[name] = {"fc1_ms": t1, "fc1_TFLOPs": fl / t1 / 1e9, "fc2_ms": t2, "fc2_TFLOPs": fl / t2 / 1e9}
        del P1, P2, xq, hq
    out["opt67b_ffn_M4096_outlier_sweep"] = c4
    del X, H, W1, W2, Y1, Y2
    cfg = sdq.Config(1, sdq.GRAN_PAIR, 64, 0)
    shapes = [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)]
    c5, layers = measure_model(sdq, dev, peaks)
    algo = c5["algorithmic_weight_bytes"]
    out["llama7b_32_layers_224_linears"] = c5
    del layers
    # ---- the same model with q, k, v packed as one 12288-row matrix and gate, up as one 22016-row matrix (the usual
    # fused projections: the rows of a linear layer are independent, so concatenating weight matrices that read the
    # same activations changes no output): 4 GEMMs + 4 quantizer launches per layer
    fshapes = [(12288, 4096), (4096, 4096), (22016, 4096), (4096, 11008)]
    flayers = []
    for l in range(32):
        ps = []
        for i, (N, K) in enumerate(fshapes):
            W = sdq_synth.make_weight(N, K, 7000 + 10 * l + i, device="cuda")
            ps.append(sdq.sdq_decompose(W, cfg))
            del W
        flayers.append(ps)
    c6 = {}
    for M in (1, 16, 128, 1024):
        X = sdq_synth.make_act(M, 4096, 5500 + M, n_outlier_channels=41, device="cuda")
        Hh = sdq_synth.make_act(M, 11008, 5600 + M, n_outlier_channels=110, device="cuda")
        bx = torch.empty(sdq.act_size(M, 4096, cfg), dtype=torch.uint8, device=dev)
        bh = torch.empty(sdq.act_size(M, 11008, cfg), dtype=torch.uint8, device=dev)
        Ys = [torch.empty((M, n), dtype=torch.bfloat16, device=dev) for n, _ in fshapes]

        def fmodel():
            for ps in flayers:
                sdq.sdq_linear(sdq.sdq_quantize_act(X, cfg, bx), ps[0], Ys[0])     # q, k, v
                sdq.sdq_linear(sdq.sdq_quantize_act(X, cfg, bx), ps[1], Ys[1])     # o
                sdq.sdq_linear(sdq.sdq_quantize_act(X, cfg, bx), ps[2], Ys[2])     # gate, up
                sdq.sdq_linear(sdq.sdq_quantize_act(Hh, cfg, bh), ps[3], Ys[3])    # down
        ms = time_graph(fmodel, reps=3 if M >= 1024 else 10)
        flops = 2.0 * M * sum(n * k for n, k in fshapes) * 32
        c6["M%d" % M] = {"ms_per_model_pass": ms, "dense_equiv_TFLOPs": flops / ms / 1e9, "weight_GBps_algorithmic": algo / ms / 1e6,
                         "frac_of_hbm_peak": algo / ms / 1e6 / peaks["hbm"]}
    out["llama7b_32_layers_fused_qkv_gate_up_128_linears"] = c6
    del flayers
    # ---- output error of every configuration against the unquantized product on the synthetic layer (a proxy only:
    # the paper's quality numbers are perplexities of real models): ||Y - X W^T|| / ||X W^T||, fp64 reference on the GPU
    M, K, N = 512, 4096, 4096
    X = sdq_synth.make_act(M, K, 6001, device="cuda")
    W = sdq_synth.make_weight(N, K, 6002, device="cuda")
    ref = X.double() @ W.double().T
    err = {}
    for name, cfg in (("4:8 pair-wise, no outliers", sdq.Config(0, sdq.GRAN_PAIR, 64, 0)),
                      ("4:8 pair-wise + 1:8", sdq.Config(1, sdq.GRAN_PAIR, 64, 0)),
                      ("4:8 pair-wise + 2:8", sdq.Config(2, sdq.GRAN_PAIR, 64, 0)),
                      ("4:8 pair-wise + 1:8, scale per 32", sdq.Config(1, sdq.GRAN_PAIR, 32, 0)),
                      ("4:8 pair-wise + 1:8, E4M3 scales per 32", sdq.Config(1, sdq.GRAN_PAIR, 32, sdq.SCALE_UE4M3)),
                      ("2:4 element-wise + 1:8, scale per 32 (literal wording)", sdq.Config(1, sdq.GRAN_ELEM, 32, 0)),
                      ("6:8 = 2:8 + 4:8 at any position", sdq.Config(2, sdq.gran_keep(6), 32, 0)),
                      ("7:8 = 1:8 + 6:8", sdq.Config(1, sdq.gran_keep(7), 32, 0)),
                      ("3:4 = 1:4 + 2:4 (S-Vectors of 4)", sdq.Config(2, sdq.GRAN_3OF4, 32, 0)),
                      ("8:8 = 1:8 + 7:8", sdq.Config(1, sdq.GRAN_DENSE, 32, 0)),
                      ("8:8 dense 4-bit, no outliers", sdq.Config(0, sdq.GRAN_DENSE, 32, 0))):
        Y = sdq.sdq_linear(sdq.sdq_quantize_act(X, cfg), sdq.sdq_decompose(W, cfg), f32=True)
        err[name] = float((Y.double() - ref).norm() / ref.norm())
    out["relative_output_error_M512_4096x4096"] = err
    assert sdq.device_status() == 0
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--sweep", action="store_true", help="measure the other configurations (OPT FFN outlier sweep, whole-model pass) and exit")
    ap.add_argument("--case", default=None, choices=["gemm_prefill", "gemm_prefill_b32", "gemm_prefill_e4m3", "gemm_prefill_dense", "gemm_prefill_mxfp4", "gemm_decode", "group_decode", "quant",
                             "pack"],
                    help="run only a small single-kernel case (for profiler captures) and exit")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--stub-body", action="store_true", help="(tests) run only the rank plumbing, on CPU, with a fixed fake duration")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not (args.sweep or args.case):
        sys.exit(spawn_ranks(args))       # no launcher around us: become one
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.sweep:
        run_sweep(args)
    elif args.case:
        run_case(args)
    elif args.stub_body:
        run_stub(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
