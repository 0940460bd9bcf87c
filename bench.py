#!/usr/bin/env python
"""Benchmark of the SIMD-structured sparse 1x1 convolution stack on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl alcs|reference] [--workload NAME]

One "step" = one pass of the whole hot path (every pointwise layer of the stack, bias + ReLU
fused) over one synthetic batch.  The default workload is the batch-64 MobileNetV1-224 pointwise
stack (fp32, g = 4, per-layer block sparsity drawn from U[0.6, 0.9]); `--workload mbv1_b1` runs the
batch-1 stack through a CUDA graph.  Prints ONE JSON line (rank 0).

`--impl reference` times the CPU oracle, as it stands, on the host cores, on a bounded sample
(a few images) of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from alcs_workloads import config_layers, make_bias, make_mask, make_weights, make_x, with_batch  # noqa: E402

METRIC = "nonzero-GFLOP/s & % of roofline, SIMD-sparse 1x1 conv stack, 1 B200, b=1/64"
UNIT = "GFLOP/s"
WORKLOADS = {"mbv1_b64": 2, "mbv1_b1": 1, "c1": 0, "rn50_b32": 3, "sweep_b256": 4}
SM_COUNT, FP32_LANES = 148, 128


def peaks():
    """Roofline denominators: measured HBM copy bandwidth if the driver wrote it, else the
    pool's fallback figure; fp32 CUDA-core peak derived from unit counts and the maximum clock."""
    hbm, src, mhz = 6650.0, "fallback", 1965.0
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            hbm, src = float(d["hbm_gbs"]), "measured"
            mhz = float(d.get("sm_max_mhz", mhz))
        except Exception:
            pass
    fp32_tflops = SM_COUNT * FP32_LANES * 2 * mhz * 1e6 / 1e12
    return hbm, src, fp32_tflops, mhz


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0=None, t1=None):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        for ts, line in self.lines:
            if t0 is not None and not (t0 - 0.05 <= ts <= t1 + 0.15):
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx = float(f[1])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm)}


def layer_stats(spec, nb):
    """Algorithmic work of one layer: nonzero FLOPs and bytes (X, Y, packed W, bias moved once)."""
    elt = 4 if spec.dtype == "f32" else 2
    q = spec.n * spec.hw
    flops = 2.0 * nb * spec.g * q
    packed = nb * (spec.g * elt + 4) + (spec.rows + 1) * 4
    byts = packed + q * spec.cin * elt + q * spec.cout * elt + 4 * spec.cout
    return flops, byts


def oracle_sample(specs, target_s=12.0):
    """Time the oracle, as it stands, on a bounded sample of the workload: the first `b` images of
    every layer, repeated until about target_s seconds of CPU work have been timed.
    Returns (nonzero GFLOP/s, threads, description, seconds)."""
    import oracle
    arrs = [(make_weights(s), make_mask(s), make_bias(s)) for s in specs]

    def run(b, xs=None):
        t = nz = 0.0
        for i, (s, (W, M, bias)) in enumerate(zip(specs, arrs)):
            sb = with_batch(s, min(b, s.n))
            X = xs[i] if xs is not None else make_x(sb)
            t0 = time.perf_counter()
            oracle.conv1x1(W, M, X, bias, s.relu, s.g)
            t += time.perf_counter() - t0
            nz += layer_stats(sb, int(M.sum()))[0]
        return t, nz

    t1, _ = run(1)
    b = int(max(1, min(specs[0].n, target_s / max(t1, 1e-3))))
    xs = [make_x(with_batch(s, min(b, s.n))) for s in specs]
    t, nz, passes = 0.0, 0.0, 0
    while t < target_s and passes < 50:
        dt, dnz = run(b, xs)
        t, nz, passes = t + dt, nz + dnz, passes + 1
    text = f"first {min(b, specs[0].n)} of {specs[0].n} images of every layer, {passes} pass(es)"
    return nz / t / 1e9, oracle.num_threads(), text, t


def kernel_source_hash():
    """Hash of the CUDA sources; stored DRAM-traffic counters are only quoted while it matches."""
    import hashlib
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2109_00170_b200", "csrc")
    for f in sorted(os.listdir(d)):
        if f.startswith(("alcs_conv2d", "alcs_project")):
            continue        # other entry points: they do not change the pointwise kernels
        h.update(open(os.path.join(d, f), "rb").read())
    return h.hexdigest()[:16]


def stored_traffic(layer_name, cfg):
    """DRAM bytes per launch of this layer's kernel from the committed ncu capture, or None if the
    kernel sources or the launch configuration have changed since it was taken."""
    p = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        d = json.load(open(p))
        if d.get("source_hash") != kernel_source_hash():
            return None
        e = d["layers"].get(layer_name)
        if e and e.get("cfg") == cfg:
            return e["dram_bytes"]
    except Exception:
        pass
    return None


def run_reference(args, specs, wl):
    """The oracle as the reference arm: each step is one pass over a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    arrs = [(make_weights(s), make_mask(s), make_bias(s)) for s in specs]
    b = 1 if specs[0].n > 1 else 1
    sub = [with_batch(s, min(b, s.n)) for s in specs]
    xs = [make_x(s) for s in sub]
    nz = sum(layer_stats(s, int(a[1].sum()))[0] for s, a in zip(sub, arrs))

    def step():
        for s, (W, M, bias), X in zip(sub, arrs, xs):
            oracle.conv1x1(W, M, X, bias, s.relu, s.g)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    val = nz / dt / 1e9
    sample = f"{b} of {specs[0].n} images of every layer per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl, "layers": len(specs), "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def rank_env():
    """(rank, world size, local rank) as torchrun exports them; a plain run is rank 0 of 1."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def max_over_ranks(ms, world, device=None):
    """The slowest rank's time: what a multi-GPU step costs.  No-op for one rank."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gflops(flops_per_rank, world, ms_per_step):
    """Weak scaling: every rank runs its own batch (replicas, no exchange), so the job's
    throughput is the ranks' work added up over the slowest rank's time."""
    return world * flops_per_rank / (ms_per_step * 1e-3) / 1e9


def measure_batch1(A, torch, dev, stream, steps, hbm_gbs, fp32_tf):
    """The same stack at batch 1 (the paper's latency setting), replayed as one CUDA graph.  A layer's
    roofline time is below a microsecond there, so the run is launch- and latency-bound; reported
    warm (working set resident in L2) and cold (a buffer larger than L2 rewritten before each step)."""
    specs = config_layers(WORKLOADS["mbv1_b1"])
    layers, flops, t_roof = [], 0.0, 0.0
    for s in specs:
        W, M, X, b = make_weights(s), make_mask(s), make_x(s), make_bias(s)
        p = A.alcs_packed_upload(A.alcs_pack(W, M, s.g), dev.index)
        xd = torch.from_numpy(X).to(dev)
        yd = torch.empty((s.n, s.cout, s.hw), dtype=torch.float32, device=dev)
        bd = torch.from_numpy(b).to(dev)
        with torch.cuda.stream(stream):
            A.alcs_spconv1x1_tune(p, xd, yd, s.n, s.h, s.w, bd, A.ALCS_RELU, stream)
        layers.append(dict(w=p, x=xd, y=yd, n=s.n, h=s.h, wd=s.w, bias=bd, flags=A.ALCS_RELU))
        fl, by = layer_stats(s, int(M.sum()))
        flops += fl
        t_roof += max(fl / (fp32_tf * 1e12), by / (hbm_gbs * 1e9))
    stack = A.alcs_stack_create(layers, A.ALCS_STACK_GRAPH)
    with torch.cuda.stream(stream):
        A.alcs_stack_tune(stack, 0, stream)
    for _ in range(5):
        A.alcs_stack_run(stack, stream)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        A.alcs_stack_run(stack, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    warm_us = e0.elapsed_time(e1) * 1e3 / steps
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    cold = []
    with torch.cuda.stream(stream):
        for k in range(min(steps, 30)):
            flush.fill_(k & 1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            A.alcs_stack_run(stack, stream)
            b.record(stream)
            cold.append((a, b))
    torch.cuda.synchronize()
    cold_us = statistics.mean(a.elapsed_time(b) for a, b in cold) * 1e3
    A.alcs_stack_destroy(stack)
    return {"workload": "mbv1_b1", "layers": len(specs), "cuda_graph": True, "nz_mflop_per_step": round(flops / 1e6, 1),
            "sum_t_roof_us": round(t_roof * 1e6, 2),
            "warm": {"us_per_step": round(warm_us, 2), "us_per_layer": round(warm_us / len(specs), 2),
                     "nz_gflops": round(flops / warm_us / 1e3, 1), "frac": round(t_roof * 1e6 / warm_us, 4)},
            "cold": {"us_per_step": round(cold_us, 2), "us_per_layer": round(cold_us / len(specs), 2),
                     "nz_gflops": round(flops / cold_us / 1e3, 1), "frac": round(t_roof * 1e6 / cold_us, 4)}}


def bench_loop_ceiling(args):
    """What bounds the hot loop, measured on this GPU with the library's probes: the fp32 FMA rate
    from registers, the cost of shared-memory loads, and the kernel's own segment loop running on
    data that is already in shared memory (no staging, barriers or stores)."""
    import torch
    import paper_2109_00170_b200 as A
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    A.lib()
    st = torch.cuda.current_stream()
    sampler = ClockSampler(0)
    sampler.start()
    out = {"metric": "fraction of the fp32 CUDA-core peak reached by the segment loop on shared-memory-resident data",
           "unit": "fraction", "n_gpus": 1, "data": "synthetic", "dtype": "f32", "higher_is_better": True,
           "config": {"workload": "loop_ceiling"}}
    out["fma_peak"] = {"scalar": A.alcs_probe_fma_peak(False, st), "packed": A.alcs_probe_fma_peak(True, st)}
    out["lds_cycles_per_warp_instruction"] = {
        f"{8 * b}-bit {'uniform' if u else 'distinct'}": round(A.alcs_probe_lds(b, u, st), 3)
        for b in (16, 8, 4) for u in (False, True)}
    loops = []
    for g, p, rw, nw, deep in [(4, 8, 2, 16, False), (4, 8, 2, 16, True), (4, 8, 2, 12, False), (4, 8, 2, 12, True),
                               (4, 8, 2, 8, True), (4, 8, 1, 16, False), (4, 16, 1, 16, False), (4, 16, 1, 12, True),
                               (4, 4, 4, 16, False), (1, 8, 2, 16, False), (8, 4, 2, 16, False), (16, 4, 1, 16, False)]:
        row = {"g": g, "pixels_per_lane": p, "rows_per_warp": rw, "warps": nw, "deep": deep, "frac_by_pairs_per_segment": {}}
        for L in (1, 2, 3, 4, 8, 32):
            r = A.alcs_probe_segment_loop(g, p, rw, nw, deep, L, st)
            row["frac_by_pairs_per_segment"][str(L)] = round(r["frac_of_fp32_peak"], 4)
            row["registers"], row["spill_bytes"] = r["registers"], r["spill_bytes"]
        loops.append(row)
    out["segment_loop"] = loops
    out["value"] = max(r["frac_by_pairs_per_segment"]["32"] for r in loops if r["g"] == 4 and r["pixels_per_lane"] == 8)
    out["clocks"] = sampler.stop()
    print(json.dumps(out))


def bench_latency_model(args):
    """`--workload latency_model`: the paper's Section 3.3 experiment on this GPU.  (1) For every layer
    of the batch-64 MobileNetV1 pointwise stack, time the sparse kernel at 11 densities (0, 0.1, ..., 1
    of the blocks kept): the (k_i, t_i) pairs of the interpolation.  (2) Draw random per-layer
    densities, time the real layers, compare with the interpolated estimate.  (3) Project the stack's
    weights onto a latency budget with alcs_project_bisection (Algorithm 1), pack the result, time it."""
    import torch
    from dataclasses import replace
    import paper_2109_00170_b200 as A
    from alcs_workloads import rng, uniform_block_mask
    specs = config_layers(2)
    if args.layers:
        specs = [specs[int(i)] for i in args.layers.split(",")]
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    A.lib()
    stream = torch.cuda.current_stream()
    reps = 20
    W = [make_weights(s) for s in specs]
    bias = [torch.from_numpy(make_bias(s)).to(dev) for s in specs]
    X = [torch.from_numpy(make_x(s)).to(dev) for s in specs]
    Y = [torch.empty((s.n, s.cout, s.hw), device=dev) for s in specs]

    def time_layer(i, mask):
        s = specs[i]
        p = A.alcs_packed_upload(A.alcs_pack(W[i], mask, s.g), 0)
        run = lambda: A.alcs_spconv1x1(p, X[i], Y[i], s.n, s.h, s.w, bias[i], A.ALCS_RELU, stream)
        for _ in range(3):
            run()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            run()
        e1.record(stream)
        e1.synchronize()
        A.alcs_packed_free(p)
        return e0.elapsed_time(e1) * 1e3 / reps          # us

    sampler = ClockSampler(0)
    sampler.start()
    t_start = time.time()
    tables = []
    for i, s in enumerate(specs):
        blocks = s.rows * s.cin
        k, t = [], []
        for j in range(11):
            m = uniform_block_mask(s.rows, s.cin, 1.0 - j / 10.0, s.seed + 50 + j)
            k.append(int(m.sum()) * s.g)
            t.append(time_layer(i, m))
        tables.append((k, t))
    # (2) random density settings, real against estimated
    trials, errs, rows = 20, [], []
    for tr in range(trials):
        u = rng.uniform01_f64(BASE_TRIAL_SEED + tr, 3, len(specs))
        real, nz = 0.0, []
        for i, s in enumerate(specs):
            m = uniform_block_mask(s.rows, s.cin, float(0.05 + 0.9 * u[i]), s.seed + 500 + tr)
            nz.append(int(m.sum()) * s.g)
            real += time_layer(i, m)
        est = A.alcs_network_latency(0.0, tables, nz)
        errs.append(abs(est - real) / real)
        rows.append({"real_us": round(real, 1), "estimated_us": round(est, 1)})
    # (3) projection of the stack's weights onto 50 % of the dense latency
    dense_t = A.alcs_network_latency(0.0, tables, [k[-1] for k, _ in tables])
    empty_t = A.alcs_network_latency(0.0, tables, [0] * len(specs))
    budget = empty_t + 0.5 * (dense_t - empty_t)
    eps = 0.002 * (dense_t - empty_t)
    ud = [torch.from_numpy(w).to(dev) for w in W]
    total = sum(s.rows * s.cin for s in specs)
    mask_d = torch.empty((total,), dtype=torch.uint8, device=dev)
    A.alcs_project_bisection(ud, specs[0].g, tables, 0.0, budget, eps, mask_d, None, stream)      # warm-up
    proj_ms = 1e30
    for _ in range(5):              # host wall clock of the whole call (it synchronises); best of five
        c0 = time.perf_counter()
        pr = A.alcs_project_bisection(ud, specs[0].g, tables, 0.0, budget, eps, mask_d, None, stream)
        proj_ms = min(proj_ms, (time.perf_counter() - c0) * 1e3)
    mask_h = mask_d.cpu().numpy()
    real, off = 0.0, 0
    for i, s in enumerate(specs):
        m = mask_h[off:off + s.rows * s.cin].reshape(s.rows, s.cin)
        off += s.rows * s.cin
        real += time_layer(i, m)
    clocks = sampler.stop(t_start, time.time())
    out = {"metric": "latency model: relative error of the interpolated stack latency; projection with bisection",
           "value": statistics.mean(errs), "unit": "mean |estimated - real| / real", "n_gpus": 1, "steps": trials,
           "warmup": 3, "higher_is_better": False, "dtype": "f32", "data": "synthetic",
           "config": {"workload": "latency_model", "stack": "mbv1_b64", "layers": len(specs), "knots": 11,
                      "runs_per_point": reps, "launch_cfgs": "planner defaults (no per-mask tuning)"},
           "estimation": {"trials": trials, "mean_rel_err": statistics.mean(errs), "max_rel_err": max(errs), "pairs": rows},
           "tables_us": [{"layer": s.name, "t": [round(x, 2) for x in t]} for s, (_, t) in zip(specs, tables)],
           "projection": {"groups": pr["n_groups"], "kept": pr["n_keep"], "iters": pr["iters"], "call_ms": round(proj_ms, 3),
                          "budget_us": round(budget, 1), "model_latency_us": round(pr["latency"], 1),
                          "measured_us": round(real, 1), "dense_model_us": round(dense_t, 1),
                          "kept_fraction_per_layer": [round(kp / (s.rows * s.cin), 3)
                                                      for kp, s in zip(pr["kept_per_layer"], specs)]},
           "clocks": clocks}
    print(json.dumps(out))


BASE_TRIAL_SEED = 2109001


def bench_conv2d(args):
    """`--workload rn18_3x3_b32`: ResNet-18's 3x3 convolutions (stride 1 and 2, pad 1) through
    alcs_spconv2d, one launch per layer on one stream; per-layer CUDA-event times, roofline as for
    the pointwise layers (kept-block FLOPs at the fp32 peak against X, packed W and Y moved once)."""
    import torch
    import oracle
    import paper_2109_00170_b200 as A
    from alcs_workloads import make_bias2d, make_mask2d, make_weights2d, make_x2d, resnet18_3x3_stack
    from dataclasses import replace
    specs = resnet18_3x3_stack(32)
    if args.layers:
        specs = [specs[int(i)] for i in args.layers.split(",")]
    hbm_gbs, peak_src, fp32_tf, _ = peaks()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    A.lib()
    stream = torch.cuda.current_stream()
    L = []
    for s in specs:
        W, M, b = make_weights2d(s), make_mask2d(s), make_bias2d(s)
        p = A.alcs_packed_upload(A.alcs_pack(W.reshape(s.cout, s.k), M, s.g), 0)
        xd = torch.from_numpy(make_x2d(s)).to(dev)
        yd = torch.empty((s.n, s.cout, s.oh, s.ow), device=dev)
        nb = int(M.sum())
        flops = 2.0 * nb * s.g * s.n * s.oh * s.ow
        byts = nb * (s.g * 4 + 4) + (s.rows + 1) * 4 + 4 * (xd.numel() + yd.numel()) + 4 * s.cout
        L.append(dict(spec=s, W=W, M=M, b=b, p=p, x=xd, y=yd, bd=torch.from_numpy(b).to(dev), nb=nb, flops=flops,
                      bytes=byts, t_roof=max(flops / (fp32_tf * 1e12), byts / (hbm_gbs * 1e9)),
                      bound="alu" if flops / (fp32_tf * 1e12) >= byts / (hbm_gbs * 1e9) else "hbm"))

    def run_layer(l):
        s = l["spec"]
        A.alcs_spconv2d(l["p"], l["x"], l["y"], s.n, s.cin, s.h, s.w, s.kh, s.kw, s.stride, s.pad, l["bd"],
                        A.ALCS_RELU if s.relu else 0, stream)

    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # larger than L2
    for _ in range(max(args.warmup, 3)):
        for l in L:
            run_layer(l)
    torch.cuda.synchronize()
    steps = min(args.steps, 50)
    sampler = ClockSampler(0)
    sampler.start()
    t0 = time.time()
    times = [[] for _ in L]
    for _ in range(steps):
        for i, l in enumerate(L):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            run_layer(l)
            e1.record(stream)
            e1.synchronize()
            times[i].append(e0.elapsed_time(e1) * 1e3)
    clocks = sampler.stop(t0, time.time())
    rows, tot_us, tot_flops, tot_roof = [], 0.0, 0.0, 0.0
    for l, ts in zip(L, times):
        s, us = l["spec"], statistics.mean(ts)
        tot_us += us; tot_flops += l["flops"]; tot_roof += l["t_roof"] * 1e6
        rows.append({"layer": s.name, "sparsity": s.sparsity, "kept_blocks": l["nb"], "nz_mflop": round(l["flops"] / 1e6, 1),
                     "mbytes": round(l["bytes"] / 1e6, 2), "t_roof_us": round(l["t_roof"] * 1e6, 2), "bound": l["bound"],
                     "us": round(us, 2), "us_min": round(min(ts), 2), "nz_gflops": round(l["flops"] / us / 1e3, 1),
                     "frac": round(l["t_roof"] * 1e6 / us, 4),
                     "cfg": A.alcs_spconv2d_plan(l["p"], s.n, s.cin, s.h, s.w, s.kh, s.kw, s.stride, s.pad)})
    dom = max(range(len(L)), key=lambda i: statistics.mean(times[i]))
    dl, dus = L[dom], statistics.mean(times[dom])
    if dl["bound"] == "alu":
        roof = {"bound": "alu", "achieved": dl["flops"] / dus / 1e6, "peak": fp32_tf, "unit": "TFLOP/s"}
    else:
        roof = {"bound": "hbm", "achieved": dl["bytes"] / dus / 1e3, "peak": hbm_gbs, "unit": "GB/s"}
    roof.update({"frac": roof["achieved"] / roof["peak"], "traffic": None, "kernel": "spconv2d_kernel",
                 "layer": dl["spec"].name, "peak_source": f"HBM {peak_src}; fp32 = 148 SMs x 128 lanes x 2 x max SM clock"})
    out = {"metric": "nonzero-GFLOP/s & % of roofline, SIMD-sparse 3x3 conv layers (ResNet-18), 1 B200, b=32",
           "value": tot_flops / tot_us / 1e3, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": max(args.warmup, 3),
           "ms_per_step": tot_us / 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
           "data": "synthetic", "config": {"workload": "rn18_3x3_b32", "layers": len(L), "batch": 32, "g": 4,
                                           "cache": "L2 flushed (256 MB written) before every timed launch"},
           "roofline": roof, "stack_roofline": {"sum_t_roof_us": round(tot_roof, 1), "sum_layer_us": round(tot_us, 1),
                                                "frac": round(tot_roof / tot_us, 4)},
           "gpu_launches": steps * len(L), "clocks": clocks, "layers": rows}
    if not args.no_cpu_baseline:
        # the oracle as it stands on one image of every layer
        t = nz = 0.0
        for l in L:
            s1 = replace(l["spec"], n=1)
            X1 = make_x2d(s1)
            c0 = time.perf_counter()
            oracle.conv2d(l["W"], l["M"], X1, l["b"], s1.relu, s1.g, s1.stride, s1.pad)
            t += time.perf_counter() - c0
            nz += l["flops"] / l["spec"].n
        out["cpu_baseline"] = {"value": nz / t / 1e9, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                               "sample": "1 of 32 images of every layer, one pass", "seconds": round(t, 2)}
    print(json.dumps(out))


def kernels_per_layer(spec, cfg):
    """Kernel launches one layer costs: the convolution kernel, plus the pass that repacks X when its rows
    are not 16-byte multiples (unless they are staged as they are, copy_mode 3) or that makes the
    tile-major copy (copy_mode 4).  The small-problem kernel (math_mode 3) never repacks."""
    if cfg.get("math_mode") == 3:
        return 1
    row_bytes = spec.hw * (4 if spec.dtype == "f32" else 2)
    cm = cfg.get("copy_mode")
    if cm == 4:
        return 2
    if row_bytes % 16 == 0 or (cm == 3 and row_bytes % 16 == 8):
        return 1
    return 2


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="alcs", choices=["alcs", "reference"])
    ap.add_argument("--workload", default="mbv1_b64", choices=sorted(WORKLOADS) + ["rn18_3x3_b32", "latency_model", "loop_ceiling"])
    ap.add_argument("--no-tune", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-batch1", action="store_true", help="skip the batch-1 (CUDA graph) measurement")
    ap.add_argument("--retune", action="store_true",
                    help="time the candidate launch configurations again and rewrite the tuning cache "
                         "(default: reuse paper_2109_00170_b200/tuned/<workload>.json while the kernel sources match)")
    ap.add_argument("--layers", default="", help="comma-separated layer indices (default: all)")
    ap.add_argument("--cfg", default="", help="force one launch configuration for every layer: "
                    "pixels_per_lane,rows_per_warp,warps,chunk_channels,stages,row_groups,min_blocks[,copy_mode]")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "alcs" else args.warmup
    wl = args.workload
    if wl in ("rn18_3x3_b32", "latency_model", "loop_ceiling"):
        if args.impl == "reference" or int(os.environ.get("WORLD_SIZE", "1")) > 1:
            raise SystemExit(f"{wl} is a single-GPU side workload of --impl alcs")
        if wl == "loop_ceiling":
            return bench_loop_ceiling(args)
        return bench_conv2d(args) if wl == "rn18_3x3_b32" else bench_latency_model(args)
    specs = config_layers(WORKLOADS[wl])
    if args.layers:
        specs = [specs[int(i)] for i in args.layers.split(",")]

    if args.impl == "reference":
        return run_reference(args, specs, wl)

    import torch
    import torch.distributed as dist
    import paper_2109_00170_b200 as A

    rank, world, local = rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    A.lib()
    stream = torch.cuda.Stream()
    graph = wl in ("mbv1_b1", "c1")

    # ---- set-up (untimed): inputs, packing, upload, tuning -----------------------------------
    layers, keep, stats = [], [], []
    host = []
    cache_path = os.path.join(ROOT, "paper_2109_00170_b200", "tuned", wl + ".json")
    cache, tuned_now = {}, {}
    if not args.retune and not args.no_tune and os.path.exists(cache_path):
        try:
            c = json.load(open(cache_path))
            if c.get("source_hash") == kernel_source_hash():
                cache = c["layers"]
        except Exception:
            cache = {}
    for s in specs:
        W, M, X, b = make_weights(s), make_mask(s), make_x(s), make_bias(s)
        p = A.alcs_packed_upload(A.alcs_pack(W, M, s.g), local)
        xd = torch.from_numpy(X).to(dev)
        ydt = torch.float32 if s.dtype == "f32" else torch.float16
        yd = torch.empty((s.n, s.cout, s.hw), dtype=ydt, device=dev)
        bd = torch.from_numpy(b).to(dev)
        flags = A.ALCS_RELU if s.relu else 0
        forced = None
        if args.cfg:
            keys = ("pixels_per_lane", "rows_per_warp", "warps", "chunk_channels", "stages", "row_groups", "min_blocks", "copy_mode", "producer_warps", "math_mode", "consumer_groups", "split_rows")
            forced = dict(zip(keys, (int(v) for v in args.cfg.split(","))))
            cfg = forced
        elif s.name in cache:       # a configuration tuned earlier for these kernel sources
            cfg = cache[s.name]
            A.alcs_spconv1x1_set_cfg(p, s.n, s.h, s.w, flags, cfg)
        else:
            with torch.cuda.stream(stream):
                cfg = (A.alcs_spconv1x1_plan(p, s.n, s.h, s.w, flags) if args.no_tune
                       else A.alcs_spconv1x1_tune(p, xd, yd, s.n, s.h, s.w, bd, flags, stream))
            if not args.no_tune:
                tuned_now[s.name] = cfg
        layers.append(dict(w=p, x=xd, y=yd, n=s.n, h=s.h, wd=s.w, bias=bd, flags=flags, cfg=forced))
        nb = int(M.sum())
        fl, by = layer_stats(s, nb)
        stats.append(dict(name=s.name, nb=nb, sparsity=1 - nb / M.size, flops=fl, bytes=by, cfg=cfg))
        host.append((X, b))
        keep.append((W, M))
    stack = None if args.cfg else A.alcs_stack_create(layers, A.ALCS_STACK_GRAPH if graph else 0)
    stack_tune_us = None
    if tuned_now and stack is not None:
        # second tuning step, in context: the layers' best few configurations are tried inside the
        # whole stack (dependent launches, the cache state the other layers leave behind)
        with torch.cuda.stream(stream):
            stack_tune_us = A.alcs_stack_tune(stack, 0, stream)
        for i, st_ in enumerate(stats):
            if st_["name"] in tuned_now:
                st_["cfg"] = tuned_now[st_["name"]] = A.alcs_stack_layer_cfg(stack, i)
    if tuned_now and rank == 0 and not args.layers:
        try:
            os.makedirs(os.path.dirname(cache_path), exist_ok=True)
            json.dump({"source_hash": kernel_source_hash(), "layers": {**cache, **tuned_now}}, open(cache_path, "w"), indent=1)
        except OSError:
            pass

    def run_stack():
        if stack is not None:
            A.alcs_stack_run(stack, stream)
        else:       # forced configuration: one explicit call per layer
            for L in layers:
                A.alcs_spconv1x1(L["w"], L["x"], L["y"], L["n"], L["h"], L["wd"], L["bias"], L["flags"], stream, L["cfg"])
    total_flops = sum(st["flops"] for st in stats)
    total_bytes = sum(st["bytes"] for st in stats)
    hbm_gbs, peak_src, fp32_tf, sm_max = peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- region A: K whole-stack steps, nothing between the launches ------------------------
    for _ in range(args.warmup):
        run_stack()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    tw0 = time.time()
    torch.cuda.nvtx.range_push("alcs_timed")      # lets a profiler select the timed launches
    e0.record(stream)
    for _ in range(args.steps):
        run_stack()
    e1.record(stream)
    barrier()
    torch.cuda.nvtx.range_pop()
    ms_total = e0.elapsed_time(e1)

    # ---- region B: the same steps with an event between layers (per-layer durations) --------
    nl = len(layers)
    # (one untimed pass through the per-layer entry point first: a packed matrix allocates its own repacking
    # scratch on its first such call, the stack above used the stack's)
    for L in layers:
        A.alcs_spconv1x1(L["w"], L["x"], L["y"], L["n"], L["h"], L["wd"], L["bias"], L["flags"], stream, L["cfg"])
    torch.cuda.synchronize()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(nl + 1)] for _ in range(args.steps)]
    for k in range(args.steps):
        evs[k][0].record(stream)
        for i, L in enumerate(layers):
            A.alcs_spconv1x1(L["w"], L["x"], L["y"], L["n"], L["h"], L["wd"], L["bias"], L["flags"], stream, L["cfg"])
            evs[k][i + 1].record(stream)
    barrier()
    tw1 = time.time()
    clocks = sampler.stop(tw0, tw1) if rank == 0 else None
    per_layer_ms = [statistics.mean(evs[k][i].elapsed_time(evs[k][i + 1]) for k in range(args.steps)) for i in range(nl)]
    per_layer_min = [min(evs[k][i].elapsed_time(evs[k][i + 1]) for k in range(args.steps)) for i in range(nl)]
    per_layer_med = [statistics.median(evs[k][i].elapsed_time(evs[k][i + 1]) for k in range(args.steps)) for i in range(nl)]
    per_layer_max = [max(evs[k][i].elapsed_time(evs[k][i + 1]) for k in range(args.steps)) for i in range(nl)]

    ms_total = max_over_ranks(ms_total, world, dev)
    ms_step = ms_total / args.steps
    value = whole_job_gflops(total_flops, world, ms_step)

    # ---- end to end: host buffers through alcs_spconv1x1_host, copies inside the timed region --
    e2e = None
    if args.e2e_steps > 0:
        ws_bytes = max(A.alcs_spconv1x1_host_workspace(L["w"], L["n"], L["h"], L["wd"], L["flags"]) for L in layers)
        # three streams with a workspace each take the layers in turn, so that the upload of one layer's
        # input overlaps the download of earlier layers' outputs (the bus is full duplex); the steps follow
        # each other without a join in between, as a serving loop would issue them
        NS = 3
        ws2 = [torch.empty(ws_bytes, dtype=torch.uint8, device=dev) for _ in range(NS)]
        st2 = [torch.cuda.Stream() for _ in range(NS)]
        xh = [torch.from_numpy(X).pin_memory() for X, _ in host]
        bh = [torch.from_numpy(b).pin_memory() for _, b in host]
        yh = [torch.empty(tuple(L["y"].shape), dtype=L["y"].dtype).pin_memory() for L in layers]
        h2d = sum(x.numel() * x.element_size() for x in xh) + sum(b.numel() * 4 for b in bh)
        d2h = sum(y.numel() * y.element_size() for y in yh)

        def e2e_steps(n_steps):
            start = torch.cuda.Event()
            start.record(stream)
            for s_ in st2:
                s_.wait_event(start)
            k = 0
            for _ in range(n_steps):
                for L, x, y, b in zip(layers, xh, yh, bh):
                    A.alcs_spconv1x1_host(L["w"], x, y, L["n"], L["h"], L["wd"], b, L["flags"], ws2[k % NS], ws_bytes, st2[k % NS])
                    k += 1
            for s_ in st2:
                done = torch.cuda.Event()
                done.record(s_)
                stream.wait_event(done)

        e2e_steps(1)
        barrier()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        e2e_steps(args.e2e_steps)
        f1.record(stream)
        barrier()
        ms_e2e = f0.elapsed_time(f1)
        ms_e2e = max_over_ranks(ms_e2e, world, dev) / args.e2e_steps
        e2e = {"value": whole_job_gflops(total_flops, world, ms_e2e), "unit": UNIT, "ms_per_step": ms_e2e,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": args.e2e_steps}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- per-layer roofline ------------------------------------------------------------------
    rows = []
    for st, ms, mn, md, mx in zip(stats, per_layer_ms, per_layer_min, per_layer_med, per_layer_max):
        t_hbm = st["bytes"] / (hbm_gbs * 1e9)
        t_alu = st["flops"] / (fp32_tf * 1e12)
        t_roof = max(t_hbm, t_alu)
        rows.append(dict(layer=st["name"], sparsity=round(st["sparsity"], 4), kept_blocks=st["nb"],
                         nz_mflop=round(st["flops"] / 1e6, 1), mbytes=round(st["bytes"] / 1e6, 2),
                         t_roof_us=round(t_roof * 1e6, 2), bound="hbm" if t_hbm >= t_alu else "alu",
                         us=round(ms * 1e3, 2), us_min=round(mn * 1e3, 2), us_median=round(md * 1e3, 2), us_max=round(mx * 1e3, 2),
                         nz_gflops=round(st["flops"] / (ms * 1e-3) / 1e9, 1),
                         frac=round(t_roof / (ms * 1e-3), 4), cfg=st["cfg"]))
    dom = max(range(nl), key=lambda i: per_layer_ms[i])
    d = rows[dom]
    if d["bound"] == "hbm":
        ach = stats[dom]["bytes"] / (per_layer_ms[dom] * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": hbm_gbs, "unit": "GB/s", "frac": ach / hbm_gbs}
    else:
        ach = stats[dom]["flops"] / (per_layer_ms[dom] * 1e-3) / 1e12
        roof = {"bound": "alu", "achieved": ach, "peak": fp32_tf, "unit": "TFLOP/s", "frac": ach / fp32_tf}
    roof.update({"traffic": stored_traffic(d["layer"], d["cfg"]), "kernel": "spconv1x1_mma_kernel" if d["cfg"].get("math_mode") == 2 else "spconv1x1_kernel", "layer": d["layer"],
                 "algorithmic_bytes": stats[dom]["bytes"], "algorithmic_flops": stats[dom]["flops"],
                 "peak_source": f"HBM {peak_src}; fp32 = {SM_COUNT} SMs x {FP32_LANES} lanes x 2 x {sm_max:.0f} MHz"})
    # the fp32 peak as this GPU delivers it from registers, measured now (a few hundred microseconds)
    with torch.cuda.stream(stream):
        pk = A.alcs_probe_fma_peak(True, stream)
    roof["peak_measured"] = {"value": round(pk["tflops"], 2), "unit": "TFLOP/s", "how": "fma.rn.f32x2 on register operands, 16 warps per SM",
                             "frac_of_derived": round(pk["frac_of_fp32_peak"], 4)}
    sum_roof = sum(r["t_roof_us"] for r in rows)
    sum_us = sum(r["us"] for r in rows)

    batch1 = None
    if wl == "mbv1_b64" and not args.no_batch1 and not args.layers and not args.cfg:
        batch1 = measure_batch1(A, torch, dev, stream, min(args.steps, 200), hbm_gbs, fp32_tf)

    cpu = None
    if not args.no_cpu_baseline:
        v, cores, sample, secs = oracle_sample(specs)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample, "seconds": round(secs, 2)}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32" if specs[0].dtype == "f32" else "f16", "data": "synthetic",
        "config": {"workload": wl, "layers": nl, "batch": specs[0].n, "g": specs[0].g,
                   "cache": "inputs larger than L2: one step touches %.0f MB of distinct X and Y" % (total_bytes / 1e6),
                   "cuda_graph": graph, "tuned": not args.no_tune,
                   "launch_cfgs": "forced" if args.cfg else ("tuning cache" if cache else ("tuned in this run" if not args.no_tune else "model")),
                   "stack_tune_us": [round(v, 2) for v in stack_tune_us] if stack_tune_us else None},
        "roofline": roof,
        "stack_roofline": {"sum_t_roof_us": round(sum_roof, 1), "sum_layer_us": round(sum_us, 1),
                           "frac": round(sum_roof / sum_us, 4), "min_layer_frac": min(r["frac"] for r in rows),
                           "step_frac": round(sum_roof / (ms_step * 1e3), 4),
                           "us_per_layer": round(ms_step * 1e3 / nl, 2)},
        "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": sum(kernels_per_layer(sp, st["cfg"]) for sp, st in zip(specs, stats)) * args.steps,
        "clocks": clocks,
        "batch1": batch1, "layers": rows,
    }
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
