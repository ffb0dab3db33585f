#!/usr/bin/env python
"""Benchmark of the block-punched CONV / block-based GEMM hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass of the hot path over one batch of the headline workload: the sweep point of
configs[4] with 16x16 blocks keeping 3 of 9 taps (3x3 CONV, 64x28x28x512 -> 512, bf16, fp32
accumulation), the largest single-call workload and a tensor-bound one.  The timed region is K
back-to-back steps replayed from CUDA graphs, rotating over buffer sets that together exceed the L2
cache, timed with CUDA events on the launching stream; a region shorter than about 50 ms is repeated
and the median is reported.  With N > 1 every rank is a replica working on its own batch (weak
scaling, no data-path collective) and the time is the max over ranks.  The JSON line also carries the
roofline of the kernel, an end-to-end number with host<->device copies in the timed region, the other
workloads (each with its own roofline block) and the CPU oracle timed on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

L2_BYTES = 126 * 1024 * 1024
GRAPH_CHUNK = 200
MIN_TIMED_MS = 50.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                 "hw_power_brake": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.01)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def conv_roofline(case, peaks, ms):
    flops = 2.0 * case.kept_macs()
    t_mma = flops / (peaks["bf16_tflops"] * 1e12)
    t_hbm = case.algorithmic_bytes() / (peaks["hbm_gbs"] * 1e9)
    t = ms * 1e-3
    return {"t_mma_us": t_mma * 1e6, "t_hbm_us": t_hbm * 1e6, "bound": "tensor" if t_mma >= t_hbm else "hbm",
            "frac": max(t_mma, t_hbm) / t}


class GraphTimer:
    """Captures runs of `step(i)` calls in CUDA graphs and times K of them with CUDA events."""

    def __init__(self, torch, step, n_sets):
        self.torch, self.step, self.n_sets = torch, step, n_sets
        self.graphs = {}

    def graph_for(self, n_steps, start):
        key = (n_steps, start % self.n_sets)
        if key not in self.graphs:
            torch = self.torch
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in range(n_steps):
                    self.step(start + i)
            self.graphs[key] = g
        return self.graphs[key]

    def plan(self, K):
        chunk = min(K, GRAPH_CHUNK)
        full, rest = divmod(K, chunk)
        g = self.graph_for(chunk, 0)
        plan = [g] * full
        if rest:
            plan.append(self.graph_for(rest, 0))
        return plan

    def time(self, K, W, barrier, agree_max=float):
        """W warm-up steps (eager, then through the graphs), every graph of the plan replayed once untimed,
        then the K-step region timed; a region under MIN_TIMED_MS is repeated and the median returned.
        Returns (ms of one K-step region, number of timed regions)."""
        torch = self.torch
        eager = min(W, 20)
        for i in range(eager):
            self.step(i)
        plan = self.plan(K)
        for g in dict.fromkeys(plan):        # each distinct graph once, untimed (first replays are slower)
            g.replay()
        done = eager + K
        while done < W:
            for g in plan:
                g.replay()
            done += K
        torch.cuda.synchronize()

        def region():
            barrier()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for g in plan:
                g.replay()
            e1.record()
            torch.cuda.synchronize()
            barrier()
            return e0.elapsed_time(e1)

        first = region()
        first_all = agree_max(first)         # every rank must run the same number of regions (they hold barriers)
        n = 1 if first_all >= MIN_TIMED_MS else int(min(200, max(3, np.ceil(MIN_TIMED_MS / max(first_all, 1e-3)))))
        times = [first] + [region() for _ in range(n - 1)]
        return float(np.median(times)), len(times)


# ------------------------------------------------------------------------------------------------
def make_conv_sets(torch, npas, case, n_sets):
    dev = torch.device("cuda")
    x0 = torch.from_numpy(case.x).to(dev).to(torch.bfloat16)
    w = torch.from_numpy(case.w).to(dev).to(torch.bfloat16)
    blob0 = npas.pack_bp(w, case.tap_mask, case.Mb, case.Nb)
    bias = torch.from_numpy(case.bias).to(dev) if case.bias is not None else None
    sets = []
    for i in range(n_sets):
        x = x0 if i == 0 else torch.roll(x0, shifts=i, dims=0).contiguous()
        blob = blob0 if i == 0 else npas.BpBlob(blob0.data.clone(), blob0.desc)
        y = torch.empty((case.N, case.P, case.Q, case.K), dtype=torch.bfloat16, device=dev)
        sets.append((x, blob, y))
    return sets, bias


def bench_conv(torch, npas, case, K, W, barrier, path=0, variant=0, agree_max=float):
    set_bytes = case.algorithmic_bytes()
    n_sets = max(2, -(-int(1.3 * L2_BYTES) // set_bytes))
    sets, bias = make_conv_sets(torch, npas, case, n_sets)
    # the workspace of the size the library asks for this layer (status words; room for the partial sums of a split
    # last round where the kept-pairs kernel runs)
    ws = npas.conv2d_bp_workspace(case.x.shape, sets[0][1], stride=case.stride, pad=case.pad, relu=case.relu,
                                  bias=bias is not None, path=path, variant=variant)

    def step(i):
        x, blob, y = sets[i % n_sets]
        npas.conv2d_bp(x, blob, bias, None, stride=case.stride, pad=case.pad, relu=case.relu, out=y, ws=ws, path=path,
                       variant=variant)

    timer = GraphTimer(torch, step, n_sets)
    ms, regions = timer.time(K, W, barrier, agree_max)
    npas.check_device_status(ws)
    kid = npas.conv2d_bp_kernel(case.x.shape, sets[0][1], stride=case.stride, pad=case.pad, relu=case.relu,
                                bias=bias is not None, path=path, variant=variant)
    return {"ms": ms, "regions": regions, "n_sets": n_sets, "sets": sets, "bias": bias, "ws": ws,
            "kernel": npas.CONV_KERNELS[kid]}


def bench_linear(torch, npas, case, K, W, barrier):
    dev = torch.device("cuda")
    set_bytes = case.algorithmic_bytes()
    n_sets = max(2, -(-int(1.3 * L2_BYTES) // set_bytes))
    x0 = torch.from_numpy(case.x).to(dev).to(torch.bfloat16)
    w = torch.from_numpy(case.w).to(dev).to(torch.bfloat16)
    blob0 = npas.pack_bb(w, case.row_keep, case.col_keep, case.Bo, case.Bi)
    bias = torch.from_numpy(case.bias).to(dev)
    sets = [(x0 if i == 0 else torch.roll(x0, i, 0).contiguous(),
             blob0 if i == 0 else npas.BbBlob(blob0.data.clone(), blob0.desc),
             torch.empty((case.M, case.O), dtype=torch.bfloat16, device=dev)) for i in range(n_sets)]
    ws = npas.workspace()

    def step(i):
        x, blob, y = sets[i % n_sets]
        npas.linear_bb(x, blob, bias, relu=case.relu, out=y, ws=ws)

    ms, regions = GraphTimer(torch, step, n_sets).time(K, W, barrier)
    npas.check_device_status(ws)
    kid = npas.linear_bb_kernel(case.M, blob0, relu=case.relu, bias=True)
    return {"ms": ms, "regions": regions, "n_sets": n_sets, "kernel": npas.LINEAR_KERNELS[kid]}


def roofline_block(case, peaks, ms_step, kernel, traffic=None):
    """The roofline of one workload: tensor-bound when the kept MACs at the measured bf16 peak take longer
    than the algorithmic bytes at the measured HBM bandwidth, else HBM-bound."""
    flops = 2.0 * case.kept_macs()
    t_mma = flops / (peaks["bf16_tflops"] * 1e12)
    t_hbm = case.algorithmic_bytes() / (peaks["hbm_gbs"] * 1e9)
    t = ms_step * 1e-3
    if t_mma >= t_hbm:
        ach, peak, unit, bound = flops / t / 1e12, peaks["bf16_tflops"], "TFLOP/s", "tensor"
    else:
        ach, peak, unit, bound = case.algorithmic_bytes() / t / 1e9, peaks["hbm_gbs"], "GB/s", "hbm"
    return {"bound": bound, "achieved": round(ach, 2), "peak": peak, "unit": unit, "frac": round(ach / peak, 4),
            "traffic": traffic, "kernel": kernel, "peak_source": peaks["source"] + (" (burst)" if bound == "tensor" else "")}


def profile_traffic(kernel):
    """dram bytes per launch of the headline kernel from the committed ncu summary (a line
    `traffic_bytes_per_launch: <number>` in profiles/<kernel>_config5_16x16_3taps.md); None when there is none."""
    path = os.path.join(ROOT, "profiles", f"{kernel}_config5_16x16_3taps.md")
    try:
        for line in open(path):
            if line.startswith("traffic_bytes_per_launch:"):
                return float(line.split(":", 1)[1])
    except OSError:
        pass
    return None


def bench_stack(torch, npas, peaks, N=64, reps=5, graph_only=False):
    """configs[3]: the ResNet-50-topology stack, whole forward in one CUDA graph, plus every layer
    alone (a graph of `reps` launches on the tensors the layer sees inside the stack)."""
    from paper_2012_00596_b200 import inputs
    from paper_2012_00596_b200.resnet50 import Resnet50Stack
    layers = inputs.config4()
    net = Resnet50Stack(layers)
    x = torch.from_numpy(inputs.config4_input(N)).cuda().to(torch.bfloat16)

    def timed(graph, n):
        graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    for _ in range(2):
        net.forward(x)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        net.forward(x)
    ms_batch = timed(g, reps)
    net.check()
    if graph_only:          # (for a launch list of the stack alone)
        return {"workload": f"configs[3]: ResNet-50-topology stack, N={N}", "ms": round(ms_batch, 4)}
    _, seen, _ = net.forward(x, keep=True)
    rows, t_roof_sum = [], 0.0
    for i, (lay, (xin, res, out)) in enumerate(zip(layers, seen)):
        net.run_layer(i, xin, res, out)
        gl = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gl):
            for _ in range(reps):
                net.run_layer(i, xin, res, out)
        ms = timed(gl, 2) / reps
        t_roof = max(2.0 * lay.kept_macs_per_image() * N / (peaks["bf16_tflops"] * 1e12),
                     (lay.algorithmic_bytes_per_image() * N + lay.weight_bytes()) / (peaks["hbm_gbs"] * 1e9))
        t_roof_sum += t_roof
        rows.append([lay.name, round(ms * 1e3, 1), round(t_roof / (ms * 1e-3), 3)])
    net.check()
    # first layer + ReLU + max-pool: the fused kernel against the two separate ones (graphs of `reps` launches)
    fused = {}
    try:
        x0, y0 = seen[0][0], seen[0][2]
        pooled = npas.maxpool2d(y0, 3, 2, 1)
        for name, f in (("fused_us", lambda: npas.conv2d_bp_maxpool(x0, net.blobs[0], net.biases[0], stride=2, pad=3, relu=True, ws=net.ws, out=pooled)),
                        ("conv_then_pool_us", lambda: (npas.conv2d_bp(x0, net.blobs[0], net.biases[0], stride=2, pad=3, relu=True, ws=net.ws, out=y0),
                                                       npas.maxpool2d(y0, 3, 2, 1)))):
            f()
            gf = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gf):
                for _ in range(reps):
                    f()
            fused[name] = round(timed(gf, 2) / reps * 1e3, 1)
    except Exception as exc:      # reported, not fatal: the stack number above stands on its own
        fused = {"error": str(exc)[:80]}
    # the same stack with every layer on the kernel and tile shape the library's tuner measured fastest for it
    tuned = {}
    try:
        plans = net.tune(x, reps=10)
        changed = sum(1 for v in plans.plans.values() if v[0] != 0)
        net.forward(x)
        gt = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gt):
            net.forward(x)
        tuned = {"ms": round(timed(gt, reps), 4), "layers_tuned": len(plans.plans), "layers_on_a_forced_kernel": changed}
        net.check()
    except Exception as exc:
        tuned = {"error": str(exc)[:80]}
    kept = sum(l.kept_macs_per_image() for l in layers) * N
    worst = sorted(rows, key=lambda r: r[1] * (1.0 - min(r[2], 1.0)), reverse=True)[:10]      # most time above their roofline
    by_kind = {}
    for lay, r in zip(layers, rows):
        k = by_kind.setdefault(lay.kind, [0.0, 0.0])
        k[0] += r[1]
        k[1] += r[1] * r[2]
    ach = t_roof_sum / (ms_batch * 1e-3)
    return {"workload": f"configs[3]: ResNet-50-topology stack, N={N}, 224x224, 53 convolutions + max-pool in one CUDA graph",
            "ms": round(ms_batch, 4), "kept_mac_tflops": round(2.0 * kept / (ms_batch * 1e-3) / 1e12, 1),
            "roofline": {"bound": "hbm (sum of the per-layer rooflines; the 14x14 and 7x7 3x3 layers are tensor-bound)",
                         "achieved": round(t_roof_sum * 1e3, 4), "peak": round(ms_batch, 4), "unit": "ms (roofline sum / measured)",
                         "frac": round(ach, 4), "traffic": None, "kernel": "53 layer kernels + max-pool"},
            "us_by_kind": {k: [round(v[0], 1), round(v[1] / v[0], 3)] for k, v in by_kind.items()},
            "first_layer_and_maxpool": fused,
            "with_tuned_plans": tuned,
            "ten_layers_furthest_from_roofline_us_frac": worst,
            "note": "per-layer times: the layer alone, back to back on the tensors it sees in the stack (small inputs stay in L2)"}


def bench_offline_steps(torch, npas, c2, c3, peaks, reps=20):
    """Offline (compile-time) steps on the two standard layers: magnitude pruning and packing."""
    w2 = torch.from_numpy(c2.w).cuda().to(torch.bfloat16)
    w3 = torch.from_numpy(c3.w).cuda().to(torch.bfloat16)

    def timed(f):
        f()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            f()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps * 1e3

    out = {"workload": "offline steps on the configs[1] / configs[2] weights (us per call, host launch overhead included)",
           "prune_bp_us": timed(lambda: npas.prune_bp_magnitude(w2, c2.Mb, c2.Nb, 3)),
           "prune_bb_us": timed(lambda: npas.prune_bb_magnitude(w3, c3.Bo, c3.Bi, 16, 16)),
           "pack_bp_us": timed(lambda: npas.pack_bp(w2, c2.tap_mask, c2.Mb, c2.Nb)),
           "pack_bb_us": timed(lambda: npas.pack_bb(w3, c3.row_keep, c3.col_keep, c3.Bo, c3.Bi)),
           "ms": 0.0, "roofline_frac": 0.0}
    return out


def dense_library_ms(torch, kind, case, iters=200):
    """cuDNN / cuBLAS dense on the same shape through torch (context row, not part of the product)."""
    try:
        if kind == "conv":
            torch.backends.cudnn.benchmark = True
            n_sets = max(2, -(-int(1.3 * L2_BYTES) // case.algorithmic_bytes()))
            xs = [torch.randn(case.N, case.C, case.H, case.W, device="cuda", dtype=torch.bfloat16).relu_()
                  .contiguous(memory_format=torch.channels_last) for _ in range(n_sets)]
            w = torch.randn(case.K, case.C, case.R, case.S, device="cuda", dtype=torch.bfloat16).contiguous(
                memory_format=torch.channels_last)
            f = lambda i: torch.nn.functional.conv2d(xs[i % n_sets], w, None, stride=case.stride, padding=case.pad)
        else:
            n_sets = max(2, -(-int(1.3 * L2_BYTES) // case.algorithmic_bytes()))
            xs = [torch.randn(case.M, case.I, device="cuda", dtype=torch.bfloat16) for _ in range(n_sets)]
            w = torch.randn(case.O, case.I, device="cuda", dtype=torch.bfloat16)
            f = lambda i: torch.nn.functional.linear(xs[i % n_sets], w)
        for i in range(10):
            f(i)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(iters):
                f(i)
        g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); g.replay(); e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters
    except Exception as exc:  # library path unavailable: context only
        return None


def e2e_conv(torch, npas, case, sets, bias, ws, steps):
    """Same metric through the public API with HOST buffers.  Every step copies its input from pinned host
    memory to the device, runs the convolution and copies its output back to pinned host memory, all inside
    the timed region.  Steps are pipelined the way a serving loop would be: the upload of step i + 1 and the
    download of step i - 1 run on their own streams beside the convolution of step i (two device buffer
    sets, events between the streams), so the figure is bounded by the slower copy direction."""
    n_buf = 2
    x_host = [torch.from_numpy(case.x).to(torch.bfloat16).pin_memory() for _ in range(n_buf)]
    y_host = [torch.empty((case.N, case.P, case.Q, case.K), dtype=torch.bfloat16).pin_memory() for _ in range(n_buf)]
    bufs = [sets[i % len(sets)] for i in range(n_buf)]
    s_up, s_run, s_down = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    up_done = [torch.cuda.Event() for _ in range(n_buf)]
    run_done = [torch.cuda.Event() for _ in range(n_buf)]
    down_done = [torch.cuda.Event() for _ in range(n_buf)]

    def run(n):
        for i in range(n):
            j = i % n_buf
            x_dev, blob, y_dev = bufs[j]
            with torch.cuda.stream(s_up):
                s_up.wait_event(run_done[j])            # the convolution that last read this input buffer
                x_dev.copy_(x_host[j], non_blocking=True)
                up_done[j].record(s_up)
            with torch.cuda.stream(s_run):
                s_run.wait_event(up_done[j])
                s_run.wait_event(down_done[j])          # the download that last read this output buffer
                npas.conv2d_bp(x_dev, blob, bias, None, stride=case.stride, pad=case.pad, relu=case.relu, out=y_dev, ws=ws)
                run_done[j].record(s_run)
            with torch.cuda.stream(s_down):
                s_down.wait_event(run_done[j])
                y_host[j].copy_(y_dev, non_blocking=True)
                down_done[j].record(s_down)

    torch.cuda.synchronize()
    run(4)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cur = torch.cuda.current_stream()
    e0.record(cur)
    for st in (s_up, s_run, s_down):
        st.wait_event(e0)
    run(steps)
    for st in (s_up, s_run, s_down):
        cur.wait_stream(st)
    e1.record(cur)
    torch.cuda.synchronize()
    npas.check_device_status(ws)
    ms = e0.elapsed_time(e1) / steps
    return ms, x_host[0].numel() * 2, y_host[0].numel() * 2


def oracle_sample(case, n_points, seed=1):
    import oracle
    from paper_2012_00596_b200 import inputs
    rng = inputs.rng_for(seed)
    pts = np.stack([rng.integers(0, case.N, n_points), rng.integers(0, case.P, n_points),
                    rng.integers(0, case.Q, n_points), rng.integers(0, case.K, n_points)], axis=1).astype(np.int32)
    if not hasattr(case, "_f64"):                    # widen once: the conversion is not part of the oracle's work
        case._f64 = (case.x.astype(np.float64), case.w.astype(np.float64))
    x64, w64 = case._f64
    t0 = time.perf_counter()
    oracle.conv2d_bp(x64, w64, case.tap_mask, Mb=case.Mb, Nb=case.Nb, stride=case.stride, pad=case.pad, bias=case.bias,
                     relu=case.relu, points=pts)
    return time.perf_counter() - t0


def kept_flops_per_output(case):
    return 2.0 * case.kept_macs() / (case.N * case.P * case.Q * case.K)


def cpu_baseline(case, budget_s=12.0):
    """The oracle as it stands, timed on the host cores on a bounded sample of the workload: passes over
    a sample of output elements (the whole batch if it is quick enough) until about `budget_s` seconds."""
    import oracle
    n = 20000
    t = oracle_sample(case, n)
    total = case.N * case.P * case.Q * case.K
    n2 = int(min(total, max(n, n * budget_s / max(t, 1e-6))))
    passes, t2 = 0, 0.0
    while passes == 0 or (t2 < budget_s and passes < 200):
        t2 += oracle_sample(case, n2, seed=2 + passes)
        passes += 1
    return {"value": kept_flops_per_output(case) * n2 * passes / t2 / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(),
            "kind": "oracle",
            "sample": f"{passes} passes over {n2} of {total} output elements of the same workload, fp64, {t2:.1f} s"}


def run_reference(args, case):
    """--impl reference: the CPU oracle, unmodified, timed on the host cores (rank 0 only)."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    oracle.build()
    total = case.N * case.P * case.Q * case.K
    t_probe = oracle_sample(case, 20000)
    per_point = t_probe / 20000
    budget = 120.0 / max(1, args.steps + args.warmup)
    n_pts = int(min(total, max(256, budget / per_point)))
    for _ in range(args.warmup):
        oracle_sample(case, n_pts, seed=3)
    t0 = time.perf_counter()
    for i in range(args.steps):
        oracle_sample(case, n_pts, seed=4 + i)
    dt = time.perf_counter() - t0
    value = kept_flops_per_output(case) * n_pts * args.steps / dt / 1e12
    sample = f"{n_pts} of {total} output elements per step, fp64"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": workload_config(case),
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


METRIC = "block-punched CONV kept-MAC TFLOP/s"
HEADLINE = dict(Mb=16, Nb=16, taps=3)


def headline_case():
    from paper_2012_00596_b200 import inputs
    return inputs.config5(HEADLINE["Mb"], HEADLINE["Nb"], HEADLINE["taps"])


def workload_config(case):
    return {"workload": "configs[4] sweep point: 3x3 CONV 64x28x28x512->512 bf16, stride 1, pad 1, blocks 16x16, 3 of 9 taps",
            "N": case.N, "H": case.H, "W": case.W, "C": case.C, "K": case.K, "Mb": case.Mb, "Nb": case.Nb,
            "kept_macs": case.kept_macs(), "algorithmic_bytes": case.algorithmic_bytes()}


def conv_entry(torch, npas, peaks, case, label, K, W, barrier, dense=True):
    r = bench_conv(torch, npas, case, K, W, barrier)
    ms = r["ms"] / K
    e = {"workload": label, "ms": round(ms, 5), "kept_mac_tflops": round(2.0 * case.kept_macs() / (ms * 1e-3) / 1e12, 1),
         "roofline": roofline_block(case, peaks, ms, r["kernel"])}
    if dense:
        d = dense_library_ms(torch, "conv", case, iters=max(20, min(200, K)))
        e["dense_library_ms"] = None if d is None else round(d, 5)
    return e


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the other workloads and the CPU baseline")
    ap.add_argument("--only", default=None, choices=["gemm", "conv2", "conv5kr", "conv5d2", "stack"],
                    help="time only the named secondary workload and print its line (for profiling its kernel): gemm = "
                         "configs[2]; conv2 = configs[1]; conv5kr = the sweep point 32x32 blocks, 2 of 9 taps (kept-pairs kernel); "
                         "conv5d2 = the headline workload forced onto the CTA-pair dense-image kernel (path 7); stack = configs[3], "
                         "the whole forward as one CUDA graph, --steps replays")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    from paper_2012_00596_b200 import inputs
    if args.impl == "reference":
        run_reference(args, headline_case())
        return

    import torch
    import paper_2012_00596_b200 as npas
    from paper_2012_00596_b200 import dist as npd
    npas.load()                                  # fails loudly when the CUDA library is missing
    rank, local_rank, world = npd.init("nccl")
    torch.cuda.set_device(local_rank)
    peaks = measured_peaks()

    if args.only:
        clk = ClockSampler(local_rank)
        clk.__enter__()
        if args.only == "stack":
            line = bench_stack(torch, npas, peaks, reps=max(1, min(args.steps, 50)), graph_only=True)
        elif args.only == "gemm":
            c3 = inputs.config3()
            r = bench_linear(torch, npas, c3, args.steps, args.warmup, npd.barrier)
            line = {"workload": "configs[2]: block-based GEMM 3136x512->2048, 64x64 blocks keep 16x16", "ms": r["ms"] / args.steps,
                    "roofline": roofline_block(c3, peaks, r["ms"] / args.steps, r["kernel"])}
        else:
            c = inputs.config2() if args.only == "conv2" else inputs.config5(32, 32, 2) if args.only == "conv5kr" else headline_case()
            r = bench_conv(torch, npas, c, args.steps, args.warmup, npd.barrier, path=7 if args.only == "conv5d2" else 0)
            line = {"workload": args.only, "ms": r["ms"] / args.steps,
                    "roofline": roofline_block(c, peaks, r["ms"] / args.steps, r["kernel"])}
        clk.__exit__(None, None, None)
        line["clocks"] = clk.summary()
        if rank == 0:
            print(json.dumps(line))
        return

    case = headline_case()
    agree = lambda v: npd.max_over_ranks(v, device="cuda")
    with ClockSampler(local_rank) as clk:
        r = bench_conv(torch, npas, case, args.steps, args.warmup, npd.barrier, agree_max=agree)
    flops_step = 2.0 * case.kept_macs()
    value, ms_step = npd.whole_job_throughput(flops_step / 1e12, args.steps, r["ms"], device="cuda")
    clocks = clk.summary()

    e2e_ms, h2d, d2h = e2e_conv(torch, npas, case, r["sets"], r["bias"], r["ws"], steps=20)
    e2e_value, _ = npd.whole_job_throughput(flops_step / 1e12, 1, e2e_ms, device="cuda")

    own_ms = r["ms"] / args.steps
    rl = roofline_block(case, peaks, own_ms, r["kernel"], traffic=profile_traffic(r["kernel"]))
    t_mma = flops_step / (peaks["bf16_tflops"] * 1e12)
    t_hbm = case.algorithmic_bytes() / (peaks["hbm_gbs"] * 1e9)
    rl.update({"t_mma_us": round(t_mma * 1e6, 2), "t_hbm_us": round(t_hbm * 1e6, 2), "target_0p60_met": bool(rl["frac"] >= 0.60)})
    if r["kernel"] in ("conv_bp_d2_kernel", "conv_bp_dn_kernel"):      # these multiply the zero-filled dense weights
        rl["dense_work_frac"] = round(2.0 * case.N * case.P * case.Q * case.K * case.C * case.R * case.S /
                                      (own_ms * 1e-3) / 1e12 / peaks["bf16_tflops"], 4)
    out = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(case),
        "timing": {"launch": f"CUDA graphs of {min(args.steps, GRAPH_CHUNK)} steps, each replayed once untimed first",
                   "timed_regions": r["regions"], "statistic": "median of the timed K-step regions" if r["regions"] > 1 else "one K-step region",
                   "l2": f"rotating {r['n_sets']} buffer sets ({r['n_sets'] * case.algorithmic_bytes() / 1e6:.0f} MB) larger than L2",
                   "batch_per_gpu": case.N, "parallelism": f"replicas x{world}"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms},
        "gpu_launches": args.steps,
        "roofline": rl,
    }
    if rank == 0 and world == 1 and not args.no_extras:
        sets = r.pop("sets")
        del sets, r
        torch.cuda.empty_cache()
        out["dense_library_ms"] = dense_library_ms(torch, "conv", case, iters=40)
        extras = []
        stack = bench_stack(torch, npas, peaks)
        torch.cuda.empty_cache()
        extras.append(stack)                                         # configs[3] first
        c3 = inputs.config3()
        r3 = bench_linear(torch, npas, c3, 2000, 100, npd.barrier)
        ms3 = r3["ms"] / 2000
        d3 = dense_library_ms(torch, "linear", c3)
        extras.append({"workload": "configs[2]: block-based GEMM 3136x512->2048, 64x64 blocks keep 16x16, bias+ReLU",
                       "ms": round(ms3, 5), "kept_mac_tflops": round(2.0 * c3.kept_macs() / (ms3 * 1e-3) / 1e12, 1),
                       "roofline": roofline_block(c3, peaks, ms3, r3["kernel"]),
                       "dense_library_ms": None if d3 is None else round(d3, 5)})
        c2 = inputs.config2()
        extras.append(conv_entry(torch, npas, peaks, c2, "configs[1]: 3x3 CONV 32x14x14x256->256, blocks 16x8, 3 of 9 taps, bias+ReLU",
                                 4000, 200, npd.barrier))
        c1 = inputs.config1()
        x1, w1 = torch.from_numpy(c1.x).cuda(), torch.from_numpy(c1.w).cuda()
        b1 = npas.pack_bp(w1, c1.tap_mask, c1.Mb, c1.Nb)
        ws1 = npas.workspace()
        y1 = npas.conv2d_bp(x1, b1, ws=ws1)
        g1 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g1):
            for _ in range(200):
                npas.conv2d_bp(x1, b1, out=y1, ws=ws1)
        g1.replay(); torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); g1.replay(); e1.record(); torch.cuda.synchronize()
        extras.append({"workload": "configs[0]: 3x3 CONV 1x16x16x32->32 fp32, blocks 8x4, 3 of 9 taps (correctness workload, launch-bound)",
                       "ms": round(e0.elapsed_time(e1) / 200, 5), "roofline": {"bound": "launch latency", "kernel": "conv_bp_simt_kernel"}})
        # the sweep: [Mb, Nb, taps, ms, kept-MAC TFLOP/s, roofline bound, fraction, kernel]
        sweep, dense5 = [], out["dense_library_ms"]
        for (Mb, Nb) in [(4, 4), (8, 8), (16, 16), (32, 32)]:
            for taps in (1, 2, 3, 5, 9):
                c5 = inputs.config5(Mb, Nb, taps)
                reps = 20 if Mb >= 16 else 4
                r5 = bench_conv(torch, npas, c5, reps, 3, npd.barrier)
                ms5 = r5["ms"] / reps
                rb = roofline_block(c5, peaks, ms5, r5["kernel"])
                sweep.append([Mb, Nb, taps, round(ms5, 4), round(2.0 * c5.kept_macs() / (ms5 * 1e-3) / 1e12), rb["bound"], rb["frac"],
                              r5["kernel"].replace("conv_bp_", "").replace("_kernel", "")])
                del c5, r5
                torch.cuda.empty_cache()
        extras.append({"workload": "configs[4]: 3x3 CONV 64x28x28x512->512, every block size x taps kept",
                       "columns": ["Mb", "Nb", "taps", "ms", "kept_mac_tflops", "bound", "roofline_frac", "kernel"],
                       "points": sweep, "dense_library_ms": dense5})
        extras.append(bench_offline_steps(torch, npas, c2, c3, peaks))
        out["per_config"] = extras
        out["cpu_baseline"] = cpu_baseline(case)
    if rank == 0:
        print(json.dumps(out))


if __name__ == "__main__":
    main()
