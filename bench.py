#!/usr/bin/env python
"""Benchmark of the decoder-layer hot path on B200 (one process per GPU; N > 1 = independent replicas).

    python bench.py --gpus 1 --steps 20 --warmup 3
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N --master-addr 127.0.0.1 --master-port P \
        bench.py --gpus N --steps K --warmup W
    python bench.py --impl reference ...        # the CPU oracle, timed on the host cores

A "step" is one pass of the whole hot path over one batch of synthetic input: forward and
backward of every layer of the workload on every micro-batch (workload 2, the default: one
decoder layer d=2048, 16x128 heads, F=8192, S=1024, B=8).  Rank 0 prints ONE JSON line.

Timing: CUDA events on the launching stream, after warm-up, barrier + synchronize on both
sides, max over ranks.  Per-kernel-class times (for the roofline object) come from a second,
instrumented pass of the same K steps in which the library brackets every launch with CUDA
events; the headline number is from the un-instrumented pass.  The end-to-end number repeats
the step with host buffers: pinned host -> device copies of x and dy and device -> host reads
of y and dx inside the timed region.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram bytes read+written per GEMM launch (average over the 12 GEMM launches of a workload-2 step),
# from one ncu pass (dram__bytes_read.sum + dram__bytes_write.sum) over those launches; None for
# workloads without a capture.
GEMM_DRAM_TRAFFIC_PER_LAUNCH = {"cfg2_d2048_s1024_b8": 220.7e6}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    except Exception:
        return dict(FALLBACK_PEAKS, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.005):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if visible:
                ids = [v for v in visible.split(",") if v.strip()]
                if index < len(ids) and ids[index].strip().isdigit():
                    phys = int(ids[index])
            self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4)}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for n, bit in names.items():
                    if mask & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def max_over_ranks(ms: float, world: int, device) -> float:
    """The slowest rank's time: what a multi-rank number is computed from (no-op for one rank)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank: float, world: int, ms: float) -> float:
    """Replicas: every rank processes the same number of units; the job's rate uses the slowest rank's time."""
    return world * units_per_rank / (ms * 1e-3)


def isolated_elementwise(pw, w, peaks, dev, iters=30, nbuf=6):
    """LayerNorm / column-sum kernels timed back to back through the single-step entry points on
    HBM-resident inputs (a rotation of `nbuf` buffer sets, far larger than the 126 MB L2), so that
    launch gaps and event brackets do not count: GB/s of algorithmic bytes vs the measured copy rate."""
    import torch
    T, d, F = w.tokens, w.d_model, w.d_ff
    g = torch.Generator(device="cpu").manual_seed(1)
    rnd = lambda *shape: torch.randn(shape, generator=g).to(torch.bfloat16).to(dev)
    xs = [rnd(T, d) for _ in range(nbuf)]
    hs = [torch.empty_like(x) for x in xs]
    gamma, beta = torch.ones(d, dtype=torch.bfloat16, device=dev), torch.zeros(d, dtype=torch.bfloat16, device=dev)
    mu, rs = torch.empty(T, device=dev), torch.empty(T, device=dev)
    outs = [torch.zeros(d, device=dev) for _ in range(4)]
    part = torch.empty(pw.op_layernorm_bwd_scratch_bytes(T, d), dtype=torch.uint8, device=dev)

    def timeit(fn):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            fn(i)
        e1.record()
        torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1) / iters

    res = {}
    ms = timeit(lambda i: pw.op_layernorm_fwd(xs[i % nbuf], gamma, beta, 1e-5, hs[i % nbuf], mu, rs))
    res["ln_fwd"] = (ms, 4.0 * T * d + 8.0 * T)
    dhs = [rnd(T, d) for _ in range(nbuf)]
    ms = timeit(lambda i: pw.op_layernorm_bwd(dhs[i % nbuf], xs[i % nbuf], mu, rs, gamma, xs[(i + 1) % nbuf], hs[i % nbuf],
                                               outs[0], outs[1], outs[2], outs[3], False, part))
    res["ln_bwd"] = (ms, 8.0 * T * d + 8.0 * T)
    del dhs
    for name, N in (("colsum_ff", F), ("colsum_qkv", 3 * d)):
        n = max(2, min(nbuf, int(1.5e9 // (2 * T * N))))
        ins = [rnd(T, N) for _ in range(n)]
        out = torch.zeros(N, device=dev)
        sc = torch.empty(pw.op_colsum_scratch_bytes(T, N), dtype=torch.uint8, device=dev)
        ms = timeit(lambda i: pw.op_colsum(ins[i % n], out, False, sc))
        res[name] = (ms, 2.0 * T * N)
        del ins
    # gradient apply over one layer's parameter tensors (a rotation of two sets: 14 bytes per element)
    shapes = [(d,), (d,), (3 * d, d), (3 * d,), (d, d), (d,), (d,), (d,), (F, d), (F,), (d, F), (d,)]
    n_el = sum(int(torch.Size(sh).numel()) for sh in shapes)
    sets = []
    for _ in range(2 if n_el * 10 * 2 < 40e9 else 1):
        ps = [torch.zeros(sh, dtype=torch.bfloat16, device=dev) for sh in shapes]
        ms_ = [torch.zeros(sh, device=dev) for sh in shapes]
        gs = [torch.full(sh, 1e-3, device=dev) for sh in shapes]
        sets.append(list(zip(ps, ms_, gs)))
    ms = timeit(lambda i: pw.sgd_apply(sets[i % len(sets)], 1e-3))
    res["sgd_apply"] = (ms, 14.0 * n_el)
    del sets
    return {k: {"us": ms * 1e3, "gbs": b / (ms * 1e-3) / 1e9, "frac_of_measured_hbm": b / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
            for k, (ms, b) in res.items()}


def gemm_roofline(g_flops, g_ms, g_n, tot_ms, ms_one_stream, steps, peaks, kernel, traffic):
    """Roofline object of the GEMM family.  `achieved` is the literal figure: the algorithmic FLOPs of
    the GEMM launches (2 M N K each) divided by the sum of their CUDA-event durations, each launch
    bracketed by its own event pair on the launching stream (the instrumented pass).  An event pair
    around every launch keeps a kernel's prologue from overlapping its predecessor's tail and adds
    launch latency, so this is a lower bound on what the kernel does inside the un-instrumented step;
    `achieved_in_step` apportions instead: (GEMM share of the bracketed times) x (event-timed step with
    every kernel on one stream and no events between launches)."""
    share = g_ms / tot_ms
    ms_gemm_step = share * ms_one_stream
    in_step = (g_flops / steps) / (ms_gemm_step * 1e-3) / 1e12
    bracketed = g_flops / (g_ms * 1e-3) / 1e12
    return {
        "kernel": kernel, "bound": "tensor", "achieved": bracketed, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
        "frac": bracketed / peaks["bf16_tflops"], "peak_source": peaks["source"] + " (burst cuBLAS bf16)",
        "frac_of_sustained_peak": bracketed / peaks["bf16_tflops_sustained"],
        "flops_per_launch": g_flops / g_n, "ms_per_launch": g_ms / g_n, "launches_per_step": g_n / steps,
        "share_of_step": share,
        "how": "algorithmic FLOPs of the GEMM launches / sum of their per-launch CUDA-event durations (instrumented pass)",
        "achieved_in_step": in_step, "frac_in_step": in_step / peaks["bf16_tflops"],
        "ms_per_launch_in_step": ms_gemm_step / (g_n / steps),
        "how_in_step": "GEMM share of the per-launch event times x the event-timed one-stream step (no events between launches)",
        "traffic": traffic,
    }


def hw_flops_per_step(w) -> float:
    """Executed FLOPs: model FLOPs plus, with recompute, one forward without the FC2 GEMM."""
    per_call = w.model_flops_per_layer_call()
    if w.recompute:
        per_call += w.fwd_flops_per_layer_call() - 2.0 * w.tokens * w.d_model * w.d_ff
    return per_call * w.n_layers * w.n_microbatches


def oracle_step(oracle, D, params, x, dy):
    y, sv = oracle.layer_fwd(D, params, x)
    oracle.layer_bwd(D, params, x, sv, dy)


def oracle_sample(w, batch):
    """Inputs of a bounded sample of workload w (first `batch` sequences, one layer, one micro-batch)."""
    from oracle import Dims
    from paper_2203_12533_b200 import inputs
    ws = w.with_(batch=batch)
    D = Dims(ws.batch, ws.seq_len, ws.d_model, ws.n_heads, ws.head_dim, ws.d_ff)
    params = [p.float().numpy() for p in inputs.layer_params(ws, 0, 0)]
    x, dy = inputs.microbatch(ws, 0, 0)
    return ws, D, params, x.float().numpy().reshape(ws.tokens, -1), dy.float().numpy().reshape(ws.tokens, -1)


def run_reference(args, w):
    """The CPU oracle as it stands, timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle as oracle_mod
    orc = oracle_mod.Oracle("f32")
    batch = 1
    ws, D, params, x, dy = oracle_sample(w, batch)
    for _ in range(args.warmup):
        oracle_step(orc, D, params, x, dy)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(orc, D, params, x, dy)
    dt = time.perf_counter() - t0
    value = ws.tokens * args.steps / dt
    cores = oracle_mod.host_threads()
    sample = (f"{batch} of {w.batch} sequences (S={w.seq_len}), one layer fwd+bwd per step, fp32 plain-loop C oracle")
    line = {
        "impl": "reference", "metric": "decoder-layer fwd+bwd tokens/s", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "sample": sample},
        "tflops_model": ws.model_flops_per_layer_call() * args.steps / dt / 1e12,
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, w, brief=False):
    """Times workload w; returns the JSON line as a dict (rank 0) or None.  brief: the short form used
    for the secondary workloads of the default run - device-resident steps and the per-class table
    only (no end-to-end pass, no isolated kernels, no CPU baseline), single rank."""
    import torch
    import torch.distributed as dist
    from paper_2203_12533_b200 import binding as pw
    from paper_2203_12533_b200 import inputs

    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if brief:
        rank, world = 0, 1
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for the product path)")
    torch.cuda.set_device(local)
    if world > 1 and not dist.is_initialized():
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    pw.lib()
    peaks = load_peaks()
    dev = torch.device("cuda", local)
    L, M, T, d = w.n_layers, w.n_microbatches, w.tokens, w.d_model
    dispatch = {"opbyop": pw.DISPATCH_OPBYOP, "async": pw.DISPATCH_ASYNC, "graph": pw.DISPATCH_GRAPH}[args.dispatch]
    schedule = pw.SCHEDULE_GPIPE

    stage = pw.Stage(L, w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch,
                     flags=pw.FLAG_LEAN_CTX if args.lean else 0)
    params = [[p.to(dev) for p in inputs.layer_params(w, args.seed, l)] for l in range(L)]
    grads = [[torch.zeros(p.shape, dtype=torch.float32, device=dev) for p in ps] for ps in params]
    host_x, host_dy = [], []
    for m in range(M):
        x, dy = inputs.microbatch(w, args.seed, m)
        host_x.append(x.view(T, d) if brief else x.view(T, d).pin_memory())
        host_dy.append(dy.view(T, d) if brief else dy.view(T, d).pin_memory())
    xs = [t.to(dev) for t in host_x]
    dys = [t.to(dev) for t in host_dy]
    ys = [torch.empty_like(t) for t in xs]
    dxs = [torch.empty_like(t) for t in xs]
    if brief:
        host_x = host_dy = host_y = host_dx = None
    else:
        host_y = [torch.empty((T, d), dtype=torch.bfloat16).pin_memory() for _ in range(M)]
        host_dx = [torch.empty((T, d), dtype=torch.bfloat16).pin_memory() for _ in range(M)]
    ws_bytes = stage.workspace_bytes(M, schedule, w.recompute)
    workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    stream = torch.cuda.Stream(device=dev)

    def step():
        stage.run_chain(params, grads, xs, dys, ys, dxs, workspace, dispatch, schedule, w.recompute, stream=stream)

    # End to end: every step copies its x and dy from pinned host memory and reads its y and dx back.
    # Two device buffer sets and two copy streams pipeline the transfers behind the compute of the
    # neighbouring steps (h2d of step i+1 and d2h of step i-1 overlap the kernels of step i).
    if brief:
        sets = [(xs, dys, ys, dxs)]
    else:
        xs2 = [torch.empty_like(t) for t in xs]
        dys2 = [torch.empty_like(t) for t in xs]
        ys2 = [torch.empty_like(t) for t in xs]
        dxs2 = [torch.empty_like(t) for t in xs]
        sets = [(xs, dys, ys, dxs), (xs2, dys2, ys2, dxs2)]
    s_h2d, s_d2h = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ev_in = [torch.cuda.Event() for _ in range(2)]       # inputs of set k are on the device
    ev_done = [torch.cuda.Event() for _ in range(2)]     # compute on set k finished
    ev_out = [torch.cuda.Event() for _ in range(2)]      # outputs of set k have been read back
    e2e_state = {"i": 0}

    def e2e_prefetch(k):
        with torch.cuda.stream(s_h2d):
            s_h2d.wait_event(ev_done[k])                 # the previous user of set k is done with its inputs
            for m in range(M):
                sets[k][0][m].copy_(host_x[m], non_blocking=True)
                sets[k][1][m].copy_(host_dy[m], non_blocking=True)
            ev_in[k].record(s_h2d)

    def step_e2e():
        i = e2e_state["i"]
        k = i & 1
        if i == 0:
            e2e_prefetch(0)
        e2e_prefetch(k ^ 1)                              # next step's inputs travel while this step computes
        stream.wait_event(ev_in[k])
        stream.wait_event(ev_out[k])                     # outputs of set k from two steps ago were read back
        a, b, c, e = sets[k]
        stage.run_chain(params, grads, a, b, c, e, workspace, dispatch, schedule, w.recompute, stream=stream)
        ev_done[k].record(stream)
        with torch.cuda.stream(s_d2h):
            s_d2h.wait_event(ev_done[k])
            for m in range(M):
                host_y[m].copy_(c[m], non_blocking=True)
                host_dx[m].copy_(e[m], non_blocking=True)
            ev_out[k].record(s_d2h)
        e2e_state["i"] = i + 1

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def timed(fn, steps, per_step=None):
        """Milliseconds for `steps` calls of fn (max over ranks).  per_step: a list that receives this
        rank's time of every single step (one more event per step)."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        marks = []
        barrier()
        with torch.cuda.stream(stream):
            e0.record(stream)
            for _ in range(steps):
                fn()
                if per_step is not None:
                    marks.append(torch.cuda.Event(enable_timing=True))
                    marks[-1].record(stream)
            stream.wait_stream(s_d2h)                    # (end-to-end runs) the last results are on the host
            e1.record(stream)
        torch.cuda.synchronize(dev)
        ms = e0.elapsed_time(e1)
        if per_step is not None:
            prev = e0
            for m in marks:
                per_step.append(prev.elapsed_time(m))
                prev = m
        barrier()
        return max_over_ranks(ms, world, dev)

    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            step()
    torch.cuda.synchronize(dev)
    code, site = stage.status()
    if code != 0:
        raise SystemExit(f"device status {code} at site {site} after warm-up")

    n0 = stage.launch_count()
    per_step = []
    with ClockSampler(local) as clocks:
        ms_total = timed(step, args.steps, per_step)
    launches = stage.launch_count() - n0
    ms_step = ms_total / args.steps
    tokens_step = T * M
    value = whole_job_value(tokens_step, world, ms_step)

    # end to end through the public API with host buffers; it follows the device-resident pass directly, so
    # that both see the same clock regime (tens of milliseconds at full clock, before the power cap bites)
    ms_e2e = e2e_value = None
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    if not brief:
        for k in range(2):
            ev_done[k].record(stream)
            ev_out[k].record(stream)
        with torch.cuda.stream(stream):
            step_e2e()
            step_e2e()
        torch.cuda.synchronize(dev)
        e2e_state["i"] = 0
        ms_e2e = timed(step_e2e, e2e_steps) / e2e_steps
        e2e_value = whole_job_value(tokens_step, world, ms_e2e)
    # instrumented pass: per-kernel-class device time from CUDA events inside the library
    prof = None
    if dispatch != pw.DISPATCH_GRAPH:
        stage.profile_begin()
        with torch.cuda.stream(stream):
            for _ in range(args.steps):
                step()
        prof = stage.profile_end()
    # the same step with every kernel on the calling stream and no events between launches: the time
    # the per-class shares of the instrumented pass are applied to
    ms_one_stream = None
    if prof is not None:
        stage.set_side_stream(False)
        with torch.cuda.stream(stream):
            step()
        ms_one_stream = timed(step, args.steps) / args.steps
        stage.set_side_stream(True)

    code, site = stage.status()
    if code != 0:
        raise SystemExit(f"device status {code} at site {site}")

    model_flops = w.model_flops_per_layer_call() * L * M
    hw_flops = hw_flops_per_step(w)
    line = {
        "metric": "decoder-layer fwd+bwd tokens/s", "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
        "ms_per_step_median": statistics.median(per_step), "ms_per_step_best": min(per_step), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "d_model": w.d_model, "heads": f"{w.n_heads}x{w.head_dim}", "d_ff": w.d_ff,
                   "seq_len": w.seq_len, "microbatch": w.batch, "layers": L, "microbatches": M,
                   "recompute": bool(w.recompute), "lean_ctx": bool(args.lean), "workspace_bytes": int(ws_bytes),
                   "dispatch": args.dispatch, "parallelism": f"replicas x{world}",
                   "l2": "working set per step (activations + weights + fp32 grads) is > 1 GB, far above the 126 MB L2"},
        "tflops_model": world * model_flops / (ms_step * 1e-3) / 1e12,
        "tflops_hw": world * hw_flops / (ms_step * 1e-3) / 1e12,
        "frac_bf16_peak_burst": hw_flops / (ms_step * 1e-3) / 1e12 / peaks["bf16_tflops"],
        "frac_bf16_peak_sustained": hw_flops / (ms_step * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
        "frac_bf16_nominal_2250": hw_flops / (ms_step * 1e-3) / 1e12 / 2250.0,   # datasheet dense bf16, for context
        "peaks": peaks,
        "clocks": clocks.summary(),
        "e2e": {"value": e2e_value, "unit": "tokens/s", "ms_per_step": ms_e2e, "steps": e2e_steps,
                "how": "pinned host x, dy -> device and y, dx -> pinned host every step, double-buffered on two copy streams",
                "h2d_bytes_per_step": 2 * M * T * d * 2, "d2h_bytes_per_step": 2 * M * T * d * 2},
        "gpu_launches": int(launches),
    }
    if brief:
        del line["e2e"], line["peaks"]
    if prof is not None:
        kernels = {}
        tot_ms = sum(v["ms"] for v in prof.values())
        for name, v in prof.items():
            if v["launches"] == 0:
                continue
            k = {"launches_per_step": v["launches"] / args.steps, "ms_per_step": v["ms"] / args.steps,
                 "share": v["ms"] / tot_ms if tot_ms > 0 else None}
            if v["flops"] > 0:
                k["tflops"] = v["flops"] / (v["ms"] * 1e-3) / 1e12
                k["frac_of_measured_bf16_burst"] = k["tflops"] / peaks["bf16_tflops"]
            if v["bytes"] > 0:
                k["gbs"] = v["bytes"] / (v["ms"] * 1e-3) / 1e9
                k["frac_of_measured_hbm"] = k["gbs"] / peaks["hbm_gbs"]
            kernels[name] = k
        line["kernels"] = kernels
        line["ms_per_step_instrumented"] = tot_ms / args.steps
        g = [prof[n] for n in ("gemm_tn", "gemm_nn", "gemm_nt")]
        g_flops, g_ms, g_n = sum(v["flops"] for v in g), sum(v["ms"] for v in g), sum(v["launches"] for v in g)
        line["roofline"] = gemm_roofline(g_flops, g_ms, g_n, tot_ms, ms_one_stream, args.steps, peaks,
                                         "gemm_pair_kernel (tcgen05 bf16 GEMM: forward, dgrad and wgrad instantiations)",
                                         GEMM_DRAM_TRAFFIC_PER_LAUNCH.get(w.name))
        line["ms_per_step_one_stream"] = ms_one_stream

    if rank == 0 and world == 1 and not brief and not args.no_isolated and w.tokens * w.d_ff <= (1 << 27):
        line["kernels_isolated"] = isolated_elementwise(pw, w, peaks, dev)
    if rank == 0 and world == 1 and not brief and not args.no_sustained:
        # Sustained regime: the same step back to back for at least a second, long enough for the power
        # cap to pull the SM clock down to where it settles; compared with the sustained cuBLAS figure.
        n_sus = max(args.sustained_steps, 1)
        with torch.cuda.stream(stream):
            for _ in range(3):
                step()
        with ClockSampler(local, period_s=0.02) as clk:
            ms_sus = timed(step, n_sus) / n_sus
        line["sustained"] = {
            "steps": n_sus, "seconds": ms_sus * n_sus * 1e-3, "ms_per_step": ms_sus, "value": tokens_step / (ms_sus * 1e-3),
            "unit": "tokens/s", "tflops_model": model_flops / (ms_sus * 1e-3) / 1e12,
            "tflops_hw": hw_flops / (ms_sus * 1e-3) / 1e12,
            "frac_bf16_peak_sustained": hw_flops / (ms_sus * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
            "frac_bf16_peak_burst": hw_flops / (ms_sus * 1e-3) / 1e12 / peaks["bf16_tflops"],
            "clocks": clk.summary()}
    if rank == 0 and world == 1 and not brief and not args.no_cpu_baseline:
        import oracle as oracle_mod
        orc = oracle_mod.Oracle("f32")
        b = min(w.batch, args.cpu_sample_batch)
        wsamp, D, ps, x, dy = oracle_sample(w, b)
        t0 = time.perf_counter()
        oracle_step(orc, D, ps, x, dy)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {
            "value": wsamp.tokens / dt, "unit": "tokens/s", "cores": oracle_mod.host_threads(), "kind": "oracle",
            "seconds": dt,
            "sample": f"{b} of {w.batch} sequences (S={w.seq_len}) through one layer fwd+bwd, fp32 plain-loop C oracle, run once"}
    return line if rank == 0 else None


def lm_flops_per_step(w):
    """(model, executed) FLOPs of one small-LM step: L layers + tied head (logits, dhf, dE: 6 T d V)."""
    head = 6.0 * w.tokens * w.d_model * w.vocab
    per_call = w.model_flops_per_layer_call()
    extra = (w.fwd_flops_per_layer_call() - 2.0 * w.tokens * w.d_model * w.d_ff) if w.recompute else 0.0
    return per_call * w.n_layers + head, (per_call + extra) * w.n_layers + head


def oracle_lm_sample(w, layers):
    """A bounded sample of the LM workload: its first sequence through `layers` layers and the full-vocabulary head."""
    from oracle import Dims
    from paper_2203_12533_b200 import inputs
    ws = w.with_(batch=1, n_layers=layers)
    D = Dims(ws.batch, ws.seq_len, ws.d_model, ws.n_heads, ws.head_dim, ws.d_ff)
    pls = [[p.float().numpy() for p in inputs.layer_params(ws, 0, l)] for l in range(layers)]
    E, g, b, ids, labels = inputs.lm_inputs(ws, 0)
    return ws, D, pls, E.float().numpy(), g.float().numpy(), b.float().numpy(), ids.numpy().ravel(), labels.numpy().ravel()


def run_ours_lm(args, w, brief=False):
    """Workload 5: the whole small language-model step (pw_lm_step) instead of a bare layer chain.
    Returns the JSON line as a dict (rank 0) or None; brief as in run_ours."""
    import torch
    import torch.distributed as dist
    from paper_2203_12533_b200 import binding as pw
    from paper_2203_12533_b200 import inputs

    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if brief:
        rank, world = 0, 1
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for the product path)")
    torch.cuda.set_device(local)
    if world > 1 and not dist.is_initialized():
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    pw.lib()
    peaks = load_peaks()
    dev = torch.device("cuda", local)
    L, T, d, V = w.n_layers, w.tokens, w.d_model, w.vocab
    stage = pw.Stage(L, w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch,
                     flags=pw.FLAG_LEAN_CTX if args.lean else 0)
    E, g, b, ids, labels = inputs.lm_inputs(w, args.seed)
    cpu_params = [inputs.layer_params(w, args.seed, l) for l in range(L)]
    replica = None
    if args.data_parallel:
        # every parameter and every gradient lives in the replica's two flat, peer-mapped buffers
        from paper_2203_12533_b200 import data_parallel
        flat_cpu = [p for ps in cpu_params for p in ps] + [E, g, b]
        replica = data_parallel.Replica([tuple(p.shape) for p in flat_cpu], dev)
        for dst, src in zip(replica.params, flat_cpu):
            dst.copy_(src)
        per = len(cpu_params[0])
        params = [replica.params[l * per:(l + 1) * per] for l in range(L)]
        grads = [replica.grads[l * per:(l + 1) * per] for l in range(L)]
        lm_params, lm_grads = tuple(replica.params[L * per:]), tuple(replica.grads[L * per:])
        if world > 1:                                        # each replica trains on its own batch
            _, _, _, ids, labels = inputs.lm_inputs(w, args.seed + 1000 * rank)
    else:
        params = [[p.to(dev) for p in ps] for ps in cpu_params]
        grads = [[torch.zeros(p.shape, dtype=torch.float32, device=dev) for p in ps] for ps in params]
        lm_params = (E.to(dev), g.to(dev), b.to(dev))
        lm_grads = (torch.zeros(E.shape, dtype=torch.float32, device=dev), torch.zeros(d, device=dev), torch.zeros(d, device=dev))
    host_ids, host_labels = ids.pin_memory(), labels.pin_memory()
    dev_ids, dev_labels = [host_ids.to(dev), host_ids.to(dev)], [host_labels.to(dev), host_labels.to(dev)]
    loss = torch.zeros(1, device=dev)
    host_loss = torch.zeros(1).pin_memory()
    workspace = torch.empty(stage.lm_workspace_bytes(V, w.recompute), dtype=torch.uint8, device=dev)
    stream = torch.cuda.Stream(device=dev)
    state = {"i": 0}

    apply_items = None
    if replica is not None:
        with torch.cuda.stream(stream):
            replica.reduce_apply(0.0, init_master=True, stream=stream)           # master slices from the bf16 parameters
    elif args.apply_lr is not None:
        flat_p = [p for ps in params for p in ps] + list(lm_params)
        flat_g = [x for gs in grads for x in gs] + list(lm_grads)
        flat_m = [torch.empty(p.shape, dtype=torch.float32, device=dev) for p in flat_p]
        apply_items = list(zip(flat_p, flat_m, flat_g))
        with torch.cuda.stream(stream):
            pw.sgd_apply(apply_items, 0.0, init_master=True, stream=stream)      # master copies from the bf16 parameters
    apply_launches = 0 if apply_items is None else -(-len(apply_items) // pw.APPLY_ITEMS_PER_LAUNCH)
    if replica is not None:
        apply_launches = 1

    def apply(lr):
        if replica is not None:
            replica.reduce_apply(lr, stream=stream)
        elif apply_items is not None:
            pw.sgd_apply(apply_items, lr, stream=stream)

    def step():
        stage.lm_step(params, grads, lm_params, lm_grads, dev_ids[0], dev_labels[0], loss, V, workspace, w.recompute, stream=stream)
        apply(args.apply_lr)

    def step_e2e():
        k = state["i"] & 1                                   # the copies are tiny: same stream, alternating buffers
        dev_ids[k].copy_(host_ids, non_blocking=True)
        dev_labels[k].copy_(host_labels, non_blocking=True)
        stage.lm_step(params, grads, lm_params, lm_grads, dev_ids[k], dev_labels[k], loss, V, workspace, w.recompute, stream=stream)
        apply(args.apply_lr)
        host_loss.copy_(loss, non_blocking=True)
        state["i"] += 1

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def timed(fn, steps, per_step=None):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        marks = []
        barrier()
        with torch.cuda.stream(stream):
            e0.record(stream)
            for _ in range(steps):
                fn()
                if per_step is not None:
                    marks.append(torch.cuda.Event(enable_timing=True))
                    marks[-1].record(stream)
            e1.record(stream)
        torch.cuda.synchronize(dev)
        ms = e0.elapsed_time(e1)
        if per_step is not None:
            prev = e0
            for m in marks:
                per_step.append(prev.elapsed_time(m))
                prev = m
        barrier()
        return max_over_ranks(ms, world, dev)

    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            step()
    torch.cuda.synchronize(dev)
    if stage.status() != (0, 0):
        raise SystemExit(f"device status {stage.status()} after warm-up")
    n0 = stage.launch_count()
    per_step = []
    with ClockSampler(local) as clocks:
        ms_step = timed(step, args.steps, per_step) / args.steps
    launches = stage.launch_count() - n0 + apply_launches * args.steps
    loss_after_timed = float(loss.item())
    stage.profile_begin()
    with torch.cuda.stream(stream):
        for _ in range(args.steps):
            step()
    prof = stage.profile_end()
    stage.set_side_stream(False)                             # every kernel on one stream, no events between launches
    with torch.cuda.stream(stream):
        step()
    ms_one_stream = timed(step, args.steps) / args.steps
    stage.set_side_stream(True)
    apply_info = None
    if apply_items is not None or replica is not None:
        n_el = replica.total if replica is not None else sum(p.numel() for p, _, _ in apply_items)
        ms_apply = timed(lambda: apply(0.0), args.steps) / args.steps            # rate 0: same traffic
        apply_info = {"lr": args.apply_lr, "optimizer": "plain SGD, fp32 master copies, bf16 working copies",
                      "tensors": len(replica.shapes) if replica is not None else len(apply_items), "elements": n_el,
                      "launches_per_step": apply_launches, "ms_per_step_alone": ms_apply}
        if replica is None or world == 1:
            gbs = 14.0 * n_el / (ms_apply * 1e-3) / 1e9     # grad 4 + master 4 + 4 + bf16 copy 2 bytes per element, all local
            apply_info.update({"gbs": gbs, "frac_of_measured_hbm": gbs / peaks["hbm_gbs"]})
        else:
            # per replica: 4 bytes per element of its slice from each peer come in, 2 bytes per element go out to each peer
            link_in = 4.0 * (n_el / world) * (world - 1)
            apply_info.update({"mode": "data parallel: fused reduce-scatter + step + all-gather over peer memory",
                               "link_bytes_in_per_replica": link_in, "link_gbs_in": link_in / (ms_apply * 1e-3) / 1e9,
                               "frac_of_measured_peer_copy_770": link_in / (ms_apply * 1e-3) / 1e9 / 770.0})
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    ms_e2e = None if brief else timed(step_e2e, e2e_steps) / e2e_steps
    if stage.status() != (0, 0):
        raise SystemExit(f"device status {stage.status()}")
    model_flops, hw_flops = lm_flops_per_step(w)
    value = whole_job_value(T, world, ms_step)
    line = {
        "metric": "small-LM training step tokens/s", "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
        "ms_per_step_median": statistics.median(per_step), "ms_per_step_best": min(per_step), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "d_model": d, "heads": f"{w.n_heads}x{w.head_dim}", "d_ff": w.d_ff,
                   "seq_len": w.seq_len, "batch": w.batch, "layers": L, "vocab": V, "recompute": bool(w.recompute),
                   "lean_ctx": bool(args.lean), "workspace_bytes": int(workspace.numel()),
                   "dispatch": "async",
                   "parallelism": (f"data parallel x{world} (gradients summed and applied through peer memory)"
                                   if args.data_parallel else f"replicas x{world}"),
                   "l2": "working set per step (logits alone are 1 GB) is far above the 126 MB L2"},
        "loss": loss_after_timed,
        "tflops_model": world * model_flops / (ms_step * 1e-3) / 1e12,
        "tflops_hw": world * hw_flops / (ms_step * 1e-3) / 1e12,
        "frac_bf16_peak_burst": hw_flops / (ms_step * 1e-3) / 1e12 / peaks["bf16_tflops"],
        "frac_bf16_peak_sustained": hw_flops / (ms_step * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
        "frac_bf16_nominal_2250": hw_flops / (ms_step * 1e-3) / 1e12 / 2250.0,   # datasheet dense bf16, for context
        "peaks": peaks, "clocks": clocks.summary(),
        "e2e": None if brief else {
            "value": world * T / (ms_e2e * 1e-3), "unit": "tokens/s", "ms_per_step": ms_e2e, "steps": e2e_steps,
            "how": "pinned host ids, labels -> device and the loss -> pinned host every step",
            "h2d_bytes_per_step": 2 * T * 4, "d2h_bytes_per_step": 4},
        "gpu_launches": int(launches),
    }
    if brief:
        del line["e2e"], line["peaks"]
    if apply_info is not None:
        line["metric"] = "small-LM training step with gradient apply tokens/s"
        line["apply"] = apply_info
    kernels, tot_ms = {}, sum(v["ms"] for v in prof.values())
    g_ms = g_flops = g_n = 0.0
    for name, v in prof.items():
        if v["launches"] == 0:
            continue
        k = {"launches_per_step": v["launches"] / args.steps, "ms_per_step": v["ms"] / args.steps, "share": v["ms"] / tot_ms}
        if v["flops"] > 0:
            k["tflops"] = v["flops"] / (v["ms"] * 1e-3) / 1e12
            k["frac_of_measured_bf16_burst"] = k["tflops"] / peaks["bf16_tflops"]
        if v["bytes"] > 0:
            k["gbs"] = v["bytes"] / (v["ms"] * 1e-3) / 1e9
            k["frac_of_measured_hbm"] = k["gbs"] / peaks["hbm_gbs"]
        kernels[name] = k
        if name.startswith("gemm"):
            g_ms += v["ms"]; g_flops += v["flops"]; g_n += v["launches"]
    line["kernels"] = kernels
    ms_apply_step = apply_info["ms_per_step_alone"] if apply_info is not None else 0.0
    line["roofline"] = gemm_roofline(g_flops, g_ms, g_n, tot_ms, ms_one_stream - ms_apply_step, args.steps, peaks,
                                     "gemm_pair_kernel (tcgen05 bf16 GEMM: layers and tied head)", None)
    line["ms_per_step_one_stream"] = ms_one_stream
    if rank == 0 and world == 1 and not brief and not args.no_cpu_baseline:
        import oracle as oracle_mod
        orc = oracle_mod.Oracle("f32")
        ws, D, pls, E_, g_, b_, ids_, labels_ = oracle_lm_sample(w, 1)
        t0 = time.perf_counter()
        orc.lm_step(D, pls, E_, g_, b_, ids_, labels_)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": ws.tokens / dt, "unit": "tokens/s", "cores": oracle_mod.host_threads(), "kind": "oracle",
                                "seconds": dt, "sample": f"1 of {w.batch} sequences (S={w.seq_len}) through 1 of {L} layers and the full-vocabulary head, fwd+bwd, fp32 plain-loop C oracle, run once"}
    if replica is not None:
        replica.close()
    return line if rank == 0 else None


def run_reference_lm(args, w):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle as oracle_mod
    orc = oracle_mod.Oracle("f32")
    ws, D, pls, E, g, b, ids, labels = oracle_lm_sample(w, 1)
    for _ in range(min(args.warmup, 1)):
        orc.lm_step(D, pls, E, g, b, ids, labels)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        orc.lm_step(D, pls, E, g, b, ids, labels)
    dt = time.perf_counter() - t0
    value = ws.tokens * args.steps / dt
    sample = f"1 of {w.batch} sequences (S={w.seq_len}) through 1 of {w.n_layers} layers and the full-vocabulary head per step, fp32 plain-loop C oracle"
    print(json.dumps({
        "impl": "reference", "metric": "small-LM training step tokens/s", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": oracle_mod.host_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=2, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--dispatch", default="async", choices=["opbyop", "async", "graph"])
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--e2e-steps", type=int, default=30)
    ap.add_argument("--cpu-sample-batch", type=int, default=6, help="sequences of the workload the timed oracle run processes (about 13 s of host time on workload 2)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-isolated", action="store_true", help="skip the back-to-back timing of the element-wise kernels")
    ap.add_argument("--no-sustained", action="store_true", help="skip the long back-to-back run of the step (sustained clocks)")
    ap.add_argument("--sustained-steps", type=int, default=600, help="steps of the sustained run (workload 2: about 1.4 s)")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="default run only: skip the short runs of workloads 3, 4, 5 and the dispatch study")
    ap.add_argument("--lean", action="store_true",
                    help="lean save set: the forward keeps neither LayerNorm output nor GeLU(u); the backward re-derives them")
    ap.add_argument("--data-parallel", action="store_true",
                    help="with --apply-lr: the ranks are data-parallel replicas; gradients are summed and applied through peer "
                         "memory by the fused kernel (each rank draws its own token batch)")
    ap.add_argument("--apply-lr", type=float, default=None,
                    help="workload 5 only: every step also applies the gradients (plain SGD, this rate) to all parameters")
    args = ap.parse_args()
    from paper_2203_12533_b200 import inputs
    w = inputs.WORKLOADS[args.workload]
    if args.apply_lr is not None and (not w.vocab or args.impl != "ours" or args.apply_lr < 0):
        raise SystemExit("--apply-lr needs --workload 5, --impl ours and a rate >= 0")
    if args.data_parallel and args.apply_lr is None:
        raise SystemExit("--data-parallel needs --apply-lr")
    if args.impl == "reference":
        (run_reference_lm if w.vocab else run_reference)(args, w)
        return
    line = (run_ours_lm if w.vocab else run_ours)(args, w)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if line is not None and world == 1 and args.workload == 2 and not args.no_other_workloads and not args.lean \
            and args.dispatch == "async":
        line["other_workloads"] = other_workloads(args)
        line["dispatch"] = dispatch_table()
    if line is not None:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()


# Steps (warm-up, timed) of the short runs of the other workloads inside the default run.
OTHER_WORKLOAD_STEPS = {3: (1, 2), 4: (3, 10), 5: (3, 10)}


def other_workloads(args):
    """Short device-resident runs of workloads 3, 4 and 5 (the large configurations and the small-LM
    step), each with its per-class kernel table and its own clock record.  They ride on the default
    line so that one run of this file shows every configuration; the headline fields stay workload 2's."""
    import copy
    import gc
    import torch
    from paper_2203_12533_b200 import inputs
    out = {}
    for wid, (warm, steps) in OTHER_WORKLOAD_STEPS.items():
        a = copy.copy(args)
        a.warmup, a.steps, a.workload = warm, steps, wid
        w = inputs.WORKLOADS[wid]
        gc.collect()
        torch.cuda.empty_cache()
        t0 = time.perf_counter()
        try:
            r = (run_ours_lm if w.vocab else run_ours)(a, w, brief=True)
        except SystemExit as e:                      # a device status other than 0: report it, keep the headline
            out[f"workload_{wid}"] = {"workload": w.name, "error": str(e)}
            continue
        keep = ("metric", "value", "unit", "steps", "warmup", "ms_per_step", "ms_per_step_best", "tflops_model", "tflops_hw",
                "frac_bf16_peak_burst", "frac_bf16_peak_sustained", "clocks", "gpu_launches", "kernels", "roofline", "loss",
                "config")
        o = {k: r[k] for k in keep if k in r}
        o["wall_s"] = time.perf_counter() - t0
        out[f"workload_{wid}"] = o
    gc.collect()
    torch.cuda.empty_cache()
    return out


def dispatch_table():
    """The dispatch study (Section 5.1 analogue): OPBYOP / ASYNC / GRAPH over a chain of small layer calls."""
    from paper_2203_12533_b200 import dispatch_study
    rows = dispatch_study.study(seq_lens=(128, 256, 512, 1024, 2048), layers=8, microbatches=8, reps=10)
    return {"what": "chain of 8 layers x 8 micro-batches at workload 1's width (recompute on): microseconds per layer call "
                    "(forward or backward) in each dispatch mode of pw_stage_run_chain; the whole_layer columns are the same chain with "
                    "PW_FLAG_WHOLE_LAYER (one cooperative launch per layer call), for the shapes that path serves",
            "rows": rows}


if __name__ == "__main__":
    main()
