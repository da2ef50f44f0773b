"""Single-GPU analogue of the paper's dispatch micro-benchmark (Section 5.1, Figures 5 and 6).

The paper compares three ways of issuing a chain of small computations - one synchronous call
per computation (OpByOp), one asynchronous call per computation (Chained) and the whole chain as
one program (Fused) - and asks how long a computation must run before the host-side cost is
hidden.  Here a computation is one decoder-layer call (forward + backward on one micro-batch) and
the three modes are the dispatch modes of ``pw_stage_run_chain``: OPBYOP (synchronise after
every layer call), ASYNC (enqueue everything) and GRAPH (one captured CUDA graph, replayed).

    python -m paper_2203_12533_b200.dispatch_study [--layers 8] [--microbatches 8] [--reps 20]

prints one JSON line per (sequence length, mode): layer calls per second and microseconds per
call, for a chain of ``layers`` x ``microbatches`` x 2 calls at the width of workload 1.  Where the
shape allows it, each mode is also run with PW_FLAG_WHOLE_LAYER (a layer call is then one kernel
launch instead of 7 or 15): the step the paper's Fused mode takes one level further down.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as pw
from . import inputs


WHOLE_LAYER_MAX_SEQ = 1024


def run(seq_len: int, layers: int, microbatches: int, reps: int, mode: int, flags: int = 0) -> float:
    """Milliseconds per chain (L x M forward calls + L x M backward calls)."""
    w = inputs.WORKLOADS[1].with_(seq_len=seq_len, n_layers=layers, n_microbatches=microbatches)
    dev = torch.device("cuda")
    stage = pw.Stage(layers, w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch, flags=flags)
    params = [[p.to(dev) for p in inputs.layer_params(w, 0, l)] for l in range(layers)]
    grads = [[torch.zeros(p.shape, dtype=torch.float32, device=dev) for p in ps] for ps in params]
    xs, dys = [], []
    for m in range(microbatches):
        x, dy = inputs.microbatch(w, 0, m)
        xs.append(x.view(w.tokens, -1).to(dev))
        dys.append(dy.view(w.tokens, -1).to(dev))
    ys = [torch.empty_like(t) for t in xs]
    dxs = [torch.empty_like(t) for t in xs]
    ws = torch.empty(stage.workspace_bytes(microbatches, pw.SCHEDULE_GPIPE, True), dtype=torch.uint8, device=dev)
    stream = torch.cuda.Stream()

    def chain():
        stage.run_chain(params, grads, xs, dys, ys, dxs, ws, mode, pw.SCHEDULE_GPIPE, True, stream=stream)

    with torch.cuda.stream(stream):
        for _ in range(3):
            chain()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            chain()
        e1.record(stream)
    torch.cuda.synchronize()
    assert stage.status() == (0, 0)
    return e0.elapsed_time(e1) / reps


def study(seq_lens=(128, 256, 512, 1024, 2048), layers=8, microbatches=8, reps=20):
    """One row per sequence length: microseconds per layer call in each dispatch mode."""
    pw.lib()
    modes = (("opbyop", pw.DISPATCH_OPBYOP), ("async", pw.DISPATCH_ASYNC), ("graph", pw.DISPATCH_GRAPH))
    calls = 2 * layers * microbatches
    rows = []
    for S in seq_lens:
        row = {"seq_len": S, "tokens_per_call": 2 * S}
        for name, mode in modes:
            row[f"us_per_layer_call_{name}"] = 1e3 * run(S, layers, microbatches, reps, mode) / calls
        row["graph_vs_opbyop"] = row["us_per_layer_call_opbyop"] / row["us_per_layer_call_graph"]
        if S <= WHOLE_LAYER_MAX_SEQ:
            for name, mode in modes:
                row[f"us_per_layer_call_whole_layer_{name}"] = 1e3 * run(S, layers, microbatches, reps, mode, pw.FLAG_WHOLE_LAYER) / calls
        rows.append(row)
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=8)
    ap.add_argument("--microbatches", type=int, default=8)
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--seq-lens", type=int, nargs="+", default=[128, 256, 512, 1024, 2048])
    args = ap.parse_args()
    pw.lib()
    modes = (("opbyop", pw.DISPATCH_OPBYOP), ("async", pw.DISPATCH_ASYNC), ("graph", pw.DISPATCH_GRAPH))
    for S in args.seq_lens:
        for flags in (0, pw.FLAG_WHOLE_LAYER):
            if flags and S > WHOLE_LAYER_MAX_SEQ:
                continue
            for name, mode in modes:
                ms = run(S, args.layers, args.microbatches, args.reps, mode, flags)
                calls = 2 * args.layers * args.microbatches
                print(json.dumps({"seq_len": S, "tokens_per_call": 2 * S, "mode": name, "whole_layer": bool(flags), "ms_per_chain": ms,
                                  "us_per_layer_call": 1e3 * ms / calls, "layer_calls_per_s": calls / (ms * 1e-3)}), flush=True)


if __name__ == "__main__":
    main()
