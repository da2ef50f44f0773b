"""Times one single step of the layer in isolation, through the C ABI (pw_op_* calls).

    python -m paper_2203_12533_b200.opbench attention --batch 8 --seq 1024 --heads 16 --head-dim 128
    python -m paper_2203_12533_b200.opbench layernorm --tokens 8192 --width 2048
    python -m paper_2203_12533_b200.opbench colsum --tokens 8192 --width 8192
    python -m paper_2203_12533_b200.opbench gemm --layout tn --m 8192 --n 6144 --k 2048

Each step is launched `--iters` times back to back on one stream between two CUDA events, after
three warm-up launches; inputs rotate over `--sets` buffer sets so that HBM-bound steps read from
HBM and not from the 126 MB L2.  Only the operands of that one step are allocated, so the
process is small enough to put under a profiler (one kernel, a few launches).  Prints one JSON
line per step: microseconds per launch and TFLOP/s (attention: the visible causal pairs only;
GEMM: 2 M N K) or GB/s of algorithmic bytes.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as pw


def _time(fn, iters):
    for i in range(3):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters * 1e3          # microseconds


def _rand(shape, gen, scale=1.0):
    return (torch.randn(shape, generator=gen) * scale).to(torch.bfloat16).cuda()


def attention(args):
    B, S, H, dh = args.batch, args.seq, args.heads, args.head_dim
    d = H * dh
    g = torch.Generator().manual_seed(0)
    qkv, dout = _rand((B * S, 3 * d), g), _rand((B * S, d), g)
    o = torch.empty((B * S, d), dtype=torch.bfloat16, device="cuda")
    lse, delta = torch.empty((B, H, S), device="cuda"), torch.empty((B, H, S), device="cuda")
    dqkv = torch.empty_like(qkv)
    shape = {"batch": B, "seq": S, "heads": H, "head_dim": dh}
    us = _time(lambda i: pw.op_attention_fwd(qkv, B, S, H, dh, o, lse), args.iters)
    fl = 2.0 * B * S * (S + 1) * d
    print(json.dumps({"step": "attention_fwd", **shape, "us": us, "tflops": fl / us / 1e6}), flush=True)
    us = _time(lambda i: pw.op_attention_bwd(qkv, o, dout, lse, B, S, H, dh, dqkv, delta), args.iters)
    print(json.dumps({"step": "attention_bwd", **shape, "us": us, "tflops": 2.5 * fl / us / 1e6, "launches_per_call": 3}), flush=True)


def layernorm(args):
    T, d, n = args.tokens, args.width, args.sets
    g = torch.Generator().manual_seed(0)
    xs, dhs = [_rand((T, d), g) for _ in range(n)], [_rand((T, d), g) for _ in range(n)]
    hs = [torch.empty_like(x) for x in xs]
    gamma, beta = torch.ones(d, dtype=torch.bfloat16, device="cuda"), torch.zeros(d, dtype=torch.bfloat16, device="cuda")
    mu, rs = torch.empty(T, device="cuda"), torch.empty(T, device="cuda")
    outs = [torch.zeros(d, device="cuda") for _ in range(4)]
    part = torch.empty(pw.op_layernorm_bwd_scratch_bytes(T, d), dtype=torch.uint8, device="cuda")
    us = _time(lambda i: pw.op_layernorm_fwd(xs[i % n], gamma, beta, 1e-5, hs[i % n], mu, rs), args.iters)
    print(json.dumps({"step": "layernorm_fwd", "tokens": T, "width": d, "us": us, "gbs": (4.0 * T * d + 8.0 * T) / us / 1e3}), flush=True)
    us = _time(lambda i: pw.op_layernorm_bwd(dhs[i % n], xs[i % n], mu, rs, gamma, xs[(i + 1) % n], hs[i % n], outs[0], outs[1],
                                             outs[2], outs[3], False, part), args.iters)
    print(json.dumps({"step": "layernorm_bwd", "tokens": T, "width": d, "us": us, "gbs": (8.0 * T * d + 8.0 * T) / us / 1e3,
                      "launches_per_call": 2}), flush=True)


def colsum(args):
    T, N, n = args.tokens, args.width, args.sets
    g = torch.Generator().manual_seed(0)
    ins = [_rand((T, N), g) for _ in range(n)]
    out = torch.zeros(N, device="cuda")
    sc = torch.empty(pw.op_colsum_scratch_bytes(T, N), dtype=torch.uint8, device="cuda")
    us = _time(lambda i: pw.op_colsum(ins[i % n], out, False, sc), args.iters)
    print(json.dumps({"step": "colsum", "tokens": T, "width": N, "us": us, "gbs": 2.0 * T * N / us / 1e3, "launches_per_call": 2}), flush=True)


def gemm(args):
    M, N, K = args.m, args.n, args.k
    g = torch.Generator().manual_seed(0)
    layout = {"tn": pw.GEMM_TN, "nn": pw.GEMM_NN, "nt": pw.GEMM_NT}[args.layout]
    if layout == pw.GEMM_TN:
        A, lda, Bm, ldb = _rand((M, K), g), K, _rand((N, K), g, 0.1), K
    elif layout == pw.GEMM_NN:
        A, lda, Bm, ldb = _rand((M, K), g), K, _rand((K, N), g, 0.1), N
    else:
        A, lda, Bm, ldb = _rand((K, M), g), M, _rand((K, N), g, 0.1), N
    f32 = layout == pw.GEMM_NT
    C = torch.empty((M, N), dtype=torch.float32 if f32 else torch.bfloat16, device="cuda")
    us = _time(lambda i: pw.op_gemm(layout, pw.EPI_F32 if f32 else pw.EPI_NONE, M, N, K, A, lda, Bm, ldb, C, N), args.iters)
    print(json.dumps({"step": "gemm_" + args.layout, "m": M, "n": N, "k": K, "us": us, "tflops": 2.0 * M * N * K / us / 1e6}), flush=True)


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    sub = ap.add_subparsers(dest="step", required=True)
    a = sub.add_parser("attention")
    a.add_argument("--batch", type=int, default=8); a.add_argument("--seq", type=int, default=1024)
    a.add_argument("--heads", type=int, default=16); a.add_argument("--head-dim", type=int, default=128)
    for name in ("layernorm", "colsum"):
        s = sub.add_parser(name)
        s.add_argument("--tokens", type=int, default=8192); s.add_argument("--width", type=int, default=2048)
        s.add_argument("--sets", type=int, default=6)
    m = sub.add_parser("gemm")
    m.add_argument("--layout", default="tn", choices=["tn", "nn", "nt"])
    m.add_argument("--m", type=int, default=8192); m.add_argument("--n", type=int, default=6144); m.add_argument("--k", type=int, default=2048)
    for s in sub.choices.values():
        s.add_argument("--iters", type=int, default=20)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("opbench needs a CUDA device (there is no CPU fallback)")
    pw.lib()
    {"attention": attention, "layernorm": layernorm, "colsum": colsum, "gemm": gemm}[args.step](args)
    code, site = pw.op_status()
    if code != 0:
        raise SystemExit(f"device status {code} at site {site}")


if __name__ == "__main__":
    main()
