"""GPU tests of the lean save set (PW_FLAG_LEAN_CTX): the forward keeps neither LayerNorm output nor
GeLU(u); the backward re-derives them.  Against the oracle (same tolerances as the full save set)
and against the full-save layer (everything that does not pass through the re-derived GeLU output
must be bit-identical)."""
import numpy as np
import pytest
import torch

from paper_2203_12533_b200 import inputs
from tests.gpu_util import ACT_TOL, GRAD_TOL, dims_of, np64, rel_l2, run_layer_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pw():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2203_12533_b200 import binding
    binding.lib()
    return binding


def _layer(pw, w, flags, act=0):
    return pw.Layer(w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch, act=act, flags=flags)


def _run(pw, layer, params, x, dy, save_ctx=True, poison_scratch=False):
    T, d = layer.T, layer.d
    y, dx = torch.empty((T, d), dtype=torch.bfloat16, device="cuda"), torch.empty((T, d), dtype=torch.bfloat16, device="cuda")
    ctx = torch.empty(layer.ctx_bytes, dtype=torch.uint8, device="cuda") if save_ctx else None
    scratch = torch.empty(layer.scratch_bytes, dtype=torch.uint8, device="cuda")
    grads = [torch.full(p.shape, float("nan"), dtype=torch.float32, device="cuda") for p in params]
    layer.fwd(params, x, y, ctx, scratch)
    if poison_scratch:
        torch.cuda.synchronize()
        scratch.fill_(0xFF)                                   # NaN patterns: nothing of the forward may be read from here
    layer.bwd(params, x, dy, dx, grads, False, ctx, scratch)
    torch.cuda.synchronize()
    assert layer.status() == (0, 0)
    return y, dx, grads


@pytest.mark.parametrize("act", [0, 1], ids=["erf", "tanh"])
def test_lean_layer_against_oracle_and_full_save_set(pw, oracle64, act):
    from oracle import Dims
    w = inputs.Workload("lean_small", 512, 4, 128, 2048, 256, 3)
    D = dims_of(w)
    D = Dims(D.B, D.S, D.d, D.H, D.dh, D.F, D.eps, act)
    cpu = inputs.layer_params(w, 0, 0, random_ln=True)
    params = [p.cuda() for p in cpu]
    x, dy = inputs.microbatch(w, 0, 0)
    xd, dyd = x.cuda().view(-1, w.d_model), dy.cuda().view(-1, w.d_model)
    full, lean = _layer(pw, w, 0, act), _layer(pw, w, pw.FLAG_LEAN_CTX, act)
    T, d, F = w.tokens, w.d_model, w.d_ff
    assert full.ctx_bytes - lean.ctx_bytes == (2 * T * d + T * F) * 2          # h1, h2 and a are not kept
    assert lean.scratch_bytes > full.scratch_bytes
    with pytest.raises(KeyError):
        lean.ctx_view(torch.empty(lean.ctx_bytes, dtype=torch.uint8, device="cuda"), "a")
    y0, dx0, g0 = _run(pw, full, params, xd, dyd)
    y1, dx1, g1 = _run(pw, lean, params, xd, dyd, poison_scratch=True)
    assert torch.equal(y0, y1) and torch.equal(dx0, dx1)                        # neither passes through the re-derived tensors
    for name, a, b in zip(pw.PARAM_NAMES, g0, g1):
        if name == "w_fc2":                                                     # dW2 = dy^T GeLU(u): u is bf16 the second time
            assert rel_l2(b, np64(a)) < 6e-3                            # one bf16 rounding of u (2^-9) through GeLU
        else:
            assert torch.equal(a, b), name
    ps = [np64(p) for p in cpu]
    yw, sv = oracle64.layer_fwd(D, ps, np64(x))
    dxw, gw = oracle64.layer_bwd(D, ps, np64(x), sv, np64(dy))
    assert rel_l2(y1, yw) < ACT_TOL and rel_l2(dx1, dxw) < GRAD_TOL
    errs = {n: rel_l2(g, want) for n, g, want in zip(pw.PARAM_NAMES, g1, gw)}
    assert max(errs.values()) < GRAD_TOL, errs
    # without a ctx (recompute inside the backward) the GeLU output comes from the forward kernel
    # again: bit-identical to the full save set
    y2, dx2, g2 = _run(pw, lean, params, xd, dyd, save_ctx=False)
    assert torch.equal(y2, y0) and torch.equal(dx2, dx0)
    for a, b in zip(g0, g2):
        assert torch.equal(a, b)


def test_lean_layer_needs_scratch_in_the_forward(pw):
    w = inputs.Workload("lean_tiny", 256, 2, 128, 512, 128, 1)
    lean = _layer(pw, w, pw.FLAG_LEAN_CTX)
    params = [p.cuda() for p in inputs.layer_params(w, 0, 0)]
    x = torch.zeros((w.tokens, w.d_model), dtype=torch.bfloat16, device="cuda")
    y = torch.empty_like(x)
    ctx = torch.empty(lean.ctx_bytes, dtype=torch.uint8, device="cuda")
    with pytest.raises(pw.PwError):
        lean.fwd(params, x, y, ctx, None)
    with pytest.raises(pw.PwError):
        pw.Layer(w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch, flags=2)   # unknown flag


def test_lean_chain_and_lm_step_follow_the_full_save_set(pw):
    """Three layers, two micro-batches (GPipe, activations kept): outputs and input gradients are
    bit-identical to the full save set, the workspace is smaller; the small LM step gives the same
    loss and the same embedding gradient."""
    w = inputs.Workload("lean_chain", 256, 2, 128, 1024, 128, 2, n_layers=3, n_microbatches=2)
    L, M = w.n_layers, w.n_microbatches
    params = [[p.cuda() for p in inputs.layer_params(w, 0, l, random_ln=True)] for l in range(L)]
    mbs = [inputs.microbatch(w, 0, m) for m in range(M)]
    xs, dys = [x.cuda() for x, _ in mbs], [dy.cuda() for _, dy in mbs]
    res = {}
    for flags in (0, pw.FLAG_LEAN_CTX):
        stage = pw.Stage(L, w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch, flags=flags)
        nbytes = stage.workspace_bytes(M, pw.SCHEDULE_GPIPE, False)
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        grads = [[torch.full(p.shape, float("nan"), dtype=torch.float32, device="cuda") for p in ps] for ps in params]
        ys, dxs = [torch.empty_like(x) for x in xs], [torch.empty_like(x) for x in xs]
        stage.run_chain(params, grads, xs, dys, ys, dxs, ws, schedule=pw.SCHEDULE_GPIPE, recompute=False)
        torch.cuda.synchronize()
        assert stage.status() == (0, 0)
        res[flags] = (nbytes, ys, dxs, grads)
    T, d, F = w.tokens, w.d_model, w.d_ff
    saved = L * M * (2 * T * d + T * F) * 2
    assert res[0][0] - res[1][0] > 0.8 * saved                                  # most of it (scratch grows once, not L * M times)
    for a, b in zip(res[0][1] + res[0][2], res[1][1] + res[1][2]):
        assert torch.equal(a, b)
    for ga, gb in zip(res[0][3], res[1][3]):
        for name, a, b in zip(pw.PARAM_NAMES, ga, gb):
            if name == "w_fc2":
                assert rel_l2(b, np64(a)) < 6e-3                            # one bf16 rounding of u (2^-9) through GeLU
            else:
                assert torch.equal(a, b), name

    wl = inputs.Workload("lean_lm", 256, 4, 64, 1024, 128, 2, n_layers=2, vocab=512)
    lp = [[p.cuda() for p in inputs.layer_params(wl, 0, l, random_ln=True)] for l in range(wl.n_layers)]
    E, g, b, ids, labels = [t.cuda() for t in inputs.lm_inputs(wl, 0, random_ln=True)]
    out = {}
    for flags in (0, pw.FLAG_LEAN_CTX):
        stage = pw.Stage(wl.n_layers, wl.d_model, wl.n_heads, wl.head_dim, wl.d_ff, wl.seq_len, wl.batch, flags=flags)
        grads = [[torch.zeros(p.shape, device="cuda") for p in ps] for ps in lp]
        eg = [torch.zeros(E.shape, device="cuda"), torch.zeros(g.shape, device="cuda"), torch.zeros(b.shape, device="cuda")]
        loss = torch.zeros(1, device="cuda")
        ws = torch.empty(stage.lm_workspace_bytes(wl.vocab, False), dtype=torch.uint8, device="cuda")
        stage.lm_step(lp, grads, (E, g, b), eg, ids, labels, loss, wl.vocab, ws, False)
        torch.cuda.synchronize()
        assert stage.status() == (0, 0)
        out[flags] = (loss.item(), eg[0], ws.numel())
    assert out[0][0] == out[1][0] and torch.equal(out[0][1], out[1][1]) and out[1][2] < out[0][2]


def test_lean_chain_as_a_captured_graph_matches_the_stream_run(pw):
    """The lean backward's extra kernels sit on the side stream; captured into a CUDA graph and
    replayed twice they give the same bits as the plain asynchronous run."""
    w = inputs.Workload("lean_graph", 256, 2, 128, 1024, 128, 2, n_layers=2, n_microbatches=2)
    L, M = w.n_layers, w.n_microbatches
    params = [[p.cuda() for p in inputs.layer_params(w, 0, l, random_ln=True)] for l in range(L)]
    mbs = [inputs.microbatch(w, 0, m) for m in range(M)]
    xs, dys = [x.cuda() for x, _ in mbs], [dy.cuda() for _, dy in mbs]
    stage = pw.Stage(L, w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch, flags=pw.FLAG_LEAN_CTX)
    ws = torch.empty(stage.workspace_bytes(M, pw.SCHEDULE_GPIPE, False), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    outs = []
    for mode, reps in ((pw.DISPATCH_ASYNC, 1), (pw.DISPATCH_GRAPH, 2)):
        grads = [[torch.full(p.shape, float("nan"), dtype=torch.float32, device="cuda") for p in ps] for ps in params]
        ys, dxs = [torch.empty_like(x) for x in xs], [torch.empty_like(x) for x in xs]
        with torch.cuda.stream(stream):
            for _ in range(reps):
                stage.run_chain(params, grads, xs, dys, ys, dxs, ws, dispatch=mode, schedule=pw.SCHEDULE_GPIPE,
                                recompute=False, stream=stream)
        torch.cuda.synchronize()
        assert stage.status() == (0, 0)
        outs.append((ys, dxs, grads))
    for a, b in zip(outs[0][0] + outs[0][1], outs[1][0] + outs[1][1]):
        assert torch.equal(a, b)
    for ga, gb in zip(outs[0][2], outs[1][2]):
        for a, b in zip(ga, gb):
            assert torch.equal(a, b)
