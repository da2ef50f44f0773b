"""GPU parity of the whole layer and of the stage chain (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2203_12533_b200 import inputs
from tests.gpu_util import (ACT_TOL, GRAD_TOL, dims_of, elem_check, make_layer, np64, rel_l2, run_layer_gpu)

# Element bounds for a whole layer.  Inside the layer the GPU path hands bf16 tensors from step to step
# while the oracle keeps full precision, so an element differs by more than one output rounding: the
# attention output of a position that sees only a few keys is as sensitive to the rounding of q and k as
# a single softmax weight is (measured at workload-3 width: worst element 0.08 rms, 99.99 % below 0.04
# rms, against 0.04 / 0.02 rms when the oracle is given the GPU's own qkv).  A mis-computed tile is off
# by about one rms in every element, so these bounds still catch what the norm hides.  The single-step
# tests (test_gpu_ops.py) use the tight bounds.
LAYER_ACT = dict(atol_rms=0.2, rtol=2.0 ** -6)
LAYER_GRAD = dict(atol_rms=0.3, rtol=2.0 ** -5)
# statistics: a row mean is itself of size rms(x) / sqrt(d), and so is its error when x carries bf16
# roundings - relative to the rms of the means that is a few 2^-9; 1 / sigma and lse move far less
ELEM_STAT = dict(atol_rms=2e-3, rtol=2e-3)
ELEM_MEAN = dict(atol_rms=2e-2, rtol=2e-3)

pytestmark = pytest.mark.gpu

SAVED_BF16 = ("h1", "qkv", "o", "x1", "h2", "u", "a")


@pytest.fixture(scope="module")
def pw():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2203_12533_b200 import binding
    binding.lib()
    return binding


def check_layer_against_oracle(pw, oracle, w, random_ln=False, act=0, save_ctx=True, flags=0):
    from oracle import Dims
    D = dims_of(w)
    D = Dims(D.B, D.S, D.d, D.H, D.dh, D.F, D.eps, act)
    params = inputs.layer_params(w, seed=0, layer=0, random_ln=random_ln)
    x, dy = inputs.microbatch(w, seed=0, m=0)
    layer = make_layer(pw, w, act, flags)
    out = run_layer_gpu(pw, layer, [p.cuda() for p in params], x.cuda().view(-1, w.d_model),
                        dy.cuda().view(-1, w.d_model), save_ctx=save_ctx)
    cast = (lambda t: t.float().numpy()) if oracle.suf == "f32" else np64
    ps = [cast(p) for p in params]
    yw, sv = oracle.layer_fwd(D, ps, cast(x))
    dxw, gw = oracle.layer_bwd(D, ps, cast(x), sv, cast(dy))
    errs = {"y": rel_l2(out["y"], yw)}
    worst = {"y": elem_check(out["y"], yw, "y", **LAYER_ACT)}
    store = out["ctx"] if save_ctx else out["scratch"]
    for name in SAVED_BF16:
        errs[name] = rel_l2(layer.ctx_view(store, name), sv[name])
        worst[name] = elem_check(layer.ctx_view(store, name), sv[name], name, **LAYER_ACT)
    for name in ("lse", "mu1", "r1", "mu2", "r2"):
        errs[name] = rel_l2(layer.ctx_view(store, name), sv[name])
        worst[name] = elem_check(layer.ctx_view(store, name), sv[name], name, **(ELEM_MEAN if name.startswith("mu") else ELEM_STAT))
    gerrs = {"dx": rel_l2(out["dx"], dxw)}
    worst["dx"] = elem_check(out["dx"], dxw, "dx", **LAYER_GRAD)
    for name, g, want in zip(pw.PARAM_NAMES, out["grads"], gw):
        gerrs["d" + name] = rel_l2(g, want)
        worst["d" + name] = elem_check(g, want, "d" + name, **LAYER_GRAD)
    assert max(errs.values()) < ACT_TOL, errs
    assert max(gerrs.values()) < GRAD_TOL, gerrs
    print("worst element ratios:", {k: round(v, 3) for k, v in worst.items()})
    return errs, gerrs


def test_cfg1_parity_all_tensors(pw, oracle64):
    check_layer_against_oracle(pw, oracle64, inputs.WORKLOADS[1])


def test_random_layernorm_params_and_tanh_gelu(pw, oracle64):
    w = inputs.Workload("ragged", 512, 4, 128, 1152, 256, 3, sigma_w=0.05)    # T = 768, F not a multiple of 256
    check_layer_against_oracle(pw, oracle64, w, random_ln=True)
    check_layer_against_oracle(pw, oracle64, w, random_ln=True, act=1)


def test_midsize_dh64(pw, oracle64):
    w = inputs.Workload("mid", 768, 12, 64, 3072, 384, 2, sigma_w=0.03)
    check_layer_against_oracle(pw, oracle64, w, random_ln=True)


def test_recompute_matches_saved_bitwise_and_is_deterministic(pw):
    w = inputs.WORKLOADS[1].with_(seq_len=256)
    params = [p.cuda() for p in inputs.layer_params(w, random_ln=True)]
    x, dy = inputs.microbatch(w)
    x, dy = x.cuda().view(-1, w.d_model), dy.cuda().view(-1, w.d_model)
    layer = make_layer(pw, w)
    a = run_layer_gpu(pw, layer, params, x, dy, save_ctx=True)
    b = run_layer_gpu(pw, layer, params, x, dy, save_ctx=False)     # backward re-runs the forward into scratch
    c = run_layer_gpu(pw, layer, params, x, dy, save_ctx=True)
    for other in (b, c):
        assert torch.equal(a["y"], other["y"]) and torch.equal(a["dx"], other["dx"])
        for g1, g2 in zip(a["grads"], other["grads"]):
            assert torch.equal(g1, g2)


def test_accumulate_adds(pw):
    w = inputs.WORKLOADS[1]
    params = [p.cuda() for p in inputs.layer_params(w)]
    x, dy = inputs.microbatch(w)
    x, dy = x.cuda().view(-1, w.d_model), dy.cuda().view(-1, w.d_model)
    layer = make_layer(pw, w)
    one = run_layer_gpu(pw, layer, params, x, dy)
    acc = run_layer_gpu(pw, layer, params, x, dy, grads=[g.clone() for g in one["grads"]], accumulate=True)
    for g1, g2 in zip(one["grads"], acc["grads"]):
        assert rel_l2(g2, 2 * g1.double()) < 1e-6


def test_dx_may_alias_dy(pw):
    w = inputs.WORKLOADS[1]
    params = [p.cuda() for p in inputs.layer_params(w)]
    x, dy = inputs.microbatch(w)
    x, dy = x.cuda().view(-1, w.d_model), dy.cuda().view(-1, w.d_model)
    layer = make_layer(pw, w)
    ref = run_layer_gpu(pw, layer, params, x, dy)
    y = torch.empty_like(x)
    ctx = torch.empty(layer.ctx_bytes, dtype=torch.uint8, device="cuda")
    scratch = torch.empty(layer.scratch_bytes, dtype=torch.uint8, device="cuda")
    g = dy.clone()
    grads = [torch.empty_like(t) for t in ref["grads"]]
    layer.fwd(params, x, y, ctx, scratch)
    layer.bwd(params, x, g, g, grads, False, ctx, scratch)
    torch.cuda.synchronize()
    assert torch.equal(g, ref["dx"])


def test_layer_argument_errors(pw):
    w = inputs.WORKLOADS[1]
    layer = make_layer(pw, w)
    params = [p.cuda() for p in inputs.layer_params(w)]
    x = torch.zeros((w.tokens, w.d_model), dtype=torch.bfloat16, device="cuda")
    y = torch.empty_like(x)
    ctx = torch.empty(layer.ctx_bytes, dtype=torch.uint8, device="cuda")
    scratch = torch.empty(layer.scratch_bytes + 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(pw.PwError) as e:
        layer.fwd(params, x, x, ctx, scratch)                      # y aliases x
    assert e.value.status == 1
    with pytest.raises(pw.PwError):
        layer.fwd(params, x, y, ctx[8:], scratch)                  # misaligned ctx
    with pytest.raises(pw.PwError):
        layer.fwd(params[:11] + [None], x, y, ctx, scratch)        # missing parameter
    grads = [torch.zeros(p.shape, dtype=torch.float32, device="cuda") for p in params]
    with pytest.raises(pw.PwError):
        layer.bwd(params, x, y, y, grads, 2, ctx, scratch)         # accumulate must be 0/1
    with pytest.raises(pw.PwError):
        pw.Layer(2048, 16, 128, 8192, 1000, 8)                     # unsupported shape, no fallback
    assert layer.status() == (0, 0)


@pytest.mark.parametrize("d,H,F,S", [(4096, 32, 16384, 256), (8192, 64, 32768, 128)], ids=["cfg3_width", "cfg4_width"])
def test_wide_layers_at_reduced_token_count(pw, oracle32, d, H, F, S):
    """The layer widths of workloads 3 and 4 (d = 4096 / 8192, 128-wide heads) on fewer tokens."""
    sigma = 0.01 if d == 8192 else 0.02
    w = inputs.Workload("wide", d, H, 128, F, S, 2 if d == 4096 else 1, sigma_w=sigma)
    check_layer_against_oracle(pw, oracle32, w)


# ------------------------------------------------------------------------------------------ stage chain
def run_chain_gpu(pw, w, L, M, dispatch, schedule, recompute, seed=0, random_ln=True, mbs=None, flags=0, counts=None):
    stage = pw.Stage(L, w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch, flags=flags)
    params = [[p.cuda() for p in inputs.layer_params(w, seed, l, random_ln=random_ln)] for l in range(L)]
    grads = [[torch.full(p.shape, float("nan"), dtype=torch.float32, device="cuda") for p in ps] for ps in params]
    if mbs is None:
        mbs = [inputs.microbatch(w, seed, m) for m in range(M)]
    xs = [x.cuda().view(-1, w.d_model) for x, _ in mbs]
    dys = [dy.cuda().view(-1, w.d_model) for _, dy in mbs]
    ys = [torch.empty_like(x) for x in xs]
    dxs = [torch.empty_like(x) for x in xs]
    ws = torch.empty(stage.workspace_bytes(M, schedule, recompute), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        reps = 2 if dispatch == pw.DISPATCH_GRAPH else 1           # second call replays the cached graph
        for _ in range(reps):
            stage.run_chain(params, grads, xs, dys, ys, dxs, ws, dispatch, schedule, recompute, stream=stream)
    torch.cuda.synchronize()
    assert stage.status() == (0, 0)
    if counts is not None:
        counts.append(stage.launch_count() // reps)
    return ys, dxs, grads


def test_chain_matches_oracle_and_modes_agree(pw, oracle64):
    w = inputs.WORKLOADS[1].with_(seq_len=256, batch=1)
    L, M = 3, 2
    D = dims_of(w)
    ref = run_chain_gpu(pw, w, L, M, pw.DISPATCH_ASYNC, pw.SCHEDULE_GPIPE, True)
    pls = [[np64(p) for p in inputs.layer_params(w, 0, l, random_ln=True)] for l in range(L)]
    mbs = [inputs.microbatch(w, 0, m) for m in range(M)]
    bf16_roundtrip = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).double().numpy()
    ys, dxs, grads = oracle64.chain(D, pls, [np64(x) for x, _ in mbs], [np64(dy) for _, dy in mbs],
                                    handoff=bf16_roundtrip)
    for m in range(M):
        assert rel_l2(ref[0][m], ys[m]) < ACT_TOL
        assert rel_l2(ref[1][m], dxs[m]) < GRAD_TOL
    for l in range(L):
        for name, g, want in zip(pw.PARAM_NAMES, ref[2][l], grads[l]):
            assert rel_l2(g, want) < GRAD_TOL, (l, name)
    # every dispatch mode, schedule and save mode gives the same bits (same kernels, same order per tensor)
    for dispatch, schedule, recompute in [(pw.DISPATCH_OPBYOP, pw.SCHEDULE_GPIPE, True),
                                          (pw.DISPATCH_GRAPH, pw.SCHEDULE_GPIPE, True),
                                          (pw.DISPATCH_ASYNC, pw.SCHEDULE_PER_MICROBATCH, True),
                                          (pw.DISPATCH_ASYNC, pw.SCHEDULE_GPIPE, False),
                                          (pw.DISPATCH_GRAPH, pw.SCHEDULE_PER_MICROBATCH, False)]:
        other = run_chain_gpu(pw, w, L, M, dispatch, schedule, recompute)
        for m in range(M):
            assert torch.equal(ref[0][m], other[0][m]) and torch.equal(ref[1][m], other[1][m]), (dispatch, schedule, recompute)
        for l in range(L):
            for g1, g2 in zip(ref[2][l], other[2][l]):
                assert torch.equal(g1, g2), (dispatch, schedule, recompute)


def test_chain_workspace_too_small_is_reported_before_launch(pw):
    w = inputs.WORKLOADS[1]
    stage = pw.Stage(2, w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch)
    params = [[p.cuda() for p in inputs.layer_params(w, 0, l)] for l in range(2)]
    grads = [[torch.zeros(p.shape, dtype=torch.float32, device="cuda") for p in ps] for ps in params]
    x = torch.zeros((w.tokens, w.d_model), dtype=torch.bfloat16, device="cuda")
    y, dy, dx = torch.empty_like(x), torch.zeros_like(x), torch.empty_like(x)
    need = stage.workspace_bytes(1)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    with pytest.raises(pw.PwError) as e:
        stage.run_chain(params, grads, [x], [dy], [y], [dx], ws, workspace_bytes=need - 1)
    assert e.value.status == 3


# ------------------------------------------------------------------------------------------ full benchmark size
def test_cfg2_full_size_parity(pw, oracle32):
    """The benchmark workload (d=2048, 16x128 heads, F=8192, S=1024, B=8) against the fp32 oracle."""
    check_layer_against_oracle(pw, oracle32, inputs.WORKLOADS[2])


def test_cfg5_layer_full_size_parity(pw, oracle32):
    """One layer of workload 5 at its full size (d=1024, 16x64 heads, F=4096, S=1024, B=16: the 64-wide
    heads in the launch configuration the benchmark times) against the fp32 oracle, every tensor."""
    check_layer_against_oracle(pw, oracle32, inputs.WORKLOADS[5].with_(n_layers=1, vocab=0))


# ------------------------------------------------------------------------------------------ full sizes of workloads 3 and 4
@pytest.mark.parametrize("wid", [3, 4], ids=["cfg3_layer_full_size", "cfg4_full_size"])
def test_full_size_wide_layer_by_the_causal_prefix_property(pw, oracle32, wid):
    """One layer of workloads 3 / 4 at its full size (B x 2048 tokens, d = 4096 / 8192), checked through a
    property that holds at any size: the model is causal and sequences are independent, so with an
    upstream gradient that is zero outside the first P tokens of every sequence, the outputs on
    those prefixes, their input gradients and ALL parameter gradients equal those of the problem
    truncated to P tokens per sequence - which the oracle can compute - and dx is exactly zero
    beyond the prefixes."""
    w = inputs.WORKLOADS[wid].with_(n_layers=1, n_microbatches=1)
    P = 64
    params = inputs.layer_params(w, 0, 0, random_ln=True)
    x, dy = inputs.microbatch(w, 0, 0)
    dy = dy.clone()
    dy[:, P:, :] = 0
    layer = make_layer(pw, w)
    out = run_layer_gpu(pw, layer, [p.cuda() for p in params], x.cuda().view(-1, w.d_model), dy.cuda().view(-1, w.d_model))
    y = out["y"].view(w.batch, w.seq_len, w.d_model)
    dx = out["dx"].view(w.batch, w.seq_len, w.d_model)
    assert torch.count_nonzero(dx[:, P:, :]) == 0
    wt = w.with_(seq_len=P)
    D = dims_of(wt)
    ps = [p.float().numpy() for p in params]
    xt = x[:, :P, :].float().numpy().reshape(-1, w.d_model)
    dyt = dy[:, :P, :].float().numpy().reshape(-1, w.d_model)
    yw, sv = oracle32.layer_fwd(D, ps, xt)
    dxw, gw = oracle32.layer_bwd(D, ps, xt, sv, dyt)
    assert rel_l2(y[:, :P, :].reshape(-1, w.d_model), yw) < ACT_TOL
    assert rel_l2(dx[:, :P, :].reshape(-1, w.d_model), dxw) < GRAD_TOL
    errs = {name: rel_l2(g, want) for name, g, want in zip(pw.PARAM_NAMES, out["grads"], gw)}
    assert max(errs.values()) < GRAD_TOL, errs


def test_cfg4_full_size_parity(pw, oracle32):
    """One layer of workload 4 at its full size (d = 8192, 64 x 128 heads, F = 32768, S = 2048, B = 1) against
    the fp32 oracle: every saved tensor, every gradient, all 2048 positions (norm and element bounds).
    The oracle needs about a minute and a half on 16 host cores."""
    check_layer_against_oracle(pw, oracle32, inputs.WORKLOADS[4].with_(n_layers=1, n_microbatches=1))


def test_cfg3_full_size_chain_one_microbatch(pw, oracle32):
    """Workload 3's stage at its full size - four layers d = 4096, 32 x 128 heads, F = 16384, 4 x 2048 tokens,
    activations recomputed, GPipe order, the launch configuration the benchmark times - on one of its
    micro-batches, against the fp32 oracle's chain with the same bf16 hand-off between layers.  To keep
    the oracle near four minutes on 16 host cores it computes two of the four sequences: the GPU run gets
    a zero upstream gradient for the other two, so every parameter gradient comes from the two compared
    sequences alone (sequences do not interact).  Compared: y and dx of those sequences at all 2048
    positions and all 48 parameter-gradient tensors, by norm and element by element; dx of the other
    two sequences must be exactly zero."""
    w = inputs.WORKLOADS[3]
    L, M, Bo = w.n_layers, 1, 2
    x, dy = inputs.microbatch(w, 0, 0)
    dy = dy.clone()
    dy[Bo:] = 0
    ys, dxs, grads = run_chain_gpu(pw, w, L, M, pw.DISPATCH_ASYNC, pw.SCHEDULE_GPIPE, True, random_ln=False, mbs=[(x, dy)])
    y = ys[0].view(w.batch, w.seq_len, w.d_model)
    dx = dxs[0].view(w.batch, w.seq_len, w.d_model)
    assert torch.count_nonzero(dx[Bo:]) == 0 and torch.isfinite(y.float()).all()
    wo = w.with_(batch=Bo)
    D = dims_of(wo)
    pls = [[p.float().numpy() for p in inputs.layer_params(w, 0, l)] for l in range(L)]
    f32 = lambda t: t[:Bo].float().numpy().reshape(wo.tokens, w.d_model)
    rt = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).float().numpy()
    yw, dxw, gw = oracle32.chain(D, pls, [f32(x)], [f32(dy)], handoff=rt)
    y2, dx2 = y[:Bo].reshape(wo.tokens, w.d_model), dx[:Bo].reshape(wo.tokens, w.d_model)
    assert rel_l2(y2, yw[0]) < ACT_TOL and rel_l2(dx2, dxw[0]) < GRAD_TOL
    worst = {"y": elem_check(y2, yw[0], "y", **LAYER_ACT), "dx": elem_check(dx2, dxw[0], "dx", **LAYER_GRAD)}
    for l in range(L):
        for name, g, want in zip(pw.PARAM_NAMES, grads[l], gw[l]):
            assert rel_l2(g, want) < GRAD_TOL, (l, name)
            worst[f"L{l}.d{name}"] = elem_check(g, want, f"layer {l} d{name}", **LAYER_GRAD)
    print("worst element ratios:", {k: round(v, 3) for k, v in worst.items()})


def test_single_tile_layer(pw, oracle64):
    """T = 128 tokens: one query tile per head (no second tile in the attention kernels), GEMMs on the one-CTA path."""
    w = inputs.Workload("single_tile", 256, 2, 128, 640, 128, 1)
    check_layer_against_oracle(pw, oracle64, w, random_ln=True)
    w = inputs.Workload("odd_tiles", 768, 12, 64, 384, 384, 1, sigma_w=0.03)    # S = 3 x 128: the last pair has one tile
    check_layer_against_oracle(pw, oracle64, w, random_ln=True, save_ctx=False)


def test_side_stream_switch_changes_no_bit(pw):
    """The backward pass with its weight-gradient GEMMs on the library's side stream (default) and
    with every kernel on the calling stream gives the same bits."""
    w = inputs.Workload("side", 512, 4, 128, 2048, 256, 4)
    params = [p.cuda() for p in inputs.layer_params(w, 0, 0, random_ln=True)]
    x, dy = inputs.microbatch(w, 0, 0)
    xd, dyd = x.cuda().view(-1, w.d_model), dy.cuda().view(-1, w.d_model)
    layer = make_layer(pw, w)
    a = run_layer_gpu(pw, layer, params, xd, dyd)
    layer.set_side_stream(False)
    b = run_layer_gpu(pw, layer, params, xd, dyd)
    layer.set_side_stream(True)
    c = run_layer_gpu(pw, layer, params, xd, dyd)
    for other in (b, c):
        assert torch.equal(a["y"], other["y"]) and torch.equal(a["dx"], other["dx"])
        for g0, g1 in zip(a["grads"], other["grads"]):
            assert torch.equal(g0, g1)
