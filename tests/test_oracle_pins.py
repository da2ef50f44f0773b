"""Pins for the CPU oracle: it is checked against things other than itself.

Finite differences in double, fp64 library routines with autograd, closed
forms, invariants (causality, softmax rows, LayerNorm moments, linearity) and
the structure identity of Section 5.3.  None of these tests touches a GPU.
"""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import ACT_GELU_ERF, ACT_GELU_TANH, Dims, Oracle, PARAM_NAMES, SAVED_NAMES

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
TINY = Dims(B=2, S=6, d=16, H=2, dh=8, F=32)
SMALL = Dims(B=2, S=33, d=64, H=4, dh=16, F=96)
CFG1 = Dims(B=2, S=128, d=256, H=4, dh=64, F=1024)


def rand_params(D, rng, scale=0.2, random_ln=True):
    ps = []
    for i, shp in enumerate(D.param_shapes()):
        if i in (0, 6):
            ps.append(1.0 + 0.3 * rng.standard_normal(shp) if random_ln else np.ones(shp))
        elif i in (1, 7):
            ps.append(0.3 * rng.standard_normal(shp) if random_ln else np.zeros(shp))
        else:
            ps.append(scale * rng.standard_normal(shp))
    return ps


def rel(a, b):
    a = np.asarray(a, np.float64).ravel()
    b = np.asarray(b, np.float64).ravel()
    n = np.linalg.norm(b)
    return np.linalg.norm(a - b) / n if n > 1e-12 else np.linalg.norm(a - b)


# ----- the same layer written with library routines (fp64 torch CPU), differentiated by autograd -----
def torch_layer(D, ps, x, act=ACT_GELU_ERF):
    g1, b1, wqkv, bqkv, wo, bo, g2, b2, w1, bf1, w2, bf2 = ps
    xx = x.reshape(D.B, D.S, D.d)
    h1 = F.layer_norm(xx, (D.d,), g1, b1, D.eps)
    qkv = F.linear(h1, wqkv, bqkv)
    q, k, v = qkv.split(D.d, dim=-1)
    sh = lambda t: t.reshape(D.B, D.S, D.H, D.dh).transpose(1, 2)
    o = F.scaled_dot_product_attention(sh(q), sh(k), sh(v), is_causal=True)
    o = o.transpose(1, 2).reshape(D.B, D.S, D.d)
    x1 = xx + F.linear(o, wo, bo)
    h2 = F.layer_norm(x1, (D.d,), g2, b2, D.eps)
    u = F.linear(h2, w1, bf1)
    a = F.gelu(u, approximate="tanh" if act == ACT_GELU_TANH else "none")
    y = x1 + F.linear(a, w2, bf2)
    inter = dict(h1=h1, qkv=qkv, o=o, x1=x1, h2=h2, u=u, a=a)
    return y.reshape(D.T, D.d), inter


@pytest.mark.parametrize("D", [TINY, SMALL, CFG1], ids=["tiny", "small", "cfg1"])
@pytest.mark.parametrize("act", [ACT_GELU_ERF, ACT_GELU_TANH], ids=["erf", "tanh"])
def test_layer_matches_fp64_library_autograd(oracle64, D, act):
    if D is CFG1 and act == ACT_GELU_TANH:
        pytest.skip("one activation is enough at this size")
    rng = np.random.default_rng(1)
    D = Dims(D.B, D.S, D.d, D.H, D.dh, D.F, D.eps, act)
    ps = rand_params(D, rng, scale=0.5 / math.sqrt(D.d) * 4)
    x = rng.standard_normal((D.T, D.d))
    dy = rng.standard_normal((D.T, D.d))
    y, sv = oracle64.layer_fwd(D, ps, x)
    dx, gr = oracle64.layer_bwd(D, ps, x, sv, dy)

    tp = [torch.tensor(p, dtype=torch.float64, requires_grad=True) for p in ps]
    tx = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    ty, inter = torch_layer(D, tp, tx, act)
    ty.backward(torch.tensor(dy, dtype=torch.float64))
    assert rel(y, ty.detach().numpy()) < 1e-12
    for name, t in inter.items():
        assert rel(sv[name], t.detach().numpy().reshape(sv[name].shape)) < 1e-12, name
    assert rel(dx, tx.grad.numpy()) < 1e-11
    for name, g, t in zip(PARAM_NAMES, gr, tp):
        assert rel(g, t.grad.numpy()) < 1e-11, name


def test_lse_matches_library_logsumexp(oracle64):
    rng = np.random.default_rng(2)
    B, S, H, dh = 2, 9, 3, 8
    qkv = rng.standard_normal((B * S, 3 * H * dh))
    _, lse = oracle64.attn_fwd(qkv, B, S, H, dh)
    t = torch.tensor(qkv).reshape(B, S, 3, H, dh)
    q, k = t[:, :, 0].transpose(1, 2), t[:, :, 1].transpose(1, 2)
    s = q @ k.transpose(-1, -2) / math.sqrt(dh)
    s = s.masked_fill(torch.ones(S, S).triu(1).bool(), float("-inf"))
    assert np.allclose(lse, torch.logsumexp(s, -1).numpy(), rtol=0, atol=1e-12)


# ----- central finite differences on every parameter and input entry -----
def test_finite_differences_every_entry(oracle64):
    D = TINY
    rng = np.random.default_rng(3)
    ps = rand_params(D, rng, scale=0.4)
    x = rng.standard_normal((D.T, D.d))
    dy = rng.standard_normal((D.T, D.d))
    y, sv = oracle64.layer_fwd(D, ps, x)
    dx, gr = oracle64.layer_bwd(D, ps, x, sv, dy)

    def loss(ps_, x_):
        yy, _ = oracle64.layer_fwd(D, ps_, x_)
        return float(np.sum(yy * dy))

    h = 1e-5
    worst = 0.0
    tensors = [(x, dx, "x")] + [(p, g, n) for p, g, n in zip(ps, gr, PARAM_NAMES)]
    for arr, grad, name in tensors:
        fd = np.empty_like(arr)
        flat, fdf = arr.reshape(-1), fd.reshape(-1)
        for i in range(flat.size):
            keep = flat[i]
            flat[i] = keep + h
            lp = loss(ps, x)
            flat[i] = keep - h
            lm = loss(ps, x)
            flat[i] = keep
            fdf[i] = (lp - lm) / (2 * h)
        err = rel(grad, fd)
        worst = max(worst, err)
        assert err < 1e-6, (name, err)
    assert worst < 1e-6


def test_adjoint_identity_midsize(oracle64):
    """<J delta, dy> from one central difference equals <delta, J^T dy> from backward."""
    D = SMALL
    rng = np.random.default_rng(4)
    ps = rand_params(D, rng, scale=0.3)
    x = rng.standard_normal((D.T, D.d))
    dy = rng.standard_normal((D.T, D.d))
    _, sv = oracle64.layer_fwd(D, ps, x)
    dx, gr = oracle64.layer_bwd(D, ps, x, sv, dy)
    dps = [rng.standard_normal(p.shape) for p in ps]
    dxx = rng.standard_normal(x.shape)
    h = 1e-6
    yp, _ = oracle64.layer_fwd(D, [p + h * q for p, q in zip(ps, dps)], x + h * dxx)
    ym, _ = oracle64.layer_fwd(D, [p - h * q for p, q in zip(ps, dps)], x - h * dxx)
    lhs = float(np.sum((yp - ym) / (2 * h) * dy))
    rhs = float(np.sum(dx * dxx) + sum(np.sum(g * q) for g, q in zip(gr, dps)))
    assert abs(lhs - rhs) < 1e-6 * max(1.0, abs(rhs))


# ----- invariants -----
def test_causality_forward_and_backward(oracle64):
    D = SMALL
    rng = np.random.default_rng(5)
    ps = rand_params(D, rng)
    x = rng.standard_normal((D.T, D.d))
    dy = rng.standard_normal((D.T, D.d))
    y0, sv0 = oracle64.layer_fwd(D, ps, x)
    dx0, _ = oracle64.layer_bwd(D, ps, x, sv0, dy)
    b, t = 1, 17
    x2 = x.copy()
    x2[b * D.S + t + 1] += 1.0
    y2, _ = oracle64.layer_fwd(D, ps, x2)
    keep = np.ones(D.T, bool)
    keep[b * D.S + t + 1:(b + 1) * D.S] = False            # positions > t of sequence b may change
    assert np.array_equal(y0[keep], y2[keep])                # bitwise: masked keys are skipped, not zeroed
    assert not np.array_equal(y0[~keep], y2[~keep])
    dy2 = dy.copy()
    dy2[b * D.S + t] += 1.0
    dx2, _ = oracle64.layer_bwd(D, ps, x, sv0, dy2)
    keep = np.ones(D.T, bool)
    keep[b * D.S:b * D.S + t + 1] = False                    # only positions <= t of sequence b may change
    assert np.array_equal(dx0[keep], dx2[keep])
    assert not np.array_equal(dx0[~keep], dx2[~keep])


@pytest.mark.parametrize("prec", ["f32", "f64"])
def test_softmax_rows_sum_to_one_and_mask(prec):
    o = Oracle(prec)
    rng = np.random.default_rng(6)
    B, S, H, dh = 2, 40, 2, 16
    qkv = 2.0 * rng.standard_normal((B * S, 3 * H * dh))
    _, _, p = o.attn_fwd(qkv, B, S, H, dh, want_probs=True)
    assert np.all(np.abs(p.sum(-1) - 1.0) < 1e-6)
    assert np.all(p >= 0)
    iu = np.triu_indices(S, 1)
    assert np.all(p[:, :, iu[0], iu[1]] == 0)


@pytest.mark.parametrize("prec", ["f32", "f64"])
def test_layernorm_moments(prec):
    o = Oracle(prec)
    rng = np.random.default_rng(7)
    x = rng.standard_normal((64, 512)) * 3.0 + 1.5
    h, mu, r = o.ln_fwd(x, np.ones(512), np.zeros(512), 1e-5)
    assert np.all(np.abs(h.mean(-1)) < 1e-6)
    v = x.var(-1)
    assert np.allclose(h.var(-1), v / (v + 1e-5), atol=1e-5)
    assert np.all(np.abs(h.var(-1) - 1.0) < 1e-4)
    assert np.allclose(mu, x.mean(-1), atol=1e-5) and np.allclose(r, 1 / np.sqrt(v + 1e-5), rtol=1e-5)
    ref = F.layer_norm(torch.tensor(x), (512,), None, None, 1e-5).numpy()
    assert rel(h, ref) < (1e-6 if prec == "f32" else 1e-13)


def test_layernorm_backward_matches_library(oracle64):
    rng = np.random.default_rng(8)
    T, d = 10, 48
    x = torch.tensor(rng.standard_normal((T, d)), requires_grad=True)
    g = torch.tensor(1 + 0.2 * rng.standard_normal(d), requires_grad=True)
    b = torch.tensor(0.2 * rng.standard_normal(d), requires_grad=True)
    dh = rng.standard_normal((T, d))
    F.layer_norm(x, (d,), g, b, 1e-5).backward(torch.tensor(dh))
    _, mu, r = oracle64.ln_fwd(x.detach().numpy(), g.detach().numpy(), b.detach().numpy())
    dx, dg, db = oracle64.ln_bwd(dh, x.detach().numpy(), mu, r, g.detach().numpy())
    assert rel(dx, x.grad.numpy()) < 1e-12 and rel(dg, g.grad.numpy()) < 1e-12 and rel(db, b.grad.numpy()) < 1e-12


# ----- closed forms / special cases -----
def test_single_token_attention_returns_v(oracle64):
    rng = np.random.default_rng(9)
    B, S, H, dh = 3, 1, 2, 8
    qkv = rng.standard_normal((B * S, 3 * H * dh))
    o, lse = oracle64.attn_fwd(qkv, B, S, H, dh)
    assert np.array_equal(o, qkv[:, 2 * H * dh:])
    q, k = qkv[:, :H * dh].reshape(B, H, dh), qkv[:, H * dh:2 * H * dh].reshape(B, H, dh)
    assert np.allclose(lse[:, :, 0], (q * k).sum(-1) / math.sqrt(dh), atol=1e-13)


def test_equal_keys_give_prefix_means(oracle64):
    rng = np.random.default_rng(10)
    B, S, H, dh = 1, 12, 2, 8
    d = H * dh
    qkv = rng.standard_normal((S, 3 * d))
    qkv[:, d:2 * d] = qkv[0, d:2 * d]                       # every key equal -> uniform weights over the prefix
    o, lse = oracle64.attn_fwd(qkv, B, S, H, dh)
    v = qkv[:, 2 * d:]
    prefix_mean = np.cumsum(v, 0) / np.arange(1, S + 1)[:, None]
    assert np.allclose(o, prefix_mean, atol=1e-13)
    q, k = qkv[:, :d].reshape(S, H, dh), qkv[:, d:2 * d].reshape(S, H, dh)
    expect = (q * k).sum(-1) / math.sqrt(dh) + np.log(np.arange(1, S + 1))[:, None]
    assert np.allclose(lse[0].T, expect, atol=1e-12)


def test_zero_output_weights_make_identity(oracle64):
    D = SMALL
    rng = np.random.default_rng(11)
    ps = rand_params(D, rng)
    for i in (4, 5, 10, 11):
        ps[i] = np.zeros_like(ps[i])
    x = rng.standard_normal((D.T, D.d))
    dy = rng.standard_normal((D.T, D.d))
    y, sv = oracle64.layer_fwd(D, ps, x)
    dx, gr = oracle64.layer_bwd(D, ps, x, sv, dy)
    assert np.array_equal(y, x) and np.array_equal(dx, dy)
    assert np.allclose(gr[5], dy.sum(0)) and np.allclose(gr[11], dy.sum(0))


def test_gelu_values_and_identities(oracle64):
    # Phi(1), Phi(2) to 16 digits (standard normal CDF): gelu(x) = x Phi(x)
    a = oracle64.gelu_fwd(np.array([0.0, 1.0, -1.0, 2.0, -2.0]))
    assert np.allclose(a, [0.0, 0.8413447460685429, -0.15865525393145707,
                           1.9544997361036416, -0.04550026389635842], atol=1e-15)
    x = np.linspace(-6, 6, 1001)
    assert np.allclose(oracle64.gelu_fwd(x) - oracle64.gelu_fwd(-x), x, atol=1e-14)
    g0 = oracle64.gelu_bwd(np.zeros(1), np.ones(1))
    assert g0[0] == 0.5
    h = 1e-6
    for act in (ACT_GELU_ERF, ACT_GELU_TANH):
        fd = (oracle64.gelu_fwd(x + h, act) - oracle64.gelu_fwd(x - h, act)) / (2 * h)
        assert np.allclose(oracle64.gelu_bwd(x, np.ones_like(x), act), fd, atol=1e-8)
    diff = np.abs(oracle64.gelu_fwd(x, ACT_GELU_TANH) - oracle64.gelu_fwd(x, ACT_GELU_ERF)).max()
    assert 1e-4 < diff < 5e-4                               # the two forms differ, so both sides must agree on one
    assert np.allclose(oracle64.gelu_fwd(x), F.gelu(torch.tensor(x)).numpy(), atol=1e-15)


def test_backward_is_linear_in_dy_and_accumulates(oracle64):
    D = TINY
    rng = np.random.default_rng(12)
    ps = rand_params(D, rng)
    x = rng.standard_normal((D.T, D.d))
    dy = rng.standard_normal((D.T, D.d))
    _, sv = oracle64.layer_fwd(D, ps, x)
    dx1, g1 = oracle64.layer_bwd(D, ps, x, sv, dy)
    dx3, g3 = oracle64.layer_bwd(D, ps, x, sv, 3.0 * dy)
    assert rel(dx3, 3 * dx1) < 1e-14
    for a, b in zip(g3, g1):
        assert rel(a, 3 * b) < 1e-13
    acc = [g.copy() for g in g1]
    oracle64.layer_bwd(D, ps, x, sv, dy, acc, accumulate=True)
    oracle64.layer_bwd(D, ps, x, sv, dy, acc, accumulate=True)
    for a, b in zip(acc, g1):
        assert rel(a, 3 * b) < 1e-14


def test_batch_permutation_equivariance(oracle64):
    D = SMALL
    rng = np.random.default_rng(13)
    ps = rand_params(D, rng)
    x = rng.standard_normal((D.B, D.S, D.d))
    y, _ = oracle64.layer_fwd(D, ps, x)
    y2, _ = oracle64.layer_fwd(D, ps, x[::-1])
    assert np.array_equal(y.reshape(D.B, D.S, D.d)[::-1], y2.reshape(D.B, D.S, D.d))


def test_bias_grads_are_column_sums(oracle64):
    rng = np.random.default_rng(14)
    x, W, dout = rng.standard_normal((7, 5)), rng.standard_normal((3, 5)), rng.standard_normal((7, 3))
    dx, dW, db = oracle64.linear_bwd(x, W, dout)
    assert np.allclose(db, dout.sum(0)) and np.allclose(dW, dout.T @ x) and np.allclose(dx, dout @ W)
    assert np.allclose(oracle64.linear_fwd(x, W, np.arange(3.0)), x @ W.T + np.arange(3.0))


def test_f32_agrees_with_f64(oracle32, oracle64):
    D = SMALL
    rng = np.random.default_rng(15)
    ps = rand_params(D, rng)
    x = rng.standard_normal((D.T, D.d)).astype(np.float32)
    ps = [p.astype(np.float32) for p in ps]
    dy = rng.standard_normal((D.T, D.d)).astype(np.float32)
    y32, s32 = oracle32.layer_fwd(D, ps, x)
    y64, s64 = oracle64.layer_fwd(D, ps, x)
    assert rel(y32, y64) < 1e-5
    dx32, g32 = oracle32.layer_bwd(D, ps, x, s32, dy)
    dx64, g64 = oracle64.layer_bwd(D, ps, x, s64, dy)
    assert rel(dx32, dx64) < 1e-5
    for a, b in zip(g32, g64):
        assert rel(a, b) < 1e-5


def test_chain_matches_library_autograd_and_sums_microbatches(oracle64):
    D = TINY
    rng = np.random.default_rng(16)
    L, M = 3, 2
    pls = [rand_params(D, rng) for _ in range(L)]
    xs = [rng.standard_normal((D.T, D.d)) for _ in range(M)]
    dys = [rng.standard_normal((D.T, D.d)) for _ in range(M)]
    ys, dxs, grads = oracle64.chain(D, pls, xs, dys)
    tps = [[torch.tensor(p, requires_grad=True) for p in ps] for ps in pls]
    for m in range(M):
        tx = torch.tensor(xs[m], requires_grad=True)
        h = tx
        for l in range(L):
            h, _ = torch_layer(D, tps[l], h)
        h.backward(torch.tensor(dys[m]))
        assert rel(ys[m], h.detach().numpy()) < 1e-12
        assert rel(dxs[m], tx.grad.numpy()) < 1e-11
    for l in range(L):
        for g, t in zip(grads[l], tps[l]):
            assert rel(g, t.grad.numpy()) < 1e-11       # autograd summed over the two micro-batches too


def test_structure_matches_section_5_3_parameter_count():
    vals = {}
    with open(os.path.join(GOLDEN, "section5_3_decoder_lm.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, *v = line.split()
                vals[k] = v
    L, d, Fh = int(vals["n_layers"][0]), int(vals["d_model"][0]), int(vals["d_ff"][0])
    D = Dims(B=1, S=1, d=d, H=16, dh=d // 16, F=Fh)
    per_layer = sum(int(np.prod(s)) for s in D.param_shapes())
    total = L * per_layer
    assert round(total / 1e9) == int(vals["params_billion"][0])
    assert abs(total - L * (4 * d * d + 2 * d * Fh)) / total < 1e-3     # biases and LN add < 0.1 %
    assert len(SAVED_NAMES) == 12 and len(PARAM_NAMES) == 12


def test_figure2_program_reproduces_the_printed_values():
    """The paper prints the input and both outputs of its Figure 2 example program."""
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "figure2_program.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, *nums = line.split()
                vals[k] = np.array([float(t) for t in nums])
    o = Oracle("f32")
    out0, out1 = o.figure2_program(vals["v"])
    assert np.array_equal(out0, vals["out0"].astype(np.float32))
    assert np.array_equal(out1, vals["out1"].astype(np.float32))
