"""Pins for the language-model ends of the oracle (embedding lookup, tied softmax head with
cross-entropy, the whole small-LM step) against things other than the oracle itself: closed
forms, scipy/torch library routines in fp64, torch autograd, central finite differences, and
the initial-loss window that the workload's recipe implies (Section 5.3 names the embedding
and softmax layers but prints no formula; the readings are in the design notes)."""
import math

import numpy as np
import pytest
import torch
from scipy.special import logsumexp

import oracle as oracle_mod
from paper_2203_12533_b200 import inputs


@pytest.fixture(scope="module")
def o64():
    return oracle_mod.Oracle("f64")


def test_zero_table_gives_log_vocab_and_uniform_gradient(o64):
    T, d, V = 7, 16, 50
    rng = np.random.default_rng(1)
    hf = rng.standard_normal((T, d))
    E = np.zeros((V, d))
    labels = rng.integers(0, V, T)
    loss, lse, z = o64.head_fwd(hf, E, labels, want_logits=True)
    assert abs(loss - math.log(V)) < 1e-12 and np.allclose(lse, math.log(V)) and np.all(z == 0)
    dE = np.zeros_like(E)
    dhf, dz = o64.head_bwd(hf, E, labels, lse, dE, want_dlogits=True)
    want = np.full((T, V), 1.0 / V)
    want[np.arange(T), labels] -= 1.0
    assert np.allclose(dz, want / T, atol=1e-15)
    assert np.allclose(dz.sum(1), 0, atol=1e-15)              # every gradient row sums to zero
    assert np.all(dhf == 0)                                    # dz E with E = 0


def test_head_matches_library_logsumexp_and_autograd(o64):
    T, d, V = 9, 12, 33
    rng = np.random.default_rng(2)
    hf = rng.standard_normal((T, d))
    E = rng.standard_normal((V, d)) * 0.5
    labels = rng.integers(0, V, T)
    loss, lse, z = o64.head_fwd(hf, E, labels, want_logits=True)
    zz = hf @ E.T
    assert np.allclose(z, zz, atol=1e-12)
    assert np.allclose(lse, logsumexp(zz, axis=1), atol=1e-12)
    th, tE = torch.tensor(hf, requires_grad=True), torch.tensor(E, requires_grad=True)
    tl = torch.nn.functional.cross_entropy(th @ tE.T, torch.tensor(labels, dtype=torch.long), reduction="mean")
    tl.backward()
    assert abs(loss - tl.item()) < 1e-12
    dE = np.zeros_like(E)
    dhf = o64.head_bwd(hf, E, labels, lse, dE)
    assert np.allclose(dhf, th.grad.numpy(), atol=1e-12)
    assert np.allclose(dE, tE.grad.numpy(), atol=1e-12)
    # large logits: the max-shifted form must not overflow
    loss_big, lse_big = o64.head_fwd(hf * 300, E, labels)
    assert np.isfinite(loss_big) and np.allclose(lse_big, logsumexp(300 * zz, axis=1), rtol=1e-12)


def test_embedding_lookup_and_scatter_add(o64):
    V, d = 11, 5
    rng = np.random.default_rng(3)
    E = rng.standard_normal((V, d))
    ids = np.array([3, 3, 0, 10, 3, 7, 0], dtype=np.int32)
    x0 = o64.embed_fwd(ids, E)
    assert np.array_equal(x0, E[ids])
    dx0 = rng.standard_normal((ids.size, d))
    dE = np.ones((V, d))                                       # accumulates on top of what is there
    o64.embed_bwd(ids, dx0, dE)
    want = np.ones((V, d))
    for t, v in enumerate(ids):                                # brute force
        want[v] += dx0[t]
    assert np.allclose(dE, want, atol=1e-15)
    assert np.allclose(dE[3] - 1, dx0[[0, 1, 4]].sum(0))       # repeated id: the rows add up
    assert np.all(dE[[1, 2, 4, 5, 6, 8, 9]] == 1)              # untouched rows
    same = np.zeros((V, d))
    o64.embed_bwd(np.full(ids.size, 4, np.int32), dx0, same)   # one id only: a column sum
    assert np.allclose(same[4], dx0.sum(0))


def _tiny_lm(seed=0):
    w = inputs.Workload("tiny_lm", 64, 1, 64, 128, 8, 2, n_layers=2, vocab=40, sigma_w=0.2)
    D = oracle_mod.Dims(w.batch, w.seq_len, w.d_model, w.n_heads, w.head_dim, w.d_ff)
    ps = [[p.double().numpy() for p in inputs.layer_params(w, seed, l, random_ln=True)] for l in range(w.n_layers)]
    E, g, b, ids, labels = inputs.lm_inputs(w, seed, random_ln=True)
    E = E.double().numpy() * 10                                # sizeable logits
    return w, D, ps, E, g.double().numpy(), b.double().numpy(), ids.numpy().ravel(), labels.numpy().ravel()


def test_lm_step_gradients_match_central_differences(o64):
    w, D, ps, E, g, b, ids, labels = _tiny_lm()
    out = o64.lm_step(D, ps, E, g, b, ids, labels)
    assert np.isfinite(out["loss"])
    rng = np.random.default_rng(4)
    eps = 1e-6

    def loss_with(mod):
        ps2 = [[p.copy() for p in layer] for layer in ps]
        E2, g2, b2 = E.copy(), g.copy(), b.copy()
        mod(ps2, E2, g2, b2)
        return o64.lm_step(D, ps2, E2, g2, b2, ids, labels)["loss"]

    # the tied table: a row that is both looked up and a label, one that is neither
    used = int(ids[0])
    for row in (used, int(labels[1]), next(v for v in range(w.vocab) if v not in ids and v not in labels)):
        c = int(rng.integers(0, w.d_model))
        fd = (loss_with(lambda p_, E_, g_, b_: E_.__setitem__((row, c), E_[row, c] + eps)) -
              loss_with(lambda p_, E_, g_, b_: E_.__setitem__((row, c), E_[row, c] - eps))) / (2 * eps)
        assert abs(fd - out["dE"][row, c]) < 1e-6 * max(1.0, abs(fd)), (row, c, fd, out["dE"][row, c])
    for name, arr, grad in (("lnf_gamma", 2, out["dlnf_gamma"]), ("lnf_beta", 3, out["dlnf_beta"])):
        c = int(rng.integers(0, w.d_model))
        def bump(sign):
            def f(p_, E_, g_, b_):
                tgt = g_ if arr == 2 else b_
                tgt[c] += sign * eps
            return f
        fd = (loss_with(bump(+1)) - loss_with(bump(-1))) / (2 * eps)
        assert abs(fd - grad[c]) < 1e-6 * max(1.0, abs(fd)), (name, fd, grad[c])
    # one weight of each layer
    for l in range(w.n_layers):
        i, j = int(rng.integers(0, 3 * w.d_model)), int(rng.integers(0, w.d_model))
        def bumpw(sign):
            def f(p_, E_, g_, b_):
                p_[l][2][i, j] += sign * eps
            return f
        fd = (loss_with(bumpw(+1)) - loss_with(bumpw(-1))) / (2 * eps)
        assert abs(fd - out["grads"][l][2][i, j]) < 1e-6 * max(1.0, abs(fd)), (l, fd, out["grads"][l][2][i, j])


def test_lm_step_matches_torch_autograd_on_the_ends(o64):
    """Embedding + final LayerNorm + tied head with the layers replaced by the identity (L = 0)."""
    w, D, _, E, g, b, ids, labels = _tiny_lm(1)
    out = o64.lm_step(D, [], E, g, b, ids, labels)
    tE = torch.tensor(E, requires_grad=True)
    tg, tb = torch.tensor(g, requires_grad=True), torch.tensor(b, requires_grad=True)
    x0 = tE[torch.tensor(ids, dtype=torch.long)]
    hf = torch.nn.functional.layer_norm(x0, (w.d_model,), tg, tb, D.eps)
    tl = torch.nn.functional.cross_entropy(hf @ tE.T, torch.tensor(labels, dtype=torch.long))
    tl.backward()
    assert abs(out["loss"] - tl.item()) < 1e-10
    assert np.allclose(out["dE"], tE.grad.numpy(), atol=1e-10)
    assert np.allclose(out["dlnf_gamma"], tg.grad.numpy(), atol=1e-10)
    assert np.allclose(out["dlnf_beta"], tb.grad.numpy(), atol=1e-10)


def test_initial_loss_of_the_lm_recipe_lies_just_above_log_vocab():
    """With E ~ N(0, 0.02) and unit-variance LayerNorm output the logits have standard deviation
    about sqrt(d) * 0.02 = 0.64, so the mean cross-entropy at initialisation is about
    ln V + 0.64^2 / 2: inside [ln V, ln V + 0.5] for the workload's d = 1024, V = 32768."""
    o32 = oracle_mod.Oracle("f32")
    w = inputs.WORKLOADS[5].with_(n_layers=1, batch=1, seq_len=128)
    D = oracle_mod.Dims(w.batch, w.seq_len, w.d_model, w.n_heads, w.head_dim, w.d_ff)
    ps = [[p.float().numpy() for p in inputs.layer_params(w, 0, 0)]]
    E, g, b, ids, labels = inputs.lm_inputs(w, 0)
    x0 = o32.embed_fwd(ids.numpy().ravel(), E.float().numpy())
    y, _ = o32.layer_fwd(D, ps[0], x0)
    hf, _, _ = o32.ln_fwd(y, g.float().numpy(), b.float().numpy(), D.eps)
    loss, _ = o32.head_fwd(hf, E.float().numpy(), labels.numpy().ravel())
    assert math.log(w.vocab) <= loss <= math.log(w.vocab) + 0.5, loss
