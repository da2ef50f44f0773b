"""Pins for the oracle's gradient apply (plain SGD on a master copy with a bf16 working copy;
the appendix's data-parallel trace has each island apply the gradients it received, the paper
names no optimizer) against things other than the oracle itself: a library bf16 conversion,
hand-computed rounding ties, the closed form after k equal steps, the exact minimiser of a
quadratic, and the first-order decrease of the small-LM loss along its own gradients."""
import numpy as np
import pytest
import torch

import oracle as oracle_mod
from paper_2203_12533_b200 import inputs


@pytest.fixture(scope="module")
def o64():
    return oracle_mod.Oracle("f64")


@pytest.mark.parametrize("prec", ["f32", "f64"])
def test_bf16_rounding_matches_the_library_conversion_and_hand_computed_ties(prec):
    o = oracle_mod.Oracle(prec)
    g = torch.Generator().manual_seed(11)
    x = torch.cat([torch.randn(4000, generator=g), torch.randn(2000, generator=g) * 1e-3,
                   torch.randn(2000, generator=g) * 1e4, torch.tensor([0.0, -0.0, 1.0, -1.0])])
    got = o.round_bf16(x.numpy())
    want = x.to(torch.bfloat16).float().numpy()
    assert np.array_equal(got.astype(np.float32), want)
    # bf16 keeps 8 significant bits: spacing 2^-7 in [1, 2).  Ties go to the even neighbour.
    u = 2.0 ** -7
    cases = {1.0 + 0.5 * u: 1.0,                 # tie between 1 (even) and 1 + u (odd)
             1.0 + 1.5 * u: 1.0 + 2 * u,         # tie between 1 + u (odd) and 1 + 2u (even)
             1.0 + 0.5 * u + 2.0 ** -20: 1.0 + u,
             -(1.0 + 0.5 * u): -1.0,
             2.0 - 0.25 * u: 2.0,                # rounds up across a power of two
             0.1: 0.10009765625}
    for v, w in cases.items():
        assert float(o.round_bf16(np.array([v]))[0]) == w, (v, w)


def test_k_equal_steps_have_a_closed_form_and_zero_rate_only_rounds(o64):
    rng = np.random.default_rng(5)
    m0 = rng.standard_normal(1000)
    g = rng.standard_normal(1000)
    m0_before, g_before = m0.copy(), g.copy()
    lr, scale, k = 0.03, 0.25, 7
    m = m0
    for _ in range(k):
        m, p = o64.sgd_apply(m, g, lr, scale)
    assert np.allclose(m, m0 - k * lr * scale * g, rtol=0, atol=1e-14)
    assert np.array_equal(p, o64.round_bf16(m))
    assert np.array_equal(p.astype(np.float32), torch.tensor(m).to(torch.bfloat16).float().numpy())
    m1, p1 = o64.sgd_apply(m0, g, 0.0)
    assert np.array_equal(m1, m0) and np.array_equal(p1, o64.round_bf16(m0))
    m2, _ = o64.sgd_apply(m0, g, lr)                               # grad_scale defaults to 1
    assert np.allclose(m2, m0 - lr * g, rtol=0, atol=1e-15)
    assert np.array_equal(m0, m0_before) and np.array_equal(g, g_before)   # inputs are left alone


def test_one_full_step_lands_on_the_minimiser_of_a_quadratic(o64):
    """f(w) = |w - w*|^2 / 2 has gradient w - w*: rate 1 reaches w* in one step, rate 1/2 halves
    the distance every step.  A wrong sign or a dropped factor fails this."""
    rng = np.random.default_rng(6)
    w, star = rng.standard_normal(64), rng.standard_normal(64)
    m, _ = o64.sgd_apply(w, w - star, 1.0)
    assert np.allclose(m, star, atol=1e-15)
    m = w
    for _ in range(10):
        m, _ = o64.sgd_apply(m, m - star, 0.5)
    assert np.allclose(m - star, (w - star) * 0.5 ** 10, atol=1e-15)


def test_applying_the_lm_gradients_lowers_the_loss_by_rate_times_gradient_norm(o64):
    """loss(w - lr g) = loss(w) - lr |g|^2 + O(lr^2): the step and the gradients of the small
    language-model step agree in sign and scale for every parameter tensor at once."""
    w = inputs.Workload("tiny_lm", 64, 1, 64, 128, 8, 2, n_layers=2, vocab=40, sigma_w=0.2)
    D = oracle_mod.Dims(w.batch, w.seq_len, w.d_model, w.n_heads, w.head_dim, w.d_ff)
    ps = [[p.double().numpy() for p in inputs.layer_params(w, 3, l, random_ln=True)] for l in range(w.n_layers)]
    E, g, b, ids, labels = inputs.lm_inputs(w, 3, random_ln=True)
    E, g, b = E.double().numpy() * 10, g.double().numpy(), b.double().numpy()
    ids, labels = ids.numpy().ravel(), labels.numpy().ravel()
    out = o64.lm_step(D, ps, E, g, b, ids, labels)
    gnorm2 = (sum(float((t ** 2).sum()) for layer in out["grads"] for t in layer) + float((out["dE"] ** 2).sum()) +
              float((out["dlnf_gamma"] ** 2).sum()) + float((out["dlnf_beta"] ** 2).sum()))
    assert gnorm2 > 0
    drops = []
    for lr in (1e-4, 5e-5):
        ps2 = [[o64.sgd_apply(p, gr, lr)[0] for p, gr in zip(layer, gl)] for layer, gl in zip(ps, out["grads"])]
        E2 = o64.sgd_apply(E, out["dE"], lr)[0]
        g2 = o64.sgd_apply(g, out["dlnf_gamma"], lr)[0]
        b2 = o64.sgd_apply(b, out["dlnf_beta"], lr)[0]
        drops.append(out["loss"] - o64.lm_step(D, ps2, E2, g2, b2, ids, labels)["loss"])
        assert abs(drops[-1] - lr * gnorm2) < 0.02 * lr * gnorm2, (lr, drops[-1], lr * gnorm2)
    assert drops[0] > drops[1] > 0


def test_data_parallel_apply_is_one_step_on_the_summed_gradient(o64):
    """Two replicas with half the batch each and grad_scale 1/2 take the step of the mean gradient;
    one replica is the plain apply; for a loss that is a sum over examples the replicas' summed
    gradients equal the gradient of the whole batch (checked on a least-squares problem)."""
    rng = np.random.default_rng(8)
    m0 = rng.standard_normal(300)
    gs = [rng.standard_normal(300) for _ in range(4)]
    m1, p1 = o64.dp_sgd_apply(m0, gs, 0.1, 0.25)
    assert np.allclose(m1, m0 - 0.1 * np.mean(gs, axis=0), rtol=0, atol=1e-15)
    assert np.array_equal(p1, o64.round_bf16(m1))
    ma, pa = o64.dp_sgd_apply(m0, gs[:1], 0.1)
    mb, pb = o64.sgd_apply(m0, gs[0], 0.1)
    assert np.array_equal(ma, mb) and np.array_equal(pa, pb)
    mr, _ = o64.dp_sgd_apply(m0, gs[::-1], 0.1, 0.25)                  # order only changes the rounding
    assert np.allclose(mr, m1, rtol=0, atol=1e-15)
    # least squares: loss = sum_i (a_i . w - y_i)^2 / 2 over 8 examples, split 3 + 5 over two replicas
    A, y, w = rng.standard_normal((8, 6)), rng.standard_normal(8), rng.standard_normal(6)
    grad = lambda rows: A[rows].T @ (A[rows] @ w - y[rows])
    whole, _ = o64.sgd_apply(w, grad(slice(0, 8)), 0.05)
    split, _ = o64.dp_sgd_apply(w, [grad(slice(0, 3)), grad(slice(3, 8))], 0.05)
    assert np.allclose(whole, split, rtol=0, atol=1e-14)
    full_loss = lambda v: 0.5 * float(((A @ v - y) ** 2).sum())
    assert full_loss(split) < full_loss(w)
