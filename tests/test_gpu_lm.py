"""GPU parity for the two ends of the language model (embedding lookup, tied softmax head with
cross-entropy) and the whole small-LM step, against the CPU oracle on the same seeded inputs."""
import math

import numpy as np
import pytest
import torch

from paper_2203_12533_b200 import inputs
from tests.gpu_util import ACT_TOL, ELEM_ACT, GRAD_TOL, dims_of, elem_check, np64, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pw():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2203_12533_b200 import binding
    binding.lib()
    return binding


def test_embedding_lookup_is_exact_and_scatter_add_is_ordered(pw, oracle64):
    g = torch.Generator().manual_seed(5)
    for T, d, V in ((300, 256, 1000), (512, 64, 4), (64, 1024, 32768)):      # V = 4: lists far longer than a warp
        E = (torch.randn((V, d), generator=g) * 0.02).to(torch.bfloat16).cuda()
        ids = torch.randint(0, V, (T,), generator=g, dtype=torch.int32).cuda()
        x0 = torch.empty((T, d), dtype=torch.bfloat16, device="cuda")
        pw.op_embedding_fwd(ids, E, x0)
        assert torch.equal(x0, E[ids.long()])
        dx0 = torch.randn((T, d), generator=g).to(torch.bfloat16).cuda()
        base = torch.randn((V, d), generator=g).cuda()
        scratch = torch.empty(pw.op_embedding_bwd_scratch_bytes(T, V), dtype=torch.uint8, device="cuda")
        outs = []
        for _ in range(2):
            dE = base.clone()
            pw.op_embedding_bwd(ids, dx0, dE, scratch)
            outs.append(dE)
        torch.cuda.synchronize()
        assert pw.op_status() == (0, 0)
        assert torch.equal(outs[0], outs[1])                                   # fixed summation order
        want = np64(base)
        oracle64.embed_bwd(ids.cpu().numpy(), np64(dx0), want)
        assert rel_l2(outs[0], want) < 1e-6


def test_softmax_xent_against_oracle_formulas(pw, oracle64):
    g = torch.Generator().manual_seed(6)
    T, V, ld = 37, 1000, 1024
    buf = (torch.randn((T, ld), generator=g) * 3).to(torch.bfloat16).cuda()
    padding_before = buf[:, V:].clone()
    logits = buf[:, :V]
    z = np64(logits)
    labels = torch.randint(0, V, (T,), generator=g, dtype=torch.int32).cuda()
    lse = torch.empty(T, device="cuda")
    rows = torch.empty(T, device="cuda")
    scale = 1.0 / T
    pw.op_softmax_xent(logits, labels, scale, lse, rows)
    torch.cuda.synchronize()
    assert pw.op_status() == (0, 0)
    lab = labels.cpu().numpy()
    # the head with hf = z and E = identity has logits z: the oracle's head formulas apply as they stand
    eye = np.eye(V)
    loss, lse_want, _ = oracle64.head_fwd(z, eye, lab, want_logits=True)
    assert np.allclose(lse.cpu().numpy(), lse_want, rtol=2e-6, atol=2e-6)
    assert abs(rows.double().mean().item() - loss) < 1e-5
    _, dz = oracle64.head_bwd(z, eye, lab, lse_want, np.zeros((V, V)), want_dlogits=True)
    assert rel_l2(logits, dz) < ACT_TOL
    elem_check(logits, dz, "dlogits", **ELEM_ACT)
    assert torch.equal(buf[:, V:], padding_before)                             # the columns between V and the row pitch are untouched


def test_softmax_xent_reports_a_label_outside_the_vocabulary(pw):
    T, V = 4, 64
    logits = torch.zeros((T, V), dtype=torch.bfloat16, device="cuda")
    labels = torch.tensor([1, 2, 99, 3], dtype=torch.int32, device="cuda")
    lse, rows = torch.empty(T, device="cuda"), torch.empty(T, device="cuda")
    pw.op_softmax_xent(logits, labels, 1.0, lse, rows)
    torch.cuda.synchronize()
    assert pw.op_status()[0] == 1                                              # PW_ERR_INVALID_ARG recorded by the kernel
    assert torch.isfinite(lse).all()
    pw.op_status_reset()
    assert pw.op_status() == (0, 0)


def run_lm_gpu(pw, w, seed=0, recompute=False, random_ln=True):
    L = w.n_layers
    stage = pw.Stage(L, w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch)
    params = [[p.cuda() for p in inputs.layer_params(w, seed, l, random_ln=random_ln)] for l in range(L)]
    grads = [[torch.full(p.shape, float("nan"), dtype=torch.float32, device="cuda") for p in ps] for ps in params]
    E, g, b, ids, labels = [t.cuda() for t in inputs.lm_inputs(w, seed, random_ln=random_ln)]
    lm_grads = [torch.full(E.shape, float("nan"), dtype=torch.float32, device="cuda"),
                torch.full(g.shape, float("nan"), dtype=torch.float32, device="cuda"),
                torch.full(b.shape, float("nan"), dtype=torch.float32, device="cuda")]
    loss = torch.full((1,), float("nan"), device="cuda")
    ws = torch.empty(stage.lm_workspace_bytes(w.vocab, recompute), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        stage.lm_step(params, grads, (E, g, b), lm_grads, ids, labels, loss, w.vocab, ws, recompute, stream=stream)
    torch.cuda.synchronize()
    assert stage.status() == (0, 0)
    return loss.item(), grads, lm_grads


def oracle_lm(oracle, w, seed=0, random_ln=True):
    D = dims_of(w)
    to = (lambda t: t.double().numpy()) if oracle.suf == "f64" else (lambda t: t.float().numpy())
    pls = [[to(p) for p in inputs.layer_params(w, seed, l, random_ln=random_ln)] for l in range(w.n_layers)]
    E, g, b, ids, labels = inputs.lm_inputs(w, seed, random_ln=random_ln)
    rt = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).to(torch.from_numpy(a).dtype).numpy()
    return oracle.lm_step(D, pls, to(E), to(g), to(b), ids.numpy().ravel(), labels.numpy().ravel(), handoff=rt)


def check_lm(pw, oracle, w, recompute=False):
    loss, grads, (dE, dg, db) = run_lm_gpu(pw, w, recompute=recompute)
    ref = oracle_lm(oracle, w)
    assert abs(loss - ref["loss"]) < 2e-3 * max(1.0, abs(ref["loss"])), (loss, ref["loss"])
    errs = {"dE": rel_l2(dE, ref["dE"]), "dlnf_gamma": rel_l2(dg, ref["dlnf_gamma"]), "dlnf_beta": rel_l2(db, ref["dlnf_beta"])}
    for l in range(w.n_layers):
        for name, got, want in zip(pw.PARAM_NAMES, grads[l], ref["grads"][l]):
            errs[f"l{l}.{name}"] = rel_l2(got, want)
    assert max(errs.values()) < GRAD_TOL, errs
    return loss, dE


def test_small_lm_step_against_oracle(pw, oracle64):
    w = inputs.Workload("lm_small", 256, 4, 64, 1024, 128, 2, n_layers=2, vocab=512)
    loss_a, dE_a = check_lm(pw, oracle64, w, recompute=False)
    loss_b, dE_b = check_lm(pw, oracle64, w, recompute=True)
    assert loss_a == loss_b and torch.equal(dE_a, dE_b)                        # recompute gives the same bits


def test_lm_step_at_the_workload_widths(pw, oracle32):
    """Workload 5's widths and vocabulary (d = 1024, 16 x 64 heads, F = 4096, V = 32768) on fewer tokens and layers."""
    w = inputs.WORKLOADS[5].with_(n_layers=2, batch=2, seq_len=256)
    loss, _ = check_lm(pw, oracle32, w)
    assert math.log(w.vocab) <= loss <= math.log(w.vocab) + 0.5


def test_lm_step_full_workload_runs_and_starts_at_the_expected_loss(pw):
    """All of workload 5 (12 layers, 16 x 1024 tokens, V = 32768): too large for the oracle, so
    the properties that hold at any size are checked - the initial-loss window of the recipe,
    finite gradients, every looked-up row of the table touched, and bitwise repeatability."""
    w = inputs.WORKLOADS[5]
    loss1, grads1, (dE1, dg1, db1) = run_lm_gpu(pw, w, random_ln=False)
    assert math.log(w.vocab) <= loss1 <= math.log(w.vocab) + 0.5, loss1
    for t in [dE1, dg1, db1] + [g for gs in grads1 for g in gs]:
        assert torch.isfinite(t).all()
    assert dE1.abs().sum(dim=1).gt(0).all()                                    # the head reaches every row of the table
    loss2, _, (dE2, _, _) = run_lm_gpu(pw, w, random_ln=False)
    assert loss1 == loss2 and torch.equal(dE1, dE2)
