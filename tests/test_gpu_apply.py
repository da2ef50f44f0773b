"""GPU parity for the gradient apply (plain SGD on an fp32 master copy, bf16 working copy) against
the CPU oracle, element by element, and a short training loop of the small language model in which
every step's loss must follow the oracle's."""
import numpy as np
import pytest
import torch

from paper_2203_12533_b200 import inputs
from tests.gpu_util import dims_of, np64, rel_l2

pytestmark = pytest.mark.gpu

CHUNK = 8192            # elements one CTA owns


@pytest.fixture(scope="module")
def pw():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2203_12533_b200 import binding
    binding.lib()
    return binding


def _bf16_ulp(x):
    """Spacing of bf16 at |x| (8 significant bits)."""
    return 2.0 ** (np.floor(np.log2(np.maximum(np.abs(x), 1e-30))) - 7)


def _check_item(oracle32, oracle64, m0, g, lr, scale, m_gpu, p_gpu):
    m_gpu, p_gpu = m_gpu.cpu().numpy(), p_gpu.float().cpu().numpy()
    m64, _ = oracle64.sgd_apply(m0.astype(np.float64), g.astype(np.float64), lr, scale)
    # the master: one fused multiply-add in fp32 per element
    assert np.all(np.abs(m_gpu - m64) <= 2.0 ** -23 * np.abs(m64) + 2.0 ** -24 * np.abs(lr * scale * g) + 1e-45)
    # the working copy is the GPU's own master rounded to nearest even (same precision on both sides)
    assert np.array_equal(p_gpu, torch.from_numpy(m_gpu).to(torch.bfloat16).float().numpy())
    assert np.array_equal(p_gpu, oracle32.round_bf16(m_gpu))
    # and against the oracle run in fp32: the same values except where the last bit of the master
    # decides a rounding tie, and then the neighbouring bf16 value
    m32, p32 = oracle32.sgd_apply(m0, g, lr, scale)
    differ = p_gpu != p32
    assert differ.mean() <= 1e-3
    assert np.all(np.abs(p_gpu - p32)[differ] <= _bf16_ulp(p32[differ]))
    assert np.all(np.abs(m_gpu - m32) <= 2.0 ** -23 * (np.abs(m32) + np.abs(lr * scale * g)))   # the rate is rounded to fp32 too


def test_sgd_apply_matches_oracle_elementwise(pw, oracle32, oracle64):
    gen = torch.Generator().manual_seed(21)
    sizes = [1, 7, 8, 9, CHUNK - 1, CHUNK, CHUNK + 1, 3 * CHUNK + 5, 100003, 0, 4 * CHUNK]
    lr, scale = 0.05, 0.25
    masters = [torch.randn(n, generator=gen) * (10.0 ** (i % 3 - 1)) for i, n in enumerate(sizes)]
    grads = [torch.randn(n, generator=gen) for n in sizes]
    m_d = [m.cuda() for m in masters]
    g_d = [g.cuda() for g in grads]
    p_d = [torch.full((n,), float("nan"), dtype=torch.bfloat16, device="cuda") for n in sizes]
    pw.sgd_apply(list(zip(p_d, m_d, g_d)), lr, scale)
    torch.cuda.synchronize()
    for n, m0, g, m, p, gd in zip(sizes, masters, grads, m_d, p_d, g_d):
        if n == 0:
            continue
        assert torch.equal(gd.cpu(), g)                                  # gradients are read only
        _check_item(oracle32, oracle64, m0.numpy(), g.numpy(), lr, scale, m, p)


def test_sgd_apply_unaligned_views_and_neighbours_untouched(pw, oracle32, oracle64):
    """Tensors that start 4 (master, grad) or 2 (param) bytes into a buffer take the element-wise path;
    what lies before and after them must not change."""
    gen = torch.Generator().manual_seed(22)
    n = 2 * CHUNK + 77
    mbuf = torch.randn(n + 2, generator=gen).cuda()
    gbuf = torch.randn(n + 2, generator=gen).cuda()
    pbuf = torch.full((n + 2,), 7.0, dtype=torch.bfloat16, device="cuda")
    m0, g0 = mbuf.cpu().clone(), gbuf.cpu().clone()
    pw.sgd_apply([(pbuf[1:n + 1], mbuf[1:n + 1], gbuf[1:n + 1])], 0.1)
    torch.cuda.synchronize()
    _check_item(oracle32, oracle64, m0[1:n + 1].numpy(), g0[1:n + 1].numpy(), 0.1, 1.0, mbuf[1:n + 1], pbuf[1:n + 1])
    assert mbuf[0].item() == m0[0].item() and mbuf[n + 1].item() == m0[n + 1].item()
    assert pbuf[0].item() == 7.0 and pbuf[n + 1].item() == 7.0
    assert torch.equal(gbuf.cpu(), g0)


def test_sgd_apply_many_items_span_several_launches(pw, oracle32, oracle64):
    gen = torch.Generator().manual_seed(23)
    sizes = [int(s) for s in torch.randint(0, 2 * CHUNK, (150,), generator=gen)]
    sizes[5] = 0
    masters = [torch.randn(n, generator=gen) for n in sizes]
    grads = [torch.randn(n, generator=gen) for n in sizes]
    m_d, g_d = [m.cuda() for m in masters], [g.cuda() for g in grads]
    p_d = [torch.zeros(n, dtype=torch.bfloat16, device="cuda") for n in sizes]
    pw.sgd_apply(list(zip(p_d, m_d, g_d)), 0.3, 0.5)
    torch.cuda.synchronize()
    for n, m0, g, m, p in zip(sizes, masters, grads, m_d, p_d):
        if n:
            _check_item(oracle32, oracle64, m0.numpy(), g.numpy(), 0.3, 0.5, m, p)


def test_sgd_apply_can_create_the_master_copy_from_the_parameters(pw, oracle64):
    gen = torch.Generator().manual_seed(24)
    for n in (5, 3 * CHUNK + 3):
        p0 = torch.randn(n, generator=gen).to(torch.bfloat16)
        g = torch.randn(n, generator=gen)
        p, gd = p0.cuda(), g.cuda()
        m = torch.full((n,), float("nan"), device="cuda")
        pw.sgd_apply([(p, m, gd)], 0.0, init_master=True)               # rate zero: only widen
        torch.cuda.synchronize()
        assert torch.equal(m.cpu(), p0.float()) and torch.equal(p.cpu(), p0)
        m.fill_(float("nan"))
        pw.sgd_apply([(p, m, gd)], 0.125, init_master=True)
        torch.cuda.synchronize()
        want, _ = oracle64.sgd_apply(np64(p0), np64(g), 0.125)
        assert np.all(np.abs(m.cpu().numpy() - want) <= 2.0 ** -23 * np.abs(want) + 1e-45)
        assert torch.equal(p.cpu(), m.cpu().to(torch.bfloat16))


def test_sgd_apply_rejects_bad_arguments(pw):
    p = torch.zeros(8, dtype=torch.bfloat16, device="cuda")
    m, g = torch.zeros(8, device="cuda"), torch.zeros(8, device="cuda")
    with pytest.raises(pw.PwError):
        pw.sgd_apply([(p, m, g)], -1.0)
    with pytest.raises(pw.PwError):
        pw.sgd_apply([(p, m, g)], 0.1, grad_scale=0.0)
    with pytest.raises(pw.PwError):
        pw.sgd_apply([(p, m, g)], float("nan"))
    with pytest.raises(pw.PwError):
        pw.sgd_apply([], 0.1)


def test_training_loop_of_the_small_lm_follows_the_oracle(pw, oracle64):
    """Five steps of (language-model step, gradient apply) on the GPU against the same loop in the
    oracle: the loss of every step agrees and goes down."""
    w = inputs.Workload("lm_small", 256, 4, 64, 1024, 128, 2, n_layers=2, vocab=512)
    L, lr, steps = w.n_layers, 0.1, 5
    cpu_params = [inputs.layer_params(w, 0, l, random_ln=True) for l in range(L)]
    E0, g0, b0, ids, labels = inputs.lm_inputs(w, 0, random_ln=True)

    # --- GPU ---
    stage = pw.Stage(L, w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch)
    params = [[p.cuda() for p in ps] for ps in cpu_params]
    ends = [E0.cuda(), g0.cuda(), b0.cuda()]
    grads = [[torch.zeros(p.shape, dtype=torch.float32, device="cuda") for p in ps] for ps in params]
    end_grads = [torch.zeros(t.shape, dtype=torch.float32, device="cuda") for t in ends]
    flat_p = [p for ps in params for p in ps] + ends
    flat_g = [g for gs in grads for g in gs] + end_grads
    flat_m = [torch.full(p.shape, float("nan"), dtype=torch.float32, device="cuda") for p in flat_p]
    loss = torch.zeros(1, device="cuda")
    ws = torch.empty(stage.lm_workspace_bytes(w.vocab, False), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    got = []
    with torch.cuda.stream(stream):
        for s in range(steps):
            stage.lm_step(params, grads, tuple(ends), end_grads, ids.cuda(), labels.cuda(), loss, w.vocab, ws, False,
                          stream=stream)
            got.append(loss.clone())
            pw.sgd_apply(list(zip(flat_p, flat_m, flat_g)), lr, init_master=(s == 0), stream=stream)
    torch.cuda.synchronize()
    assert stage.status() == (0, 0)
    got = [x.item() for x in got]

    # --- oracle ---
    D = dims_of(w)
    rt = oracle64.round_bf16
    work = [[np64(p) for p in ps] for ps in cpu_params]
    wE, wg, wb = np64(E0), np64(g0), np64(b0)
    master = [[p.copy() for p in ps] for ps in work]
    mE, mg, mb = wE.copy(), wg.copy(), wb.copy()
    want = []
    for s in range(steps):
        out = oracle64.lm_step(D, work, wE, wg, wb, ids.numpy().ravel(), labels.numpy().ravel(), handoff=rt)
        want.append(out["loss"])
        new = [[oracle64.sgd_apply(m, g, lr) for m, g in zip(ml, gl)] for ml, gl in zip(master, out["grads"])]
        master = [[x[0] for x in l] for l in new]
        work = [[x[1] for x in l] for l in new]
        mE, wE = oracle64.sgd_apply(mE, out["dE"], lr)
        mg, wg = oracle64.sgd_apply(mg, out["dlnf_gamma"], lr)
        mb, wb = oracle64.sgd_apply(mb, out["dlnf_beta"], lr)
    for s in range(steps):
        assert abs(got[s] - want[s]) < 3e-3 * want[s], (s, got, want)
    assert all(got[s + 1] < got[s] for s in range(steps - 1)), got
    assert got[0] - got[-1] > 0.3, got
    # the final parameters: the GPU's working copies against the oracle's
    assert rel_l2(ends[0], wE) < 1e-2
    assert rel_l2(params[1][8], work[1][8]) < 1e-2                      # w_fc1 of the last layer
