"""GPU tests of the data-parallel gradient apply over peer memory: replicas emulated inside one
process (every "peer" buffer is local), and two real processes that map each other's buffers
(both on GPU 0, ordering over gloo).  No kernel here waits on another."""
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch

from tests import dp_worker
from tests.gpu_util import np64, rel_l2

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def pw():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2203_12533_b200 import binding
    binding.lib()
    return binding


def _check(oracle64, m0, grads, lr, scale, m_gpu, p_gpu):
    """m_gpu (fp32) and p_gpu (bf16 as fp32) against the oracle's step on the summed gradient."""
    want, _ = oracle64.dp_sgd_apply(m0, grads, lr, scale)
    mag = np.abs(m0) + lr * scale * sum(np.abs(g) for g in grads)
    assert np.all(np.abs(m_gpu - want) <= 2.0 ** -22 * mag + 1e-45)       # fp32 sum in rank order, one FMA
    assert np.array_equal(p_gpu, torch.from_numpy(m_gpu.astype(np.float32)).to(torch.bfloat16).float().numpy())


@pytest.mark.parametrize("world,n", [(1, 4099), (3, 50003), (8, 8 * 8192 + 8), (4, 5)])
def test_emulated_replicas_reduce_apply(pw, oracle64, world, n):
    gen = torch.Generator().manual_seed(31 + world)
    p0 = torch.randn(n, generator=gen).to(torch.bfloat16)
    grads = [torch.randn(n, generator=gen) for _ in range(world)]
    g_d = [g.cuda() for g in grads]
    p_d = [p0.clone().cuda() for _ in range(world)]
    slices = [pw.dp_slice(n, world, r) for r in range(world)]
    assert slices[0][0] == 0 and slices[-1][1] == n
    assert all(a[1] == b[0] for a, b in zip(slices, slices[1:])) and all(lo % 8 == 0 or lo == n for lo, _ in slices)
    masters = [torch.full((max(hi - lo, 1),), float("nan"), device="cuda") for lo, hi in slices]
    gp, pp = [t.data_ptr() for t in g_d], [t.data_ptr() for t in p_d]
    lr, scale = 0.1, 1.0 / world
    for r in range(world):                                           # one launch per replica, one after the other
        pw.dp_reduce_apply(r, gp, pp, masters[r], n, lr, scale, init_master=True)
    torch.cuda.synchronize()
    for k in range(1, world):
        assert torch.equal(p_d[k], p_d[0])                           # every replica holds the same parameters
    m_gpu = np.concatenate([masters[r][:hi - lo].cpu().numpy() for r, (lo, hi) in enumerate(slices)])
    _check(oracle64, np64(p0), [np64(g) for g in grads], lr, scale, m_gpu, p_d[0].float().cpu().numpy())
    for g, gd in zip(grads, g_d):
        assert torch.equal(gd.cpu(), g)
    # a second step from the masters
    grads2 = [torch.randn(n, generator=gen) for _ in range(world)]
    for gd, g in zip(g_d, grads2):
        gd.copy_(g)
    for r in range(world):
        pw.dp_reduce_apply(r, gp, pp, masters[r], n, lr, scale)
    torch.cuda.synchronize()
    m2 = np.concatenate([masters[r][:hi - lo].cpu().numpy() for r, (lo, hi) in enumerate(slices)])
    _check(oracle64, m_gpu.astype(np.float64), [np64(g) for g in grads2], lr, scale, m2, p_d[-1].float().cpu().numpy())


def test_one_replica_equals_the_plain_apply_bit_for_bit(pw):
    gen = torch.Generator().manual_seed(41)
    n = 3 * 8192 + 11
    p0 = torch.randn(n, generator=gen).to(torch.bfloat16)
    g = torch.randn(n, generator=gen).cuda()
    pa, pb = p0.clone().cuda(), p0.clone().cuda()
    ma, mb = torch.empty(n, device="cuda"), torch.empty(n, device="cuda")
    pw.sgd_apply([(pa, ma, g)], 0.2, 0.5, init_master=True)
    pw.dp_reduce_apply(0, [g.data_ptr()], [pb.data_ptr()], mb, n, 0.2, 0.5, init_master=True)
    torch.cuda.synchronize()
    assert torch.equal(ma, mb) and torch.equal(pa, pb)


def test_reduce_apply_rejects_bad_arguments(pw):
    g, p, m = torch.zeros(16, device="cuda"), torch.zeros(16, dtype=torch.bfloat16, device="cuda"), torch.zeros(16, device="cuda")
    with pytest.raises(pw.PwError):
        pw.dp_reduce_apply(1, [g.data_ptr()], [p.data_ptr()], m, 16, 0.1, 1.0)           # rank outside the world
    with pytest.raises(pw.PwError):
        pw.dp_reduce_apply(0, [g.data_ptr()] * 9, [p.data_ptr()] * 9, m, 16, 0.1, 1.0)   # more than 8 replicas
    with pytest.raises(pw.PwError):
        pw.dp_reduce_apply(0, [g.data_ptr()], [p.data_ptr()], m, 16, 0.1, 0.0)
    with pytest.raises(pw.PwError):
        pw.dp_slice(16, 0, 0)


def test_shared_buffers_round_trip_and_reject_foreign_pointers(pw):
    ptr, handle = pw.shared_alloc(4096)
    assert ptr and len(handle) == 64
    from paper_2203_12533_b200.data_parallel import tensor_at
    t = tensor_at(ptr, 1024, torch.float32, torch.device("cuda", 0))
    t.fill_(3.0)
    assert t.sum().item() == 3072.0 and t.data_ptr() == ptr
    b = tensor_at(ptr, 2048, torch.bfloat16, torch.device("cuda", 0))
    assert b.dtype == torch.bfloat16 and b.data_ptr() == ptr
    del t, b
    with pytest.raises(pw.PwError):
        pw.shared_close(ptr)                                          # not an opened mapping
    with pytest.raises(pw.PwError):
        pw.shared_free(ptr + 256)                                     # not the start of a shared buffer
    pw.shared_free(ptr)
    with pytest.raises(pw.PwError):
        pw.shared_free(ptr)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_processes_map_each_others_buffers(pw, oracle64, tmp_path):
    world, port = 2, _free_port()
    procs = [subprocess.Popen([sys.executable, os.path.join(ROOT, "tests", "dp_worker.py"), str(r), str(world), str(port), str(tmp_path)],
                              cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True) for r in range(world)]
    outs = []
    for p in procs:
        try:
            outs.append(p.communicate(timeout=240)[0])
        except subprocess.TimeoutExpired:
            for q in procs:
                q.kill()
            raise
    assert all(p.returncode == 0 for p in procs), "\n".join(o[-1500:] for o in outs)
    res = [torch.load(os.path.join(tmp_path, f"rank{r}.pt")) for r in range(world)]
    total, offsets = res[0]["total"], res[0]["offsets"]
    assert res[1]["total"] == total and res[0]["lo"] == 0 and res[0]["hi"] == res[1]["lo"] and res[1]["hi"] == total
    assert all(r["grads_untouched"] for r in res)
    flat = lambda ts: np.concatenate([np.pad(np64(t).ravel(), (0, -t.numel() % 8)) for t in ts])
    master = flat(dp_worker.initial_params())
    assert master.size == total
    for step in range(dp_worker.STEPS):
        for a, b in zip(res[0]["params"][step], res[1]["params"][step]):
            assert torch.equal(a, b)                                  # both replicas hold the same parameters
        grads = [flat(dp_worker.grads_of(r, step)) for r in range(world)]
        want_m, want_p = oracle64.dp_sgd_apply(master, grads, dp_worker.LR, 1.0 / world)
        got_p = flat(res[0]["params"][step])
        differ = got_p != want_p                                      # fp32 vs fp64 masters across a rounding tie
        assert differ.mean() < 2e-3
        assert np.all(np.abs(got_p - want_p)[differ] <= 2.0 ** (np.floor(np.log2(np.abs(want_p[differ]) + 1e-30)) - 7) * 1.001)
        master = want_m
    got_m = np.concatenate([res[r]["master"][:res[r]["hi"] - res[r]["lo"]].numpy() for r in range(world)])
    assert np.all(np.abs(got_m - master) <= 1e-6 * (np.abs(master) + 1.0))


def test_lm_training_through_a_replica_matches_separate_tensors(pw):
    """The small language model trained for three steps with all parameters and gradients in a
    replica's flat buffers (one replica: its own gradients only) gives the same losses and the same
    parameters, bit for bit, as with separate tensors and the plain apply."""
    from paper_2203_12533_b200 import data_parallel, inputs
    w = inputs.Workload("lm_small", 256, 4, 64, 1024, 128, 2, n_layers=2, vocab=512)
    L, lr, steps = w.n_layers, 0.1, 3
    cpu_params = [inputs.layer_params(w, 0, l, random_ln=True) for l in range(L)]
    E0, g0, b0, ids, labels = inputs.lm_inputs(w, 0, random_ln=True)
    ids, labels = ids.cuda(), labels.cuda()
    stage = pw.Stage(L, w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch)
    ws = torch.empty(stage.lm_workspace_bytes(w.vocab, False), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()

    def run(params, grads, ends, end_grads, apply):
        loss, losses = torch.zeros(1, device="cuda"), []
        with torch.cuda.stream(stream):
            for s in range(steps):
                stage.lm_step(params, grads, tuple(ends), end_grads, ids, labels, loss, w.vocab, ws, False, stream=stream)
                losses.append(loss.clone())
                apply(s)
        torch.cuda.synchronize()
        assert stage.status() == (0, 0)
        return [x.item() for x in losses]

    # separate tensors
    params = [[p.cuda() for p in ps] for ps in cpu_params]
    ends = [E0.cuda(), g0.cuda(), b0.cuda()]
    grads = [[torch.zeros(p.shape, device="cuda") for p in ps] for ps in params]
    end_grads = [torch.zeros(t.shape, device="cuda") for t in ends]
    flat_p = [p for ps in params for p in ps] + ends
    flat_g = [x for gs in grads for x in gs] + end_grads
    flat_m = [torch.empty(p.shape, device="cuda") for p in flat_p]
    a = run(params, grads, ends, end_grads,
            lambda s: pw.sgd_apply(list(zip(flat_p, flat_m, flat_g)), lr, init_master=(s == 0), stream=stream))

    # one replica's flat buffers
    flat_cpu = [p for ps in cpu_params for p in ps] + [E0, g0, b0]
    rep = data_parallel.Replica([tuple(p.shape) for p in flat_cpu], torch.device("cuda", 0))
    try:
        for dst, src in zip(rep.params, flat_cpu):
            dst.copy_(src)
        per = len(cpu_params[0])
        b = run([rep.params[l * per:(l + 1) * per] for l in range(L)], [rep.grads[l * per:(l + 1) * per] for l in range(L)],
                rep.params[L * per:], rep.grads[L * per:],
                lambda s: rep.reduce_apply(lr, init_master=(s == 0), stream=stream))
        assert a == b and a[-1] < a[0]
        for x, y in zip(flat_p, rep.params):
            assert torch.equal(x, y)
    finally:
        rep.close()


def test_two_pipeline_stages_in_two_processes_match_one_chain(pw, tmp_path):
    """Two stage processes (two layers each, three micro-batches, GPipe) whose last kernels store
    straight into the neighbour's mapped buffers, against the same four layers run as one chain in
    this process: outputs, input gradients and every parameter gradient agree bit for bit."""
    from paper_2203_12533_b200 import inputs
    from tests import pp_worker
    world, port = 2, _free_port()
    procs = [subprocess.Popen([sys.executable, os.path.join(ROOT, "tests", "pp_worker.py"), str(r), str(world), str(port), str(tmp_path)],
                              cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True) for r in range(world)]
    outs = []
    for p in procs:
        try:
            outs.append(p.communicate(timeout=240)[0])
        except subprocess.TimeoutExpired:
            for q in procs:
                q.kill()
            raise
    assert all(p.returncode == 0 for p in procs), "\n".join(o[-1500:] for o in outs)
    res = [torch.load(os.path.join(tmp_path, f"stage{r}.pt")) for r in range(world)]
    assert all(r["status"] == (0, 0) for r in res)
    M = pp_worker.MICRO
    assert res[0]["signals"] == [("send", 1)] * M + [("recv", 1)] * M
    assert res[1]["signals"] == [("recv", 0)] * M + [("send", 0)] * M

    w = pp_worker.workload()
    L = w.n_layers
    stage = pw.Stage(L, w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch)
    params = [[p.cuda() for p in inputs.layer_params(w, 0, l, random_ln=True)] for l in range(L)]
    grads = [[torch.zeros(p.shape, dtype=torch.float32, device="cuda") for p in ps] for ps in params]
    mbs = [inputs.microbatch(w, 0, m) for m in range(M)]
    xs, dys = [x.cuda() for x, _ in mbs], [dy.cuda() for _, dy in mbs]
    ys, dxs = [torch.empty_like(x) for x in xs], [torch.empty_like(x) for x in xs]
    ws = torch.empty(stage.workspace_bytes(M, pw.SCHEDULE_GPIPE, False), dtype=torch.uint8, device="cuda")
    stage.run_chain(params, grads, xs, dys, ys, dxs, ws, schedule=pw.SCHEDULE_GPIPE, recompute=False)
    torch.cuda.synchronize()
    assert stage.status() == (0, 0)
    for m in range(M):
        assert torch.equal(res[1]["y"][m], ys[m].view(-1, w.d_model).cpu())
        assert torch.equal(res[0]["dx"][m], dxs[m].view(-1, w.d_model).cpu())
    per = pp_worker.LAYERS_PER_STAGE
    for l in range(L):
        for got, want in zip(res[l // per]["grads"][l % per], grads[l]):
            assert torch.equal(got, want.cpu())


def test_two_replicas_train_like_one_process_on_the_whole_batch(pw, tmp_path):
    """Two replicas (two sequences each, own tokens, gradients averaged through the mapped buffers)
    against one process that runs all four sequences as one batch with the plain apply: the mean of
    the replica losses follows the whole-batch loss step by step and the parameters end up together
    (different batch shapes round differently, so this is a tolerance check, not a bitwise one)."""
    from tests import dp_lm_worker as wk
    world, port = 2, _free_port()
    procs = [subprocess.Popen([sys.executable, os.path.join(ROOT, "tests", "dp_lm_worker.py"), str(r), str(world), str(port), str(tmp_path)],
                              cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True) for r in range(world)]
    outs = []
    for p in procs:
        try:
            outs.append(p.communicate(timeout=240)[0])
        except subprocess.TimeoutExpired:
            for q in procs:
                q.kill()
            raise
    assert all(p.returncode == 0 for p in procs), "\n".join(o[-1500:] for o in outs)
    res = [torch.load(os.path.join(tmp_path, f"lm_rank{r}.pt")) for r in range(world)]
    assert all(r["status"] == (0, 0) for r in res)
    for a, b in zip(res[0]["params"], res[1]["params"]):
        assert torch.equal(a, b)                                      # replicas stay identical

    w = wk.workload(world * wk.SEQS_PER_REPLICA)
    L = w.n_layers
    layers, ends = wk.initial_parameters()
    params = [[p.cuda() for p in ps] for ps in layers]
    ends = [t.cuda() for t in ends]
    toks = [wk.replica_tokens(r) for r in range(world)]
    ids = torch.cat([t[0] for t in toks]).cuda()
    labels = torch.cat([t[1] for t in toks]).cuda()
    grads = [[torch.zeros(p.shape, device="cuda") for p in ps] for ps in params]
    end_grads = [torch.zeros(t.shape, device="cuda") for t in ends]
    flat_p = [p for ps in params for p in ps] + ends
    flat_g = [x for gs in grads for x in gs] + end_grads
    flat_m = [torch.empty(p.shape, device="cuda") for p in flat_p]
    stage = pw.Stage(L, w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch)
    ws = torch.empty(stage.lm_workspace_bytes(w.vocab, False), dtype=torch.uint8, device="cuda")
    loss, whole = torch.zeros(1, device="cuda"), []
    for s in range(wk.STEPS):
        stage.lm_step(params, grads, tuple(ends), end_grads, ids, labels, loss, w.vocab, ws, False)
        whole.append(loss.item())
        pw.sgd_apply(list(zip(flat_p, flat_m, flat_g)), wk.LR, init_master=(s == 0))
    torch.cuda.synchronize()
    assert stage.status() == (0, 0)
    for s in range(wk.STEPS):
        mean = 0.5 * (res[0]["losses"][s] + res[1]["losses"][s])
        assert abs(mean - whole[s]) < 2e-3 * whole[s], (s, res[0]["losses"], res[1]["losses"], whole)
    assert whole[-1] < whole[0]
    for got, want in zip(res[0]["params"], flat_p):
        assert rel_l2(got.cuda(), np64(want)) < 1e-2
