"""The N > 1 path on CPU: the path does not shard (replicas only), so what more than one rank adds
is the max-over-ranks timing, the whole-job rate, and the rule that only rank 0 reports.  Run as
two gloo ranks on 127.0.0.1."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    my_ms = 2.0 + rank                                   # rank 1 is the slow one
    ms = bench.max_over_ranks(my_ms, world, torch.device("cpu"))
    dist.barrier()
    out[rank] = (ms, bench.whole_job_value(1000.0, world, ms))
    dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time_and_the_whole_job_rate():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, value = res[0]
    assert ms == 3.0                                     # max over ranks, not the mean or rank 0's
    assert abs(value - 2 * 1000.0 / 3.0e-3) < 1e-6       # both replicas' units over the slowest time


def test_one_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.25, 1, torch.device("cpu")) == 1.25


def test_reference_arm_under_torchrun_prints_one_line_from_rank_0():
    """bench.py --impl reference launched as the driver launches it for N = 2: rank 0 runs and prints, rank 1 exits 0."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--workload", "1", "--steps", "2", "--warmup", "1"]
    r = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0


class _FakeLibrary:
    """Stands in for the CUDA library in the host-logic test of the data-parallel replica: buffers
    are numbers, handles name their owner, and every call is recorded."""

    def __init__(self, rank):
        self.rank, self.calls, self.next = rank, [], 1000 * (rank + 1)

    def shared_alloc(self, nbytes):
        self.next += 1
        self.calls.append(("alloc", nbytes))
        return self.next, f"{self.rank}:{self.next}".encode().ljust(64, b"\0")

    def shared_free(self, ptr): self.calls.append(("free", ptr))

    def shared_open(self, handle):
        owner, ptr = handle.rstrip(b"\0").decode().split(":")
        assert int(owner) != self.rank, "a replica must not open its own handle"
        self.calls.append(("open", int(owner), int(ptr)))
        return 100000 * (int(owner) + 1) + int(ptr)

    def shared_close(self, ptr): self.calls.append(("close", ptr))

    def dp_slice(self, n, world, rank):
        per = -(-(-(-n // world)) // 8) * 8
        return min(per * rank, n), min(per * rank + per, n)

    def dp_reduce_apply(self, rank, gp, pp, master, n, lr, scale, init_master=False, stream=None):
        self.calls.append(("apply", rank, tuple(gp), tuple(pp), n, lr, scale, init_master))

    def tensor_at(self, ptr, numel, dtype, device): return torch.zeros(numel, dtype=dtype)

    def empty_master(self, numel, device): return torch.zeros(max(numel, 1))

    def synchronize(self, device, stream=None): self.calls.append(("sync",))


def _replica_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2203_12533_b200 import data_parallel
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    fake = _FakeLibrary(rank)
    rep = data_parallel.Replica([(3, 5), (7,), (16,)], torch.device("cpu"), library=fake)
    rep.reduce_apply(0.5, init_master=True)
    rep.reduce_apply(0.25, grad_scale=1.0)
    info = {"offsets": rep.offsets, "total": rep.total, "slice": (rep.lo, rep.hi), "grad_ptrs": rep.grad_ptrs,
            "param_ptrs": rep.param_ptrs, "shapes": [tuple(t.shape) for t in rep.params]}
    rep.close()
    info["calls"] = fake.calls
    out[rank] = info
    dist.destroy_process_group()


def test_replica_host_logic_with_two_gloo_ranks():
    """Arena layout, slice ownership, handle exchange in rank order, default gradient scale, and the
    close-before-free order, with the CUDA library replaced by a recorder."""
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_replica_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for r in range(world):
        info = res[r]
        assert info["offsets"] == [0, 16, 24] and info["total"] == 40          # 15 -> 16, 7 -> 8, 16
        assert info["shapes"] == [(3, 5), (7,), (16,)]
        own_g, own_p = 1000 * (r + 1) + 1, 1000 * (r + 1) + 2
        other = 1 - r
        peer_g, peer_p = 100000 * (other + 1) + 1000 * (other + 1) + 1, 100000 * (other + 1) + 1000 * (other + 1) + 2
        want_g = [own_g, peer_g] if r == 0 else [peer_g, own_g]
        want_p = [own_p, peer_p] if r == 0 else [peer_p, own_p]
        assert info["grad_ptrs"] == want_g and info["param_ptrs"] == want_p      # rank order, own buffer at own rank
        applies = [c for c in info["calls"] if c[0] == "apply"]
        assert applies[0] == ("apply", r, tuple(want_g), tuple(want_p), 40, 0.5, 0.5, True)    # scale defaults to 1 / world
        assert applies[1] == ("apply", r, tuple(want_g), tuple(want_p), 40, 0.25, 1.0, False)
        names = [c[0] for c in info["calls"]]
        assert names.count("open") == 2 and names.count("close") == 2 and names.count("free") == 2
        assert max(i for i, n in enumerate(names) if n == "close") < min(i for i, n in enumerate(names) if n == "free")
        # a host synchronise before each barrier around each apply (gloo backend: host ordering)
        first_apply = names.index("apply")
        assert "sync" in names[:first_apply] and "sync" in names[first_apply + 1:]
    assert res[0]["slice"] == (0, 24) and res[1]["slice"] == (24, 40)


class _FakeLayer:
    T, d, ctx_bytes, scratch_bytes = 4, 8, 16, 16

    def __init__(self): self.calls = []

    def fwd(self, params, x, y, ctx, scratch, stream=None):
        self.calls.append(("fwd", params, y if isinstance(y, int) else "local"))

    def bwd(self, params, x, dy, dx, grads, accumulate, ctx, scratch, stream=None):
        self.calls.append(("bwd", params, dx if isinstance(dx, int) else "local", bool(accumulate)))


def _stage_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2203_12533_b200 import pipeline_parallel
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    fake, layer = _FakeLibrary(rank), _FakeLayer()
    st = pipeline_parallel.PipelineStage(layer, 2, 3, torch.device("cpu"), library=fake)
    st.run(["p0", "p1"], ["g0", "g1"], stream="s")
    out[rank] = {"signals": st.signals, "calls": layer.calls, "lib": fake.calls, "first": st.is_first, "last": st.is_last,
                 "y_ptrs": st._y_ptrs, "dx_ptrs": st._dx_ptrs,
                 "own_y": [t.data_ptr() for t in st.y_out] if st.is_last else None,
                 "own_dx": [t.data_ptr() for t in st.dx_out] if st.is_first else None}
    st.close()
    dist.destroy_process_group()


def test_pipeline_stage_host_logic_with_three_gloo_ranks():
    """Three stages, two layers each, three micro-batches: GPipe order of the layer calls, the last
    kernel of a stage writes into the neighbour's mapped buffer, gradients accumulate from the
    second micro-batch on, and the send / receive pattern cannot deadlock (it completes)."""
    world, port = 3, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_stage_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    M = 3
    assert res[0]["signals"] == [("send", 1)] * M + [("recv", 1)] * M
    assert res[1]["signals"] == [("recv", 0), ("send", 2)] * M + [("recv", 2), ("send", 0)] * M
    assert res[2]["signals"] == [("recv", 1)] * M + [("send", 1)] * M
    act_bytes = _FakeLayer.T * _FakeLayer.d * 2
    for r in range(world):
        calls = res[r]["calls"]
        fw, bw = [c for c in calls if c[0] == "fwd"], [c for c in calls if c[0] == "bwd"]
        assert calls == fw + bw and len(fw) == 2 * M and len(bw) == 2 * M          # all forwards first
        assert [c[1] for c in fw] == ["p0", "p1"] * M and [c[1] for c in bw] == ["p1", "p0"] * M
        assert [c[3] for c in bw] == [False, False] + [True] * 4                    # overwrite, then accumulate
        opens = [c for c in res[r]["lib"] if c[0] == "open"]
        if r < world - 1:                                                           # y of the last layer: next stage's x_in
            base = 100000 * (r + 2) + 1000 * (r + 2) + 1
            assert res[r]["y_ptrs"] == [base + m * act_bytes for m in range(M)]
            assert [c[2] for c in fw[1::2]] == res[r]["y_ptrs"] and ("open", r + 1, 1000 * (r + 2) + 1) in opens
        else:
            assert [c[2] for c in fw[1::2]] == res[r]["own_y"] and all(c[2] == "local" for c in fw[0::2])
        if r > 0:                                                                   # dx of the first layer: previous stage's dy_in
            base = 100000 * r + 1000 * r + 2
            assert res[r]["dx_ptrs"] == [base + m * act_bytes for m in range(M)]
            assert [c[2] for c in bw[1::2]] == res[r]["dx_ptrs"] and ("open", r - 1, 1000 * r + 2) in opens
        else:
            assert [c[2] for c in bw[1::2]] == res[r]["own_dx"] and all(c[2] == "local" for c in bw[0::2])
        assert len(opens) == (1 if r in (0, world - 1) else 2)
