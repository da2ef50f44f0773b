"""One replica of the two-process data-parallel test (run by tests/test_gpu_data_parallel.py):
    python tests/dp_worker.py RANK WORLD PORT OUT_DIR
Both processes use GPU 0; they exchange buffer handles and barriers over gloo.  Their kernels never
wait on one another (the ordering is on the host), so sharing one GPU is only slower, not unsafe."""
import datetime
import os
import sys

import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

SHAPES = [(300, 64), (64,), (8192 + 24,), (5, 7, 11), (40000,)]
STEPS = 3
LR = 0.05


def initial_params():
    g = torch.Generator().manual_seed(1234)
    return [torch.randn(s, generator=g).to(torch.bfloat16) for s in SHAPES]


def grads_of(rank, step):
    g = torch.Generator().manual_seed(1000 * (step + 1) + rank)
    return [torch.randn(s, generator=g) for s in SHAPES]


def main():
    rank, world, port, out_dir = int(sys.argv[1]), int(sys.argv[2]), int(sys.argv[3]), sys.argv[4]
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world,
                            timeout=datetime.timedelta(seconds=90))
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    from paper_2203_12533_b200 import binding, data_parallel
    binding.lib()
    rep = data_parallel.Replica(SHAPES, dev)
    for dst, src in zip(rep.params, initial_params()):
        dst.copy_(src)
    seen = []
    for step in range(STEPS):
        for dst, src in zip(rep.grads, grads_of(rank, step)):
            dst.copy_(src)
        rep.reduce_apply(LR, init_master=(step == 0))
        torch.cuda.synchronize()
        seen.append([p.clone().cpu() for p in rep.params])
    torch.save({"params": seen, "master": rep.master.cpu(), "lo": rep.lo, "hi": rep.hi, "total": rep.total,
                "offsets": rep.offsets, "grads_untouched": all(torch.equal(a.cpu(), b) for a, b in zip(rep.grads, grads_of(rank, STEPS - 1)))},
               os.path.join(out_dir, f"rank{rank}.pt"))
    rep.close()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
