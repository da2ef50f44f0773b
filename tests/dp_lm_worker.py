"""One data-parallel replica training the small language model (run by tests/test_gpu_data_parallel.py):
    python tests/dp_lm_worker.py RANK WORLD PORT OUT_DIR
Every replica holds the same parameters and draws its own token batch; gradients are summed and
applied through the mapped buffers.  Both processes use GPU 0 and order themselves over gloo."""
import datetime
import os
import sys

import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

STEPS, LR, SEQS_PER_REPLICA = 3, 0.1, 2


def workload(batch):
    from paper_2203_12533_b200 import inputs
    return inputs.Workload("dp_lm", 256, 4, 64, 1024, 128, batch, n_layers=2, vocab=512)


def replica_tokens(rank):
    from paper_2203_12533_b200 import inputs
    _, _, _, ids, labels = inputs.lm_inputs(workload(SEQS_PER_REPLICA), 100 + rank, random_ln=True)
    return ids, labels


def initial_parameters():
    """Per-layer parameter lists and (E, lnf_gamma, lnf_beta): the same on every replica."""
    from paper_2203_12533_b200 import inputs
    w = workload(SEQS_PER_REPLICA)
    layers = [inputs.layer_params(w, 0, l, random_ln=True) for l in range(w.n_layers)]
    E, g, b, _, _ = inputs.lm_inputs(w, 0, random_ln=True)
    return layers, [E, g, b]


def main():
    rank, world, port, out_dir = int(sys.argv[1]), int(sys.argv[2]), int(sys.argv[3]), sys.argv[4]
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world,
                            timeout=datetime.timedelta(seconds=90))
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    from paper_2203_12533_b200 import binding, data_parallel
    binding.lib()
    w = workload(SEQS_PER_REPLICA)
    L = w.n_layers
    layers, ends = initial_parameters()
    flat_cpu = [p for ps in layers for p in ps] + ends
    rep = data_parallel.Replica([tuple(p.shape) for p in flat_cpu], dev)
    for dst, src in zip(rep.params, flat_cpu):
        dst.copy_(src)
    per = len(layers[0])
    params = [rep.params[l * per:(l + 1) * per] for l in range(L)]
    grads = [rep.grads[l * per:(l + 1) * per] for l in range(L)]
    ids, labels = [t.to(dev) for t in replica_tokens(rank)]
    stage = binding.Stage(L, w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch)
    ws = torch.empty(stage.lm_workspace_bytes(w.vocab, False), dtype=torch.uint8, device=dev)
    loss, losses = torch.zeros(1, device=dev), []
    for s in range(STEPS):
        stage.lm_step(params, grads, tuple(rep.params[L * per:]), rep.grads[L * per:], ids, labels, loss, w.vocab, ws, False)
        losses.append(loss.item())
        rep.reduce_apply(LR, init_master=(s == 0))           # mean over the replicas
    torch.cuda.synchronize()
    torch.save({"losses": losses, "params": [p.clone().cpu() for p in rep.params], "status": stage.status()},
               os.path.join(out_dir, f"lm_rank{rank}.pt"))
    rep.close()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
