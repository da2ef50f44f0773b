"""One pipeline stage of the two-process test (run by tests/test_gpu_data_parallel.py):
    python tests/pp_worker.py RANK WORLD PORT OUT_DIR
Both stages use GPU 0 and signal each other over gloo; no kernel waits on another."""
import datetime
import os
import sys

import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

LAYERS_PER_STAGE, MICRO = 2, 3


def workload():
    from paper_2203_12533_b200 import inputs
    return inputs.Workload("pp_small", 256, 2, 128, 512, 128, 2, n_layers=4, n_microbatches=MICRO)


def main():
    rank, world, port, out_dir = int(sys.argv[1]), int(sys.argv[2]), int(sys.argv[3]), sys.argv[4]
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world,
                            timeout=datetime.timedelta(seconds=90))
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    from paper_2203_12533_b200 import binding, inputs, pipeline_parallel
    binding.lib()
    w = workload()
    layer = binding.Layer(w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch)
    st = pipeline_parallel.PipelineStage(layer, LAYERS_PER_STAGE, MICRO, dev)
    mine = range(rank * LAYERS_PER_STAGE, (rank + 1) * LAYERS_PER_STAGE)
    params = [[p.to(dev) for p in inputs.layer_params(w, 0, l, random_ln=True)] for l in mine]
    grads = [[torch.full(p.shape, float("nan"), dtype=torch.float32, device=dev) for p in ps] for ps in params]
    for m in range(MICRO):
        x, dy = inputs.microbatch(w, 0, m)
        if st.is_first:
            st.x_in[m].copy_(x.view(-1, w.d_model))
        if st.is_last:
            st.dy_in[m].copy_(dy.view(-1, w.d_model))
    torch.cuda.synchronize()
    dist.barrier()
    st.run(params, grads)
    torch.cuda.synchronize()
    out = {"grads": [[g.cpu() for g in gs] for gs in grads], "status": layer.status(), "signals": st.signals}
    if st.is_last:
        out["y"] = [t.cpu() for t in st.y_out]
    if st.is_first:
        out["dx"] = [t.cpu() for t in st.dx_out]
    torch.save(out, os.path.join(out_dir, f"stage{rank}.pt"))
    st.close()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
