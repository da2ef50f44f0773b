"""The whole-layer kernels (PW_FLAG_WHOLE_LAYER: forward and backward are one cooperative launch each)
against the CPU oracle, against the default multi-kernel path, and inside the stage chain."""
import pytest
import torch

from paper_2203_12533_b200 import inputs
from tests.gpu_util import make_layer, rel_l2, run_layer_gpu
from tests.test_gpu_layer import check_layer_against_oracle, run_chain_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pw():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2203_12533_b200 import binding
    binding.lib()
    return binding


def test_workload1_every_tensor_against_the_oracle(pw, oracle64):
    """Workload 1 (the shape this path exists for): y, all 12 saved tensors, dx and all 12 gradients."""
    w = inputs.WORKLOADS[1]
    check_layer_against_oracle(pw, oracle64, w, flags=pw.FLAG_WHOLE_LAYER)
    check_layer_against_oracle(pw, oracle64, w, random_ln=True, act=1, flags=pw.FLAG_WHOLE_LAYER)
    check_layer_against_oracle(pw, oracle64, w, random_ln=True, save_ctx=False, flags=pw.FLAG_WHOLE_LAYER)   # recompute


@pytest.mark.parametrize("d,H,F,S,B", [(512, 8, 1536, 256, 3), (256, 4, 640, 384, 1), (512, 8, 2048, 128, 5)],
                         ids=["d512_S256_B3", "d256_F640_S384", "d512_S128_B5"])
def test_other_small_shapes(pw, oracle64, d, H, F, S, B):
    """Widths on both sides of the LayerNorm lane split, K ranges that are cut in 1 ... 8 slices, several
    key blocks per head (S = 384: six), token counts that are not a power of two."""
    w = inputs.Workload("small", d, H, 64, F, S, B, sigma_w=0.05)
    check_layer_against_oracle(pw, oracle64, w, random_ln=True, flags=pw.FLAG_WHOLE_LAYER)


def test_agrees_with_the_default_path_and_repeats_bitwise(pw):
    w = inputs.WORKLOADS[1].with_(seq_len=256)
    params = [p.cuda() for p in inputs.layer_params(w, random_ln=True)]
    x, dy = inputs.microbatch(w)
    x, dy = x.cuda().view(-1, w.d_model), dy.cuda().view(-1, w.d_model)
    ref = run_layer_gpu(pw, make_layer(pw, w), params, x, dy)
    layer = make_layer(pw, w, flags=pw.FLAG_WHOLE_LAYER)
    a = run_layer_gpu(pw, layer, params, x, dy, save_ctx=True)
    b = run_layer_gpu(pw, layer, params, x, dy, save_ctx=False)
    c = run_layer_gpu(pw, layer, params, x, dy, save_ctx=True)
    assert layer.launch_count() == 2 + 3 + 2                  # forward + backward; recompute adds one forward
    for other in (b, c):
        assert torch.equal(a["y"], other["y"]) and torch.equal(a["dx"], other["dx"])
        for g1, g2 in zip(a["grads"], other["grads"]):
            assert torch.equal(g1, g2)
    assert rel_l2(a["y"], ref["y"].double()) < 4e-3 and rel_l2(a["dx"], ref["dx"].double()) < 2e-2
    for name, g1, g2 in zip(pw.PARAM_NAMES, a["grads"], ref["grads"]):
        assert rel_l2(g1, g2.double()) < 2e-2, name
    # accumulate adds; dx may alias dy
    acc = run_layer_gpu(pw, layer, params, x, dy, grads=[g.clone() for g in a["grads"]], accumulate=True)
    for g1, g2 in zip(a["grads"], acc["grads"]):
        assert rel_l2(g2, 2 * g1.double()) < 1e-6
    y = torch.empty_like(x)
    ctx = torch.empty(layer.ctx_bytes, dtype=torch.uint8, device="cuda")
    scratch = torch.empty(layer.scratch_bytes, dtype=torch.uint8, device="cuda")
    g = dy.clone()
    grads = [torch.empty_like(t) for t in a["grads"]]
    layer.fwd(params, x, y, ctx, scratch)
    layer.bwd(params, x, g, g, grads, False, ctx, scratch)
    torch.cuda.synchronize()
    assert torch.equal(g, a["dx"]) and layer.status() == (0, 0)


def test_chain_in_every_dispatch_mode(pw, oracle64):
    """A 3-layer, 2-micro-batch chain of whole-layer calls: one launch per call (also as nodes of the
    replayed graph), the same bits in every dispatch mode, schedule and save mode, and the default
    path's results within rounding."""
    w = inputs.WORKLOADS[1].with_(seq_len=256, batch=1)
    L, M = 3, 2
    counts = []
    ref = run_chain_gpu(pw, w, L, M, pw.DISPATCH_ASYNC, pw.SCHEDULE_GPIPE, True, flags=pw.FLAG_WHOLE_LAYER, counts=counts)
    assert counts == [3 * L * M]                              # forward, recomputed forward, backward
    for dispatch, schedule, recompute, n in [(pw.DISPATCH_OPBYOP, pw.SCHEDULE_GPIPE, True, 3),
                                             (pw.DISPATCH_GRAPH, pw.SCHEDULE_GPIPE, True, 3),
                                             (pw.DISPATCH_ASYNC, pw.SCHEDULE_PER_MICROBATCH, False, 2),
                                             (pw.DISPATCH_GRAPH, pw.SCHEDULE_PER_MICROBATCH, False, 2)]:
        counts = []
        other = run_chain_gpu(pw, w, L, M, dispatch, schedule, recompute, flags=pw.FLAG_WHOLE_LAYER, counts=counts)
        assert counts == [n * L * M], (dispatch, counts)
        for m in range(M):
            assert torch.equal(ref[0][m], other[0][m]) and torch.equal(ref[1][m], other[1][m]), (dispatch, schedule, recompute)
        for l in range(L):
            for g1, g2 in zip(ref[2][l], other[2][l]):
                assert torch.equal(g1, g2), (dispatch, schedule, recompute)
    base = run_chain_gpu(pw, w, L, M, pw.DISPATCH_ASYNC, pw.SCHEDULE_GPIPE, True)
    for m in range(M):
        assert rel_l2(ref[0][m], base[0][m].double()) < 1e-2 and rel_l2(ref[1][m], base[1][m].double()) < 3e-2
    for l in range(L):
        for name, g1, g2 in zip(pw.PARAM_NAMES, ref[2][l], base[2][l]):
            assert rel_l2(g1, g2.double()) < 3e-2, (l, name)


def test_unsupported_shapes_are_refused_at_create(pw):
    with pytest.raises(pw.PwError) as e:
        pw.Layer(256, 2, 128, 1024, 128, 2, flags=pw.FLAG_WHOLE_LAYER)           # 128-wide heads
    assert e.value.status == 2
    with pytest.raises(pw.PwError) as e:
        pw.Layer(1024, 16, 64, 4096, 128, 2, flags=pw.FLAG_WHOLE_LAYER)          # too wide for the LayerNorm panel
    assert e.value.status == 2
    with pytest.raises(pw.PwError) as e:
        pw.Layer(256, 4, 64, 1024, 128, 2, flags=pw.FLAG_WHOLE_LAYER | pw.FLAG_LEAN_CTX)
    assert e.value.status == 1
