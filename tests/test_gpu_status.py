"""The failure path on a live GPU, without hanging or faulting it: a wait that nothing will ever
satisfy runs into its (short) limit, the kernel records PW_ERR_TIMEOUT and returns, the host
reads the status word, and the context keeps working."""
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pw():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2203_12533_b200 import binding
    binding.lib()
    return binding


def test_bounded_wait_gives_up_reports_and_leaves_the_context_usable(pw):
    pw.op_status_reset()
    assert pw.op_status() == (0, 0)
    assert pw.op_selftest_wait_timeout(2_000_000) == 1          # about a millisecond of waiting, then the kernel goes on
    assert pw.op_status() == (6, 990)                           # PW_ERR_TIMEOUT at the self-test's site
    pw.op_status_reset()
    assert pw.op_status() == (0, 0)
    # the same context still computes: a small column sum through the library
    x = torch.ones((64, 256), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(256, device="cuda")
    scratch = torch.empty(pw.op_colsum_scratch_bytes(64, 256), dtype=torch.uint8, device="cuda")
    pw.op_colsum(x, out, False, scratch)
    torch.cuda.synchronize()
    assert torch.equal(out, torch.full((256,), 64.0, device="cuda"))
    assert pw.op_status() == (0, 0)


def test_injected_launch_failure_is_reported_and_nothing_of_that_launch_runs(pw):
    """Host-side fault injection: the library's launch wrapper is told to refuse the k-th launch
    before enqueueing it.  The call returns PW_ERR_CUDA with a message naming the kernel family,
    the launch counter shows only the launches that really went out, the output of the refused
    launch is untouched, the device status stays clean and the next call works."""
    from paper_2203_12533_b200 import inputs
    from tests.gpu_util import make_layer
    w = inputs.WORKLOADS[1]
    layer = make_layer(pw, w)
    params = [p.cuda() for p in inputs.layer_params(w)]
    x, _ = inputs.microbatch(w)
    x = x.cuda().view(-1, w.d_model)
    ctx = torch.empty(layer.ctx_bytes, dtype=torch.uint8, device="cuda")
    scratch = torch.empty(layer.scratch_bytes, dtype=torch.uint8, device="cuda")
    y = torch.full_like(x, 7.0)
    for k, family in ((1, "layernorm"), (2, "gemm")):           # first launch of the forward is LN1, second the QKV GEMM
        n0 = layer.launch_count()
        pw.set_tuning(pw.TUNE_FAIL_LAUNCH, k)
        with pytest.raises(pw.PwError) as e:
            layer.fwd(params, x, y, ctx, scratch)
        assert e.value.status == 4                              # PW_ERR_CUDA
        assert family in str(e.value).lower()
        assert pw.get_tuning(pw.TUNE_FAIL_LAUNCH) == 0          # one shot
        assert layer.launch_count() - n0 == k - 1               # only the launches before the refused one
        torch.cuda.synchronize()
        assert torch.equal(y, torch.full_like(x, 7.0))          # the last GEMM, which writes y, never ran
        assert layer.status() == (0, 0)
    n0 = layer.launch_count()
    layer.fwd(params, x, y, ctx, scratch)
    torch.cuda.synchronize()
    assert layer.launch_count() - n0 == 7 and layer.status() == (0, 0)
    assert not torch.equal(y, torch.full_like(x, 7.0)) and torch.isfinite(y.float()).all()


def test_info_log_and_nvtx_ranges_on_a_live_step(pw):
    """With the log sink at INFO and NVTX ranges on, creating a layer and running a forward produce the
    documented lines and change nothing in the result (no timeline tool is attached: the ranges are calls
    into an empty dispatch table)."""
    from paper_2203_12533_b200 import inputs
    w = inputs.WORKLOADS[1]
    params = [p.cuda() for p in inputs.layer_params(w, 0, 0)]
    x, _ = inputs.microbatch(w, 0, 0)
    xd = x.cuda().view(-1, w.d_model)

    def forward():
        layer = pw.Layer(w.d_model, w.n_heads, w.head_dim, w.d_ff, w.seq_len, w.batch)
        y = torch.empty_like(xd)
        ctx = torch.empty(layer.ctx_bytes, dtype=torch.uint8, device="cuda")
        scratch = torch.empty(layer.scratch_bytes, dtype=torch.uint8, device="cuda")
        layer.fwd(params, xd, y, ctx, scratch)
        torch.cuda.synchronize()
        assert layer.status() == (0, 0)
        return y

    want = forward()
    lines = []
    pw.set_log(pw.LOG_INFO, lambda level, msg: lines.append((level, msg)))
    pw.set_tuning(pw.TUNE_NVTX, 1)
    try:
        got = forward()
    finally:
        pw.set_tuning(pw.TUNE_NVTX, 0)
        pw.set_log(pw.LOG_OFF)
    assert torch.equal(got, want)
    assert any(level == pw.LOG_INFO and msg.startswith("pw_layer_create: d_model 256, 4 heads x 64") for level, msg in lines)
    assert not any(level == pw.LOG_ERROR for level, _ in lines)
