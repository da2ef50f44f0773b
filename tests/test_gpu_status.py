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
