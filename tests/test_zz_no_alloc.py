"""The allocation-free column-sum entry point against the allocating one (collected last on purpose).

pw_op_colsum_noalloc exists for callers that are not allowed to allocate device memory at the
moment they call in (a server whose pools own all of HBM, a host callback, a plugin that gets
buffers but no allocator); its scratch is a fixed array inside the library.  The check is the
existing pw_op_colsum on the same input, twice in a row, because the array is shared between
calls and keeps what the previous call left in it.
"""
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


def _rel(a, b):
    return float((a.double() - b.double()).norm() / b.double().norm())


def test_noalloc_colsum_matches_allocating_entry_point_twice(pw):
    g = torch.Generator().manual_seed(11)
    for call, (T, N) in enumerate([(1000, 3072), (777, 8192)]):      # second call reuses the array with other sizes
        a = (torch.randn((T, N), generator=g)).to(torch.bfloat16).cuda()
        base = torch.randn(N, generator=g).cuda()
        want = base.clone()
        part = torch.empty(pw.op_colsum_scratch_bytes(T, N), dtype=torch.uint8, device="cuda")
        pw.op_colsum(a, want, True, part)                           # existing entry point: want = base + sums
        got = base.clone()
        warm = base.clone()
        pw.op_colsum_noalloc(a, warm, True)                         # the first call on a device looks up the array's address
        torch.cuda.synchronize()
        before, free_before = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        pw.op_colsum_noalloc(a, got, True)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before              # the binding allocated nothing
        assert torch.cuda.mem_get_info()[0] == free_before          # and neither did the library: the device's free memory is unchanged
        assert _rel(got, want) < 1e-5, (call, _rel(got, want))
        over = torch.empty(N, device="cuda")
        pw.op_colsum_noalloc(a, over, False)                        # overwrite mode ignores what `over` held
        torch.cuda.synchronize()
        assert _rel(over, want - base) < 1e-4


def test_noalloc_colsum_rejects_sizes_beyond_its_scratch(pw):
    a = torch.zeros((1, 8), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(8, device="cuda")
    too_wide = 262144 + 8
    status = pw.lib().pw_op_colsum_noalloc(a.data_ptr(), 1, too_wide, too_wide, out.data_ptr(), 0, None)
    assert status == 3                                               # PW_ERR_WORKSPACE_TOO_SMALL, nothing launched
    assert b"262144" in pw.lib().pw_last_error()
