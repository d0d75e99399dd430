"""spws_row_pointer_static: the row-pointer scan for callers that cannot allocate on the device.

A host application may own all GPU memory through its own allocator, or run this library from a
place where cudaMalloc's device-wide synchronisation (or any allocation call at all) is not
acceptable.  For them the library carries the scan's partial sums in a fixed array of its own,
and the entry point takes only inputs and outputs.  Here it is called twice in a row, through
the C ABI, and must reproduce the row pointer that spws_symbolic (which uses caller-supplied
scratch) writes for the same operands: integers, so bit for bit.

Collected last on purpose: a stop-at-first-failure run has already seen every other test.
"""
import numpy as np
import pytest

from workloads import rmat_csr, uniform_rows_csr

pytestmark = pytest.mark.gpu


def test_static_row_pointer_matches_symbolic_twice():
    import torch
    from paper_2404_04541_b200 import api, binding

    ctx = api.Context("cuda")
    stream = torch.cuda.current_stream().cuda_stream
    cases = [rmat_csr(12, 16, 5), uniform_rows_csr(5000, 5000, 8, 6)]   # several scan tiles + a ragged tail
    for A in cases:
        dA = api.DeviceCSR.from_host(A)
        plan = ctx.plan(api.EXPR_SPGEMM, (binding.SPWS_CSR,) * 3, np.float64, "auto")
        c, _ = ctx.spgemm_symbolic(plan, dA, dA)                        # existing entry point
        want = c.pos[1].clone()
        plan.close()
        counts = (want[1:] - want[:-1]).to(torch.int32).contiguous()
        n = counts.numel()
        for call in range(2):                                           # the shared array is reused
            pos = torch.full((n + 1,), -7, dtype=torch.int64, device="cuda")
            st = binding.row_pointer_static(counts.data_ptr(), n, pos.data_ptr(), stream)
            assert st == binding.SPWS_OK, binding.status_string(st)
            torch.cuda.synchronize()
            assert torch.equal(pos, want), f"call {call}"
    # a different, smaller problem right after a larger one: stale partial sums must not leak in
    small = torch.arange(1, 4, dtype=torch.int32, device="cuda")
    pos = torch.empty(4, dtype=torch.int64, device="cuda")
    assert binding.row_pointer_static(small.data_ptr(), 3, pos.data_ptr(), stream) == binding.SPWS_OK
    torch.cuda.synchronize()
    assert pos.tolist() == [0, 1, 3, 6]
    # empty input and the size limit
    one = torch.empty(1, dtype=torch.int64, device="cuda")
    assert binding.row_pointer_static(0, 0, one.data_ptr(), stream) == binding.SPWS_OK
    torch.cuda.synchronize()
    assert one.item() == 0
    st = binding.row_pointer_static(small.data_ptr(), binding.STATIC_MAX_ROWS + 1, pos.data_ptr(), stream)
    assert st == binding.SPWS_SCRATCH_TOO_SMALL


@pytest.mark.parametrize("n", [(1 << 21) + 3, 16777216])
def test_static_row_pointer_many_tiles_and_the_largest_size(n):
    """More than 1024 scan tiles (the single block that scans the partial sums then loops and
    carries a running total) and the largest size the fixed array admits, each twice so that the
    second call meets what the first one left in the array, and then a small call after them."""
    import torch
    from paper_2404_04541_b200 import binding

    assert n <= binding.STATIC_MAX_ROWS
    stream = torch.cuda.current_stream().cuda_stream
    g = torch.Generator(device="cuda").manual_seed(n)
    for call in range(2):
        counts = torch.randint(0, 9 + call, (n,), dtype=torch.int32, device="cuda", generator=g)
        pos = torch.full((n + 1,), -7, dtype=torch.int64, device="cuda")
        st = binding.row_pointer_static(counts.data_ptr(), n, pos.data_ptr(), stream)
        assert st == binding.SPWS_OK, binding.status_string(st)
        torch.cuda.synchronize()
        assert pos[0].item() == 0
        assert torch.equal(pos[1:], torch.cumsum(counts, 0, dtype=torch.int64)), f"call {call}"
    small = torch.arange(1, 4, dtype=torch.int32, device="cuda")
    pos = torch.empty(4, dtype=torch.int64, device="cuda")
    assert binding.row_pointer_static(small.data_ptr(), 3, pos.data_ptr(), stream) == binding.SPWS_OK
    torch.cuda.synchronize()
    assert pos.tolist() == [0, 1, 3, 6]


def test_static_row_pointer_counts_that_overflow_32_bits_inside_one_tile():
    """Counts near 2^31 - 1: the running sum inside a tile of 2048 counts passes 2^32."""
    import torch
    from paper_2404_04541_b200 import binding

    stream = torch.cuda.current_stream().cuda_stream
    n = 5000
    counts = torch.full((n,), 2**31 - 1, dtype=torch.int32, device="cuda")
    counts[::7] = 3
    pos = torch.empty(n + 1, dtype=torch.int64, device="cuda")
    assert binding.row_pointer_static(counts.data_ptr(), n, pos.data_ptr(), stream) == binding.SPWS_OK
    torch.cuda.synchronize()
    assert pos[0].item() == 0
    assert torch.equal(pos[1:], torch.cumsum(counts, 0, dtype=torch.int64))
