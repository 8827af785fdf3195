"""saps_pack_noalloc: the compaction for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is not an option: inside a process whose
framework owns all of the GPU's memory, in a loop that cannot take the device-wide stall
of an allocation, or as a plug-in that is given buffers and a stream and nothing else.
For them the library carries a fixed scratch array of its own.  This test calls the entry
point through the C ABI twice in a row (the second call finds the array as the first one
left it) and wants exactly what saps_pack produces: indices, count and values bit for bit.

The file name sorts last on purpose: a run that stops at the first failure has then
already been through every other test.
"""
import numpy as np
import pytest

from paper_2002_09692_b200 import synth
from gpu_util import DeviceMatrix, assert_bits_equal, round_up, torch_cuda

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sb():
    torch_cuda()
    from paper_2002_09692_b200 import binding
    return binding


def _outputs(torch, n, cap):
    return (torch.full((n, cap), 123.0, dtype=torch.float32, device="cuda"),
            torch.full((cap,), -1, dtype=torch.int32, device="cuda"),
            torch.full((1,), -1, dtype=torch.int32, device="cuda"))


def test_noalloc_pack_matches_pack_on_two_calls_in_a_row(sb):
    torch = torch_cuda()
    n, N = 8, 700_001                     # 342 column tiles, ragged last tile
    ld = round_up(N, 32)
    x = synth.gaussian_matrix(n, N, 1.0, 77, 0)
    dx = DeviceMatrix(x, ld)
    ctx = sb.saps_create_ld(n, N, ld, 77)
    status = torch.full((1,), 99, dtype=torch.int32, device="cuda")
    # two different rounds back to back: a larger count first, so stale tile states would show
    for t, p in ((1, 0.05), (2, 0.01)):
        cap = sb.saps_pack_capacity(ctx, p)
        want_vals, want_idx, want_count = _outputs(torch, n, cap)
        sb.saps_pack(ctx, dx.ptr, t, p, want_vals, want_idx, want_count)
        got_vals, got_idx, got_count = _outputs(torch, n, cap)
        sb.saps_pack_noalloc(ctx, dx.ptr, t, p, got_vals, got_idx, got_count, status)
        torch.cuda.synchronize()
        assert sb.saps_status(ctx) == 0
        assert int(status[0]) == 0
        c = int(want_count[0])
        assert 0 < c <= cap
        assert int(got_count[0]) == c
        assert torch.equal(got_idx, want_idx)
        assert_bits_equal(got_vals.cpu().numpy(), want_vals.cpu().numpy(), f"no-alloc pack, call t={t}")
    assert dx.canaries_intact()
    sb.saps_destroy(ctx)


def test_noalloc_pack_reports_overflow_and_refuses_oversize(sb):
    torch = torch_cuda()
    n, N, p = 2, 50_000, 0.2
    x = synth.gaussian_matrix(n, N, 1.0, 78, 0)
    dx = DeviceMatrix(x, N)
    ctx = sb.saps_create(n, N, 78)
    sb.saps_set_pack_capacity(ctx, 1000)
    vals, idx, count = _outputs(torch, n, 1000)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sb.saps_pack_noalloc(ctx, dx.ptr, 1, p, vals, idx, count, status)
    torch.cuda.synchronize()
    assert int(status[0]) == sb.SAPS_ERR_OVERFLOW and int(count[0]) > 1000
    # the next call starts clean
    sb.saps_set_pack_capacity(ctx, 0)
    cap = sb.saps_pack_capacity(ctx, p)
    vals, idx, count = _outputs(torch, n, cap)
    sb.saps_pack_noalloc(ctx, dx.ptr, 1, p, vals, idx, count, status)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    sb.saps_destroy(ctx)
    # a context beyond the static area's reach is refused on the host, nothing is launched
    big = sb.saps_create(2, sb.SAPS_NOALLOC_MAX_N + 1, 0)
    rc = sb._lib.saps_pack_noalloc(big, 0x1000, 1, 0.5, 0x1000, None, 0x1000, None, None)
    assert rc == sb.SAPS_ERR_TOO_LARGE
    assert "static scratch" in sb.saps_strerror(rc)
    sb.saps_destroy(big)
