"""saps_pack_noalloc: the compaction for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is not an option: inside a process whose
framework owns all of the GPU's memory, in a loop that cannot take the device-wide stall
of an allocation, or as a plug-in that is given buffers and a stream and nothing else.
For them the library carries a fixed scratch array of its own.  This test calls the entry
point through the C ABI twice in a row (the second call finds the array as the first one
left it) and wants exactly what the CPU oracle's definition of the compaction gives, and what
saps_pack produces: indices, count and values bit for bit.  Further cases: the largest size
the array covers, a bounded wait that runs out on it, and the refusal of anything larger.

The file name sorts last on purpose: a run that stops at the first failure has then
already been through every other test.
"""
import numpy as np
import pytest

import oracle
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
        # and against the definition itself (Eq. 2): ascending kept columns, their values
        ov, oi, oc = oracle.pack(x, oracle.mask(77, t, p, N), cap)
        assert oc == c
        assert (got_idx.cpu().numpy().view(np.uint32)[:c] == oi[:c]).all()
        assert (got_idx.cpu().numpy()[c:] == -1).all()                      # slots past count untouched
        gv = got_vals.cpu().numpy()
        assert_bits_equal(gv[:, :c], ov[:, :c], f"no-alloc pack against the oracle, call t={t}")
        assert (gv[:, c:] == 123.0).all()
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


def test_noalloc_pack_at_the_largest_size_the_array_covers(sb):
    # N = SAPS_NOALLOC_MAX_N uses every one of the 65,536 tile states of the built-in array
    torch = torch_cuda()
    n, N, seed, t, p = 1, sb.SAPS_NOALLOC_MAX_N, 5, 9, 1e-4
    x = torch.empty(n, N, dtype=torch.float32, device="cuda").normal_(0.0, 1.0)
    ctx = sb.saps_create(n, N, seed)
    cap = sb.saps_pack_capacity(ctx, p)
    vals, idx, count = _outputs(torch, n, cap)
    status = torch.full((1,), 99, dtype=torch.int32, device="cuda")
    sb.saps_pack_noalloc(ctx, x, t, p, vals, idx, count, status)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    m = oracle.mask(seed, t, p, N)                        # the oracle's mask on all 134M columns
    kept = np.nonzero(m)[0].astype(np.uint32)
    c = int(count[0])
    assert c == len(kept) <= cap
    assert (idx.cpu().numpy().view(np.uint32)[:c] == kept).all()
    assert torch.equal(vals[0, :c], x[0, torch.from_numpy(kept.astype(np.int64)).cuda()])
    sb.saps_destroy(ctx)
    del x
    torch.cuda.empty_cache()


def test_noalloc_pack_bounded_wait_runs_out_on_the_static_array(sb):
    # tile 3 never publishes its state; its successors give up after 200 polls and the call
    # reports SAPS_ERR_TIMEOUT through out_status; nothing hangs, the next call is clean
    torch = torch_cuda()
    n, N, p = 2, 40 * 2048, 0.05
    x = synth.gaussian_matrix(n, N, 1.0, 79, 0)
    dx = DeviceMatrix(x, N)
    ctx = sb.saps_create(n, N, 79)
    cap = sb.saps_pack_capacity(ctx, p)
    vals, idx, count = _outputs(torch, n, cap)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sb.saps_debug_inject(ctx, 3, 200)
    sb.saps_pack_noalloc(ctx, dx.ptr, 1, p, vals, idx, count, status)
    torch.cuda.synchronize()
    assert int(status[0]) == sb.SAPS_ERR_TIMEOUT
    sb.saps_debug_inject(ctx, 0xFFFFFFFF, 0)
    vals, idx, count = _outputs(torch, n, cap)
    sb.saps_pack_noalloc(ctx, dx.ptr, 1, p, vals, idx, count, status)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    ov, oi, oc = oracle.pack(x, oracle.mask(79, 1, p, N), cap)
    assert int(count[0]) == oc
    assert (idx.cpu().numpy().view(np.uint32)[:oc] == oi[:oc]).all()
    assert_bits_equal(vals.cpu().numpy()[:, :oc], ov[:, :oc], "clean call after a timed-out one")
    sb.saps_destroy(ctx)
