"""GPU parity of mask bitmap, compaction and the fused emission against the CPU oracle."""
import numpy as np
import pytest

import oracle
from paper_2002_09692_b200 import synth
from gpu_util import DeviceMatrix, assert_bits_equal, bits_from_mask, round_up, torch_cuda

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=["auto", "bulk"])
def staging(request, monkeypatch):
    # every test of this file runs with the default choice of the round's staging and with the
    # bulk-copy form forced (the default only picks it for launches of several thousand blocks)
    from gpu_util import force_staging
    force_staging(monkeypatch, request.param)


@pytest.fixture(scope="module")
def sb():
    torch_cuda()
    from paper_2002_09692_b200 import binding
    return binding


@pytest.mark.parametrize("N", [1, 31, 32, 33, 255, 256, 257, 2048, 2049, 65_536, 272_474, 1_000_003])
def test_mask_bitmap(sb, N):
    torch = torch_cuda()
    for seed, t, p in ((0, 1, 0.1), (1, 1, 0.01), (2, 20, 0.5), (0xDEADBEEFCAFEF00D, 2 ** 32 + 5, 0.001),
                       (3, 3, 1.0), (3, 3, 0.0)):
        words = round_up(N, 32) // 32
        bits = torch.full((words + 2,), -1, dtype=torch.int32, device="cuda")
        ctx = sb.saps_create(2, N, seed)
        sb.saps_mask(ctx, t, p, bits)
        torch.cuda.synchronize()
        sb.saps_destroy(ctx)
        got = bits.cpu().numpy().view(np.uint32)
        want = bits_from_mask(oracle.mask(seed, t, p, N))
        assert (got[:words] == want).all(), (N, seed, t, p)
        assert (got[words:] == 0xFFFFFFFF).all()       # nothing written past the last word


def test_mask_golden_columns_on_gpu(sb):
    # the golden first/last kept columns of the tiny configuration come out of the CUDA hash
    torch = torch_cuda()
    N = 65_536
    ctx = sb.saps_create(4, N, 0)
    bits = torch.zeros(N // 32, dtype=torch.int32, device="cuda")
    for t, count, first, last in ((1, 6617, [12, 15, 32, 40, 45, 70, 72, 111], 65520),
                                  (2, 6765, [59, 68, 80, 116], 65528), (3, 6648, [0, 21, 43, 46], 65529)):
        sb.saps_mask(ctx, t, 0.1, bits)
        m = np.unpackbits(bits.cpu().numpy().view(np.uint8), bitorder="little")
        idx = np.nonzero(m)[0]
        assert len(idx) == count and list(idx[:len(first)]) == first and idx[-1] == last
    sb.saps_destroy(ctx)


def _pack_both(sb, n, N, ld, p, seed, t, with_idx=True, cap_override=0):
    torch = torch_cuda()
    x = synth.gaussian_matrix(n, N, 1.0, seed + 3, 0)
    dx = DeviceMatrix(x, ld)
    ctx = sb.saps_create_ld(n, N, ld, seed)
    if cap_override:
        sb.saps_set_pack_capacity(ctx, cap_override)
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.full((n * cap + 32,), 123.0, dtype=torch.float32, device="cuda")
    idx = torch.full((cap + 32,), -1, dtype=torch.int32, device="cuda")
    count = torch.full((2,), -1, dtype=torch.int32, device="cuda")
    sb.saps_pack(ctx, dx.ptr, t, p, vals, idx if with_idx else None, count)
    torch.cuda.synchronize()
    status = sb.saps_status(ctx)
    sb.saps_destroy(ctx)
    m = oracle.mask(seed, t, p, N)
    wv, wi, wc = oracle.pack(x, m, cap)
    got_count = int(count.cpu().numpy().view(np.uint32)[0])
    assert got_count == wc, (N, p)
    assert int(count[1]) == -1
    k = min(wc, cap)
    gv = vals.cpu().numpy()
    gi = idx.cpu().numpy().view(np.uint32)
    if with_idx:
        assert (gi[:k] == wi[:k]).all()
        assert (gi[k:] == 0xFFFFFFFF).all()              # slots past count untouched
    else:
        assert (gi == 0xFFFFFFFF).all()
    got_vals = gv[:n * cap].reshape(n, cap)
    assert_bits_equal(got_vals[:, :k], wv[:, :k], f"packed values N={N} p={p}")
    assert (got_vals[:, k:] == 123.0).all() and (gv[n * cap:] == 123.0).all()
    assert dx.canaries_intact()
    return status, wc, cap


@pytest.mark.parametrize("N", [1, 5, 33, 2047, 2048, 2049, 3 * 2048 + 1, 70_001])
@pytest.mark.parametrize("p", [0.0, 0.01, 0.1, 0.5, 1.0])
def test_pack_small(sb, N, p):
    for n, ld in ((1, N), (4, N), (5, round_up(N, 32))):
        status, _, _ = _pack_both(sb, n, N, ld, p, seed=N % 7, t=2)
        assert status == 0


def test_pack_many_tiles_and_no_index_list(sb):
    # hundreds of tiles: the look-back crosses several 32-tile windows
    for p in (0.001, 0.01, 0.1):
        status, count, cap = _pack_both(sb, 8, 1_500_007, round_up(1_500_007, 32), p, seed=4, t=7)
        assert status == 0 and count <= cap
    status, _, _ = _pack_both(sb, 3, 300_000, 300_000, 0.05, seed=4, t=8, with_idx=False)
    assert status == 0


def test_pack_resnet20_shape(sb):
    w = synth.WORKLOADS["resnet20"]
    status, count, _ = _pack_both(sb, w.n, w.N, round_up(w.N, 32), 0.01, seed=1, t=1)
    assert status == 0 and count == 2655                # golden count for seed 1, t 1


def test_pack_overflow_is_reported_not_written(sb):
    status, count, cap = _pack_both(sb, 4, 100_000, 100_000, 0.1, seed=2, t=1, cap_override=5000)
    assert cap == 5000 and count > cap
    assert status == sb.SAPS_ERR_OVERFLOW
    # the status word is cleared by reading it: a clean call afterwards reports ok
    status, _, _ = _pack_both(sb, 4, 100_000, 100_000, 0.1, seed=2, t=1)
    assert status == 0


def test_repeated_packs_reuse_the_scratch(sb):
    torch = torch_cuda()
    n, N, p = 4, 500_000, 0.02
    x = synth.gaussian_matrix(n, N, 1.0, 8, 0)
    dx = DeviceMatrix(x, N)
    ctx = sb.saps_create(n, N, 8)
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.zeros(n * cap, dtype=torch.float32, device="cuda")
    idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
    count = torch.zeros(1, dtype=torch.int32, device="cuda")
    for t in range(1, 8):
        sb.saps_pack(ctx, dx.ptr, t, p, vals, idx, count)      # back to back, no sync
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == 0
    sb.saps_destroy(ctx)
    m = oracle.mask(8, 7, p, N)
    wv, wi, wc = oracle.pack(x, m, cap)
    assert int(count[0]) == wc
    assert (idx.cpu().numpy().view(np.uint32)[:wc] == wi[:wc]).all()
    assert_bits_equal(vals.cpu().numpy().reshape(n, cap)[:, :wc], wv[:, :wc], "7th pack")


@pytest.mark.parametrize("N,ld", [(7, 7), (2050, 2050), (2050, 2052), (40_003, 40_032), (40_003, 40_003),
                                  (6 * 2048, 6 * 2048)])
@pytest.mark.parametrize("p", [0.0, 0.05, 0.5, 1.0])
@pytest.mark.parametrize("has_g", [True, False])
def test_round_pack_emits_what_each_worker_sends(sb, N, ld, p, has_g):
    torch = torch_cuda()
    n = 6
    pairs = [1, 0, 2, 5, 4, 3]                 # workers 2 and 4 have no peer
    x = synth.gaussian_matrix(n, N, 1.0, 17, 0)
    g = synth.gaussian_matrix(n, N, 0.01, 17, 1) if has_g else None
    lr = 0.1 if has_g else 0.0
    dx = DeviceMatrix(x, ld)
    dg = DeviceMatrix(g, ld) if has_g else None
    ctx = sb.saps_create_ld(n, N, ld, 17)
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.full((n * cap,), 123.0, dtype=torch.float32, device="cuda")
    idx = torch.full((cap,), -1, dtype=torch.int32, device="cuda")
    count = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    sb.saps_round_pack(ctx, dx.ptr, dg.ptr if has_g else None, lr, pairs, 5, p, vals, idx, count)
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == 0
    sb.saps_destroy(ctx)
    a = x.copy()
    oracle.sgd(a, g, lr)
    m = oracle.mask(17, 5, p, N)
    wv, wi, wc = oracle.pack(a, m, cap)
    want = x.copy()
    oracle.gossip_round(want, g, lr, pairs, 17, 5, p)
    assert int(count.cpu().numpy().view(np.uint32)[0]) == wc
    assert (idx.cpu().numpy().view(np.uint32)[:wc] == wi[:wc]).all()
    got_vals = vals.cpu().numpy().reshape(n, cap)
    assert_bits_equal(got_vals[:, :wc], wv[:, :wc], "emitted wire buffer")
    assert (got_vals[:, wc:] == 123.0).all()
    assert_bits_equal(dx.host(), want, "round result with emission")
    assert dx.canaries_intact()


@pytest.mark.parametrize("N,ld", [(7, 7), (2050, 2052), (40_003, 40_032), (40_003, 40_003), (6 * 2048, 6 * 2048)])
@pytest.mark.parametrize("p", [0.05, 1.0])
def test_round_pack_rows_writes_each_worker_to_its_own_destination(sb, N, ld, p):
    # Per-worker destinations (the form that lets a pass store its wire buffers straight into the
    # receivers' memory): every worker's packed values must land, bit for bit, at the address its
    # table entry names and nowhere else; a worker with a NULL entry emits nothing; the model,
    # the index list and the count are those of the ordinary emitting round.
    torch = torch_cuda()
    n = 6
    pairs = [1, 0, 2, 5, 4, 3]                 # workers 2 and 4 have no peer
    x = synth.gaussian_matrix(n, N, 1.0, 19, 0)
    g = synth.gaussian_matrix(n, N, 0.01, 19, 1)
    dx, dg = DeviceMatrix(x, ld), DeviceMatrix(g, ld)
    ctx = sb.saps_create_ld(n, N, ld, 19)
    cap = sb.saps_pack_capacity(ctx, p)
    # one arena, rows handed out in a scrambled order with a guard stretch behind each
    slot = cap + 16
    arena = torch.full((n * slot,), 123.0, dtype=torch.float32, device="cuda")
    order = [3, 0, 5, 1, 4, 2]
    skipped = 4
    table = [0 if i == skipped else arena.data_ptr() + 4 * slot * order[i] for i in range(n)]
    d_table = torch.tensor(table, dtype=torch.int64, device="cuda")
    idx = torch.full((cap,), -1, dtype=torch.int32, device="cuda")
    count = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    for t in (5, 6):                            # the second round takes its counts from the first one's kernel
        a = dx.host().copy()
        want = a.copy()
        oracle.sgd(a, g, 0.1)
        arena.fill_(123.0)
        sb.saps_round_pack_rows(ctx, dx.ptr, dg.ptr, 0.1, pairs, t, p, d_table, idx, count)
        torch.cuda.synchronize()
        assert sb.saps_status(ctx) == 0
        m = oracle.gossip_round(want, g, 0.1, pairs, 19, t, p)
        wv, wi, wc = oracle.pack(a, m, cap)
        assert int(count.cpu().numpy().view(np.uint32)[0]) == wc
        assert (idx.cpu().numpy().view(np.uint32)[:wc] == wi[:wc]).all()
        got = arena.cpu().numpy().reshape(n, slot)
        for i in range(n):
            row = got[order[i]]
            if i == skipped:
                assert (row == 123.0).all()
            else:
                assert_bits_equal(row[:wc], wv[i, :wc], f"worker {i}, round {t}")
                assert (row[wc:] == 123.0).all()
        assert_bits_equal(dx.host(), want, "round result with per-worker destinations")
    assert dx.canaries_intact() and dg.canaries_intact()
    assert sb._lib.saps_round_pack_rows(ctx, dx.ptr, dg.ptr, 0.1, sb._pairs(pairs), 7, p, None, sb._ptr(idx),
                                        sb._ptr(count), None) == sb.SAPS_ERR_INVALID
    sb.saps_destroy(ctx)


def test_unfused_wire_path_equals_fused_round(sb):
    # SGD-only round -> pack -> average the two packed buffers -> scatter  ==  fused round
    torch = torch_cuda()
    n, N, p, lr = 4, 50_000, 0.1, 0.05
    pairs = [3, 2, 1, 0]
    x = synth.gaussian_matrix(n, N, 1.0, 61, 0)
    g = synth.gaussian_matrix(n, N, 0.01, 61, 1)
    ctx = sb.saps_create(n, N, 61)
    fused, dg = DeviceMatrix(x, N), DeviceMatrix(g, N)
    sb.saps_round(ctx, fused.ptr, dg.ptr, lr, pairs, 2, p)
    unf = DeviceMatrix(x, N)
    sb.saps_round(ctx, unf.ptr, dg.ptr, lr, list(range(n)), 2, p)        # SGD step only
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.zeros(n, cap, dtype=torch.float32, device="cuda")
    idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
    count = torch.zeros(1, dtype=torch.int32, device="cuda")
    sb.saps_pack(ctx, unf.ptr, 2, p, vals, idx, count)
    torch.cuda.synchronize()
    c = int(count[0])
    cols = idx[:c].long()
    peer = torch.tensor(pairs, device="cuda")
    merged = 0.5 * (vals[:, :c] + vals[peer, :c])
    unf.view[:, :N].index_copy_(1, cols, merged)
    assert_bits_equal(unf.host(), fused.host(), "wire path")
    # after the round a worker and its peer hold identical kept coordinates
    sb.saps_pack(ctx, fused.ptr, 2, p, vals, idx, count)
    torch.cuda.synchronize()
    v = vals.cpu().numpy()[:, :c]
    for i in range(n):
        assert_bits_equal(v[i], v[pairs[i]], "peers send identical buffers")
    sb.saps_destroy(ctx)


@pytest.mark.parametrize("prefetch", [True, False])
def test_round_pack_sequence_with_scan_run_ahead(sb, prefetch):
    # consecutive rounds find their mask scan already done by the previous call; jumps in t,
    # a changed keep_frac and a changed capacity fall back to an in-line scan; same results
    torch = torch_cuda()
    n, N = 4, 9 * 2048 + 77
    ld = round_up(N, 32)
    pairs = [1, 0, 3, 2]
    x = synth.gaussian_matrix(n, N, 1.0, 91, 0)
    g = synth.gaussian_matrix(n, N, 0.01, 91, 1)
    dx, dg = DeviceMatrix(x, ld), DeviceMatrix(g, ld)
    ctx = sb.saps_create_ld(n, N, ld, 91)
    sb.saps_set_run_ahead(ctx, prefetch)
    want = x.copy()
    schedule = [(1, 0.1), (2, 0.1), (3, 0.1), (10, 0.1), (11, 0.3), (12, 0.3), (12, 0.3), (13, 0.05)]
    for step, (t, p) in enumerate(schedule):
        if step == 5:
            sb.saps_set_pack_capacity(ctx, 7000)
        cap = sb.saps_pack_capacity(ctx, p)
        vals = torch.full((n, cap), 123.0, dtype=torch.float32, device="cuda")
        idx = torch.full((cap,), -1, dtype=torch.int32, device="cuda")
        count = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        sb.saps_round_pack(ctx, dx.ptr, dg.ptr, 0.05, pairs, t, p, vals, idx, count)
        a = want.copy()
        oracle.sgd(a, g, 0.05)
        m = oracle.mask(91, t, p, N)
        wv, wi, wc = oracle.pack(a, m, cap)
        oracle.pair_average(a, pairs, m)
        want = a
        torch.cuda.synchronize()
        assert int(count[0]) == wc, (step, t, p)
        assert (idx.cpu().numpy().view(np.uint32)[:wc] == wi[:wc]).all(), (step, t, p)
        assert_bits_equal(vals.cpu().numpy()[:, :wc], wv[:, :wc], f"wire buffer step {step}")
        assert_bits_equal(dx.host(), want, f"model step {step}")
    assert sb.saps_status(ctx) == 0
    sb.saps_destroy(ctx)


def test_threshold_comparison_is_strict_on_the_gpu(sb):
    # a column whose hash equals the threshold is dropped; one more and it is kept
    torch = torch_cuda()
    seed, t, N = 12, 34, 100_001
    k0, k1 = oracle.round_key(seed, t)
    ctx = sb.saps_create(2, N, seed)
    bits = torch.zeros(round_up(N, 32) // 32, dtype=torch.int32, device="cuda")
    for k in (0, 1, 77, 4095, 100_000):
        h = oracle.hash_k(k, k0, k1)
        for thr, want in ((h, 0), (h + 1, 1)):
            sb.saps_mask(ctx, t, thr / 2.0 ** 32, bits)
            word = int(bits[k >> 5].cpu().numpy().view(np.uint32))
            assert (word >> (k & 31)) & 1 == want
    sb.saps_destroy(ctx)


@pytest.mark.parametrize("N,ld", [(70_003, 70_016), (70_003, 70_003), (70_002, 70_002)])   # 128-, 32-, 64-bit access
@pytest.mark.parametrize("scheduler", [False, True, "rows"])
def test_fused_emission_overflow_is_clamped_and_reported(sb, N, ld, scheduler):
    # The count is Binomial(N, p), so a hard wire-buffer size can be exceeded (Eq. 2 / Section II-B).
    # With a capacity below the true count the emitting round must: keep the model exactly
    # right, report the true count, write the first `cap` entries only, leave everything behind
    # them alone, and raise SAPS_ERR_OVERFLOW in the status word.
    torch = torch_cuda()
    n, p, lr, seed, cap = 6, 0.1, 0.05, 23, 4000
    pairs_list = np.array([[1, 0, 2, 5, 4, 3], [5, 4, 3, 2, 1, 0], [0, 2, 1, 4, 3, 5]], dtype=np.int32)
    x = synth.gaussian_matrix(n, N, 1.0, seed, 0)
    g = synth.gaussian_matrix(n, N, 0.01, seed, 1)
    dx, dg = DeviceMatrix(x, ld), DeviceMatrix(g, ld)
    ctx = sb.saps_create_ld(n, N, ld, seed)
    sb.saps_set_pack_capacity(ctx, cap)
    assert sb.saps_pack_capacity(ctx, p) == cap
    guard = 64
    vals = torch.full((n * cap + guard,), 123.0, dtype=torch.float32, device="cuda")
    idx = torch.full((cap + guard,), -1, dtype=torch.int32, device="cuda")
    T = len(pairs_list)
    counts = torch.full((T + 1,), -1, dtype=torch.int32, device="cuda")
    if scheduler == "rows":                              # one destination per worker, same clamp
        table = torch.tensor([vals.data_ptr() + 4 * cap * i for i in range(n)], dtype=torch.int64, device="cuda")
        for r in range(T):
            sb.saps_round_pack_rows(ctx, dx.ptr, dg.ptr, lr, pairs_list[r], 1 + r, p, table, idx, counts[r:])
    elif scheduler:
        sb.saps_run_rounds_pack(ctx, dx.ptr, dg.ptr, lr, 1, T, p, vals, idx, counts, pairs_list=pairs_list)
    else:
        for r in range(T):
            sb.saps_round_pack(ctx, dx.ptr, dg.ptr, lr, pairs_list[r], 1 + r, p, vals, idx, counts[r:])
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == sb.SAPS_ERR_OVERFLOW
    assert sb.saps_status(ctx) == 0                       # reading the status clears it
    want = x.copy()
    for r in range(T):
        a = want.copy()
        oracle.sgd(a, g, lr)
        m = oracle.mask(seed, 1 + r, p, N)
        wv, wi, wc = oracle.pack(a, m, cap)               # the oracle clamps the same way
        oracle.pair_average(a, pairs_list[r], m)
        want = a
        assert wc > cap
        assert int(counts[r]) == wc, f"round {r}: the true count is reported"
    assert int(counts[T]) == -1
    assert_bits_equal(dx.host(), want, "model after overflowing rounds")
    gv, gi = vals.cpu().numpy(), idx.cpu().numpy().view(np.uint32)
    assert (gi[:cap] == wi[:cap]).all() and (gi[cap:] == 0xFFFFFFFF).all()
    assert_bits_equal(gv[:n * cap].reshape(n, cap), wv, "first cap entries of the last round's wire buffer")
    assert (gv[n * cap:] == 123.0).all()
    assert dx.canaries_intact() and dg.canaries_intact()
    # with the formula capacity back, the same context emits a complete buffer again
    sb.saps_set_pack_capacity(ctx, 0)
    full = sb.saps_pack_capacity(ctx, p)
    vals2 = torch.zeros(n, full, dtype=torch.float32, device="cuda")
    idx2 = torch.zeros(full, dtype=torch.int32, device="cuda")
    sb.saps_round_pack(ctx, dx.ptr, dg.ptr, lr, pairs_list[0], T + 1, p, vals2, idx2, counts)
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == 0
    a = want.copy()
    oracle.sgd(a, g, lr)
    m = oracle.mask(seed, T + 1, p, N)
    wv, wi, wc = oracle.pack(a, m, full)
    assert int(counts[0]) == wc <= full
    assert (idx2.cpu().numpy().view(np.uint32)[:wc] == wi[:wc]).all()
    assert_bits_equal(vals2.cpu().numpy()[:, :wc], wv[:, :wc], "wire buffer after the capacity was restored")
    sb.saps_destroy(ctx)
