"""GPU parity: the CUDA round (through the C ABI) against the CPU oracle, bit for bit."""
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


def _pairs_with_singles(n, rng, singles=0):
    perm = list(rng.permutation(n))
    pairs = list(range(n))
    free = perm[singles:]
    for a in range(0, len(free) - 1, 2):
        i, j = int(free[a]), int(free[a + 1])
        pairs[i], pairs[j] = j, i
    return pairs


def _run_both(sb, n, N, ld, lead, has_g, lr, p, pairs, seed, t, x_std=1.0):
    torch = torch_cuda()
    x = synth.gaussian_matrix(n, N, x_std, seed + 11, 0)
    g = synth.gaussian_matrix(n, N, 0.01, seed + 11, 1) if has_g else None
    dx = DeviceMatrix(x, ld, lead)
    dg = DeviceMatrix(g, ld, lead) if has_g else None
    ctx = sb.saps_create_ld(n, N, ld, seed)
    sb.saps_round(ctx, dx.ptr, dg.ptr if has_g else None, lr, pairs, t, p)
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == 0
    sb.saps_destroy(ctx)
    want = x.copy()
    oracle.gossip_round(want, g, lr, pairs, seed, t, p)
    assert_bits_equal(dx.host(), want, f"n={n} N={N} ld={ld} lead={lead} g={has_g} p={p}")
    assert dx.canaries_intact()
    if has_g:
        assert_bits_equal(dg.host(), g, "gradient must not change")
        assert dg.canaries_intact()


@pytest.mark.parametrize("N", list(range(1, 13)) + [31, 32, 33, 63, 64, 65, 66, 67, 2047, 2048, 2049, 2050,
                                                     4095, 4097, 6151])
def test_small_sizes_every_tail(sb, N):
    rng = np.random.default_rng(N)
    for n, singles in ((2, 0), (4, 0), (5, 1), (6, 2)):
        pairs = _pairs_with_singles(n, rng, singles)
        for ld, lead in ((N, 0), (round_up(N, 4), 0), (round_up(N, 32), 0), (N + 1, 1), (round_up(N, 4), 2)):
            _run_both(sb, n, N, ld, lead, True, 0.1, 0.3, pairs, seed=N, t=3)
    _run_both(sb, 4, N, round_up(N, 4), 0, False, 0.0, 0.5, [1, 0, 3, 2], seed=1, t=1)


@pytest.mark.parametrize("p", [0.0, 0.001, 0.01, 0.1, 0.5, 1.0])
@pytest.mark.parametrize("has_g", [True, False])
def test_keep_frac_sweep_several_tiles(sb, p, has_g):
    n, N = 8, 5 * 2048 + 777
    pairs = synth.random_perfect_matching(n, synth.matching_rng(3))
    for ld in (N, round_up(N, 32)):
        _run_both(sb, n, N, ld, 0, has_g, 0.05 if has_g else 0.0, p, pairs, seed=2, t=9)


def test_lr_zero_with_gradient_and_huge_t(sb):
    _run_both(sb, 4, 9000, 9024, 0, True, 0.0, 0.2, [1, 0, 3, 2], seed=0xDEADBEEFCAFEF00D, t=2 ** 32 + 5)


def test_subnormals_and_signed_zeros_survive(sb):
    # no flush-to-zero on either side: tiny values and -0.0 must come back with the same bits
    torch = torch_cuda()
    n, N = 4, 4096
    x = synth.gaussian_matrix(n, N, 1.0, 5, 0)
    x[:, ::3] *= np.float32(1e-41)          # subnormal inputs
    x[:, 1::7] = np.float32(-0.0)
    g = synth.gaussian_matrix(n, N, 1e-38, 5, 1)
    dx, dg = DeviceMatrix(x, N), DeviceMatrix(g, N)
    ctx = sb.saps_create(n, N, 5)
    sb.saps_round(ctx, dx.ptr, dg.ptr, 0.5, [1, 0, 3, 2], 1, 0.5)
    torch.cuda.synchronize()
    sb.saps_destroy(ctx)
    want = x.copy()
    oracle.gossip_round(want, g, 0.5, [1, 0, 3, 2], 5, 1, 0.5)
    assert_bits_equal(dx.host(), want, "subnormals")


def test_tiny_workload_three_rounds(sb):
    # n=4, N=65,536, x ~ N(0,1), g ~ N(0,0.01), lr 0.1, keep 0.1, pairs (0,1),(2,3), seed 0
    torch = torch_cuda()
    w = synth.WORKLOADS["tiny"]
    x, g = synth.model_and_grad(w)
    dx, dg = DeviceMatrix(x, w.N), DeviceMatrix(g, w.N)
    ctx = sb.saps_create(w.n, w.N, w.seed)
    want = x.copy()
    for t in range(1, w.rounds + 1):
        sb.saps_round(ctx, dx.ptr, dg.ptr, w.lr, w.fixed_pairs, t, w.keep_fracs[0])
        oracle.gossip_round(want, g, w.lr, w.fixed_pairs, w.seed, t, w.keep_fracs[0])
        torch.cuda.synchronize()
        assert_bits_equal(dx.host(), want, f"round {t}")
    sb.saps_destroy(ctx)


def test_max_workers_and_all_singles(sb):
    n, N = 64, 3000
    rng = np.random.default_rng(64)
    _run_both(sb, n, N, round_up(N, 4), 0, True, 0.1, 0.2, _pairs_with_singles(n, rng, 0), seed=1, t=1)
    _run_both(sb, n, N, round_up(N, 4), 0, True, 0.1, 0.2, list(range(n)), seed=1, t=1)
    _run_both(sb, n, N, round_up(N, 4), 0, False, 0.0, 0.2, list(range(n)), seed=1, t=1)
    _run_both(sb, 1, N, N, 0, True, 0.1, 0.2, [0], seed=1, t=1)


def test_properties_on_the_gpu_result(sb):
    # the invariants the paper fixes, checked on the CUDA result itself
    torch = torch_cuda()
    n, N, p, lr = 8, 40_000, 0.25, 0.05
    x = synth.gaussian_matrix(n, N, 1.0, 21, 0)
    g = synth.gaussian_matrix(n, N, 0.01, 21, 1)
    pairs = synth.random_perfect_matching(n, synth.matching_rng(21))
    ld = round_up(N, 32)
    dx, dg = DeviceMatrix(x, ld), DeviceMatrix(g, ld)
    ctx = sb.saps_create_ld(n, N, ld, 21)
    bits = torch.zeros(round_up(N, 32) // 32, dtype=torch.int32, device="cuda")
    sb.saps_mask(ctx, 4, p, bits)
    sb.saps_round(ctx, dx.ptr, dg.ptr, lr, pairs, 4, p)
    torch.cuda.synchronize()
    sb.saps_destroy(ctx)
    out = dx.host()
    m = np.unpackbits(bits.cpu().numpy().view(np.uint8), bitorder="little")[:N].astype(bool)
    a = x - np.float32(lr) * g
    assert_bits_equal(out[:, ~m], a[:, ~m], "unmasked = SGD step only")
    phat = oracle.threshold(p) / 2.0 ** 32
    assert abs(m.sum() - N * phat) < 5 * np.sqrt(N * phat * (1 - phat))
    for i in range(n):
        j = int(pairs[i])
        assert_bits_equal(out[i, m], out[j, m], "peers agree")
        assert (out[i, m] + out[j, m] == a[i, m] + a[j, m]).all()


def test_hypercube_consensus_on_gpu(sb):
    torch = torch_cuda()
    n, N = 32, 10_000
    x = synth.gaussian_matrix(n, N, 1.0, 9, 0)
    dx = DeviceMatrix(x, round_up(N, 32))
    ctx = sb.saps_create_ld(n, N, round_up(N, 32), 9)
    for r in range(5):
        sb.saps_round(ctx, dx.ptr, None, 0.0, synth.hypercube_pairs(n, r), r + 1, 1.0)
    torch.cuda.synchronize()
    sb.saps_destroy(ctx)
    out = dx.host()
    assert (out.view(np.uint32) == out[0].view(np.uint32)[None, :]).all()
    assert np.abs(out[0] - x.astype(np.float64).mean(axis=0)).max() < 5 * 2.0 ** -24 * 8


def test_column_shards_reproduce_the_whole(sb):
    # two contexts with column offsets compute the same round as one context over all columns
    torch = torch_cuda()
    n, N, p = 4, 3 * 2048 + 100, 0.2
    cut = 2 * 2048
    x = synth.gaussian_matrix(n, N, 1.0, 31, 0)
    g = synth.gaussian_matrix(n, N, 0.01, 31, 1)
    pairs = [2, 3, 0, 1]
    want = x.copy()
    oracle.gossip_round(want, g, 0.1, pairs, 31, 6, p)
    parts = []
    for lo, hi in ((0, cut), (cut, N)):
        xs, gs = np.ascontiguousarray(x[:, lo:hi]), np.ascontiguousarray(g[:, lo:hi])
        dx, dg = DeviceMatrix(xs, round_up(hi - lo, 4)), DeviceMatrix(gs, round_up(hi - lo, 4))
        ctx = sb.saps_create_ld(n, hi - lo, round_up(hi - lo, 4), 31)
        sb.saps_set_column_offset(ctx, lo)
        sb.saps_round(ctx, dx.ptr, dg.ptr, 0.1, pairs, 6, p)
        torch.cuda.synchronize()
        sb.saps_destroy(ctx)
        parts.append(dx.host())
    assert_bits_equal(np.concatenate(parts, axis=1), want, "column shards")


def test_run_rounds_with_given_matchings(sb):
    torch = torch_cuda()
    n, N, T, p = 8, 30_000, 12, 0.1
    x = synth.gaussian_matrix(n, N, 0.05, 41, 0)
    g = synth.gaussian_matrix(n, N, 0.01, 41, 1)
    rng = synth.matching_rng(41)
    plist = np.stack([synth.random_perfect_matching(n, rng) for _ in range(T)]).astype(np.int32)
    ld = round_up(N, 32)
    dx, dg = DeviceMatrix(x, ld), DeviceMatrix(g, ld)
    ctx = sb.saps_create_ld(n, N, ld, 41)
    log = np.zeros((T, n), dtype=np.int32)
    sb.saps_run_rounds(ctx, dx.ptr, dg.ptr, 0.05, 1, T, p, pairs_list=plist, out_pairs_log=log)
    torch.cuda.synchronize()
    sb.saps_destroy(ctx)
    assert (log == plist).all()
    want = x.copy()
    for t in range(1, T + 1):
        oracle.gossip_round(want, g, 0.05, plist[t - 1], 41, t, p)
    assert_bits_equal(dx.host(), want, "scheduler, given matchings")


def test_run_rounds_with_adaptive_peer_selection(sb):
    # the ResNet-20-sized configuration: n=32, N=272,474, keep 0.01, U[1,100] Mb/s, 100 rounds
    torch = torch_cuda()
    w = synth.WORKLOADS["resnet20"]
    T = w.rounds
    x, g = synth.model_and_grad(w)
    B = synth.bandwidth_matrix(w.n, *w.bw_range, seed=w.seed)
    ld = round_up(w.N, 32)
    dx, dg = DeviceMatrix(x, ld), DeviceMatrix(g, ld)
    ctx = sb.saps_create_ld(w.n, w.N, ld, w.seed)
    log = np.zeros((T, w.n), dtype=np.int32)
    sb.saps_run_rounds(ctx, dx.ptr, dg.ptr, w.lr, 1, T, w.keep_fracs[0], bandwidth=B, out_pairs_log=log)
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == 0
    # the scheduler used the same matchings a fresh selection sequence gives
    ctx2 = sb.saps_create(w.n, w.N, w.seed)
    for t in range(1, T + 1):
        assert sb.saps_select_peers(ctx2, B, t, w.n) == list(log[t - 1])
    sb.saps_destroy(ctx2)
    sb.saps_destroy(ctx)
    want = x.copy()
    for t in range(1, T + 1):
        oracle.gossip_round(want, g, w.lr, log[t - 1], w.seed, t, w.keep_fracs[0])
    assert_bits_equal(dx.host(), want, "scheduler, adaptive selection")
    assert dx.canaries_intact()


def test_round_host_entry_point(sb):
    torch = torch_cuda()
    n, N, p = 6, 2_300_000, 0.01           # three pipeline chunks with a ragged last one
    x = synth.gaussian_matrix(n, N, 0.05, 51, 0)
    g = synth.gaussian_matrix(n, N, 0.01, 51, 1)
    pairs = [1, 0, 3, 2, 5, 4]
    want = x.copy()
    oracle.gossip_round(want, g, 0.05, pairs, 51, 2, p)
    hx = torch.from_numpy(x.copy()).pin_memory()
    hg = torch.from_numpy(g).pin_memory()
    ld = round_up(N, 32)
    d_x = torch.empty(n * ld, dtype=torch.float32, device="cuda")
    d_g = torch.empty(n * ld, dtype=torch.float32, device="cuda")
    ctx = sb.saps_create_ld(n, N, ld, 51)
    sb.saps_round_host(ctx, hx, hg, 0.05, pairs, 2, p, d_x, d_g)
    assert_bits_equal(hx.numpy(), want, "host entry point")
    # without a gradient, with many small chunks over all six lanes
    hx2 = torch.from_numpy(x.copy()).pin_memory()
    sb.saps_set_host_pipeline(ctx, 100_000, 6)
    sb.saps_round_host(ctx, hx2, None, 0.0, pairs, 3, p, d_x, None)
    want2 = x.copy()
    oracle.gossip_round(want2, None, 0.0, pairs, 51, 3, p)
    assert_bits_equal(hx2.numpy(), want2, "host entry point, no gradient")
    sb.saps_destroy(ctx)


def test_round_pack_host_entry_point(sb):
    torch = torch_cuda()
    n, N, p = 6, 2_300_000, 0.01
    x = synth.gaussian_matrix(n, N, 0.05, 52, 0)
    g = synth.gaussian_matrix(n, N, 0.01, 52, 1)
    pairs = [1, 0, 3, 2, 5, 4]
    ld = round_up(N, 32)
    ctx = sb.saps_create_ld(n, N, ld, 52)
    cap = sb.saps_pack_capacity(ctx, p)
    hx = torch.from_numpy(x.copy()).pin_memory()
    hg = torch.from_numpy(g).pin_memory()
    hv = torch.full((n, cap), 123.0, dtype=torch.float32).pin_memory()
    hi = torch.full((cap,), -1, dtype=torch.int32).pin_memory()
    hc = torch.full((1,), -1, dtype=torch.int32).pin_memory()
    d_x = torch.empty(n * ld, dtype=torch.float32, device="cuda")
    d_g = torch.empty(n * ld, dtype=torch.float32, device="cuda")
    d_v = torch.empty(n * cap, dtype=torch.float32, device="cuda")
    d_i = torch.empty(cap, dtype=torch.int32, device="cuda")
    d_c = torch.empty(1, dtype=torch.int32, device="cuda")
    sb.saps_round_pack_host(ctx, hx, hg, 0.05, pairs, 4, p, d_x, d_g, hv, hi, hc, d_v, d_i, d_c)
    assert sb.saps_status(ctx) == 0
    sb.saps_destroy(ctx)
    a = x.copy()
    oracle.sgd(a, g, 0.05)
    m = oracle.mask(52, 4, p, N)
    wv, wi, wc = oracle.pack(a, m, cap)
    want = x.copy()
    oracle.gossip_round(want, g, 0.05, pairs, 52, 4, p)
    assert int(hc[0]) == wc
    assert (hi.numpy().view(np.uint32)[:wc] == wi[:wc]).all()
    assert_bits_equal(hv.numpy()[:, :wc], wv[:, :wc], "host wire buffer")
    assert_bits_equal(hx.numpy(), want, "host entry point with wire buffer")
    # model resident on the device (x_host = NULL): only g goes in, the wire buffer comes out;
    # one lane, and a row stride that only allows 64-bit accesses
    ld = N + 2
    d_x = torch.empty(n * ld, dtype=torch.float32, device="cuda")
    d_g = torch.empty(n * ld, dtype=torch.float32, device="cuda")
    ctx = sb.saps_create_ld(n, N, ld, 52)
    sb.saps_set_host_pipeline(ctx, 4096, 1)
    d_x.view(n, ld)[:, :N].copy_(torch.from_numpy(x))
    sb.saps_round_pack_host(ctx, None, hg, 0.05, pairs, 4, p, d_x, d_g, hv, hi, hc, d_v, d_i, d_c)
    assert int(hc[0]) == wc
    assert_bits_equal(hv.numpy()[:, :wc], wv[:, :wc], "host wire buffer, resident model")
    assert_bits_equal(d_x.view(n, ld)[:, :N].cpu().numpy(), want, "resident model after the round")
    sb.saps_destroy(ctx)


def test_run_rounds_pack_emits_every_round(sb):
    # the scheduler with the wire buffer: counts of all rounds, buffers of the last one
    torch = torch_cuda()
    w = synth.WORKLOADS["resnet20"]
    T, p = 12, w.keep_fracs[0]
    x, g = synth.model_and_grad(w)
    B = synth.bandwidth_matrix(w.n, *w.bw_range, seed=w.seed)
    ld = round_up(w.N, 32)
    dx, dg = DeviceMatrix(x, ld), DeviceMatrix(g, ld)
    ctx = sb.saps_create_ld(w.n, w.N, ld, w.seed)
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.full((w.n, cap), 123.0, dtype=torch.float32, device="cuda")
    idx = torch.full((cap,), -1, dtype=torch.int32, device="cuda")
    counts = torch.full((T + 1,), -1, dtype=torch.int32, device="cuda")
    log = np.zeros((T, w.n), dtype=np.int32)
    sb.saps_run_rounds_pack(ctx, dx.ptr, dg.ptr, w.lr, 1, T, p, vals, idx, counts, bandwidth=B, out_pairs_log=log)
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == 0
    want = x.copy()
    for t in range(1, T + 1):
        oracle.sgd(want, g, w.lr)
        m = oracle.mask(w.seed, t, p, w.N)
        assert int(counts[t - 1]) == int(m.sum())
        if t == T:
            wv, wi, wc = oracle.pack(want, m, cap)
        oracle.pair_average(want, log[t - 1], m)
    assert int(counts[T]) == -1
    assert (idx.cpu().numpy().view(np.uint32)[:wc] == wi[:wc]).all()
    assert_bits_equal(vals.cpu().numpy()[:, :wc], wv[:, :wc], "last round's wire buffer")
    assert_bits_equal(dx.host(), want, "scheduler with emission")
    # Table 1: total traffic of a worker over T rounds is 2 sum_t count_t, about 2 T N / c
    total = int(counts[:T].sum())
    phat = oracle.threshold(p) / 2.0 ** 32
    assert abs(total - T * w.N * phat) < 5 * np.sqrt(T * w.N * phat * (1 - phat))
    # a given list of matchings works too, and invalid arguments are refused
    sb.saps_run_rounds_pack(ctx, dx.ptr, dg.ptr, w.lr, T + 1, 2, p, vals, idx, counts, pairs_list=log[:2].copy())
    torch.cuda.synchronize()
    rc = sb._lib.saps_run_rounds_pack(ctx, dx.ptr, dg.ptr, w.lr, 1, 2, p, None, None, None, None, None, None, None,
                                      None, None)
    assert rc == sb.SAPS_ERR_INVALID
    sb.saps_destroy(ctx)


@pytest.mark.parametrize("n,N,ld,emit", [(4, 5_000, 5_000, True), (6, 2_050, 2_052, True), (4, 700, 700, False),
                                         (8, 9_001, 9_001, True)])
def test_many_small_rounds_back_to_back(sb, n, N, ld, emit):
    # Launches of a handful of blocks, 150 of them in one scheduler call: consecutive round
    # kernels are launched as programmatic dependents, so with grids this small several of them
    # are resident at once, each waiting for its predecessor before it touches memory, and the
    # per-tile mask counts pass from each kernel to the next.  Every round's count and the final
    # model and wire buffer must equal the oracle's.
    torch = torch_cuda()
    T, p, lr, seed = 150, 0.08, 0.05, 77
    x = synth.gaussian_matrix(n, N, 1.0, seed, 0)
    g = synth.gaussian_matrix(n, N, 0.01, seed, 1)
    rng = synth.matching_rng(seed)
    pairs_list = np.asarray([synth.random_perfect_matching(n, rng) for _ in range(T)], dtype=np.int32)
    dx, dg = DeviceMatrix(x, ld), DeviceMatrix(g, ld)
    ctx = sb.saps_create_ld(n, N, ld, seed)
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.zeros(n, cap, dtype=torch.float32, device="cuda")
    idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
    counts = torch.zeros(T, dtype=torch.int32, device="cuda")
    if emit:
        sb.saps_run_rounds_pack(ctx, dx.ptr, dg.ptr, lr, 1, T, p, vals, idx, counts, pairs_list=pairs_list)
    else:
        sb.saps_run_rounds(ctx, dx.ptr, dg.ptr, lr, 1, T, p, pairs_list=pairs_list)
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == 0
    want = x.copy()
    got_counts = counts.cpu().numpy().view(np.uint32)
    for t in range(1, T + 1):
        a = want.copy()
        oracle.sgd(a, g, lr)
        m = oracle.gossip_round(want, g, lr, pairs_list[t - 1], seed, t, p)
        if emit:
            assert int(got_counts[t - 1]) == int(m.sum()), t
    assert_bits_equal(dx.host(), want, "150 small rounds in one call")
    if emit:
        kept = np.nonzero(m)[0]
        assert (idx[:len(kept)].cpu().numpy().view(np.uint32) == kept.astype(np.uint32)).all()
        assert_bits_equal(vals[:, :len(kept)].cpu().numpy(), a[:, kept], "wire buffer of the last round")
    assert dx.canaries_intact() and dg.canaries_intact()
    sb.saps_destroy(ctx)


def test_scheduler_loop_captured_in_a_cuda_graph_and_replayed(sb):
    # Every device operation of the library is enqueued on the caller's stream and, after the
    # first use of a context, nothing is allocated: a round loop can be captured in a CUDA graph.
    # saps_set_run_ahead just before the capture makes the captured sequence self-contained (its
    # first round counts its own mask inside the graph instead of relying on a kernel that ran
    # before the capture).  Replaying the graph repeats the same rounds t = 1..T on the model as
    # it is then; both executions are checked against the oracle.
    torch = torch_cuda()
    w = synth.WORKLOADS["resnet20"]
    T, p = 10, w.keep_fracs[0]
    x, g = synth.model_and_grad(w)
    ld = round_up(w.N, 32)
    dx, dg = DeviceMatrix(x, ld), DeviceMatrix(g, ld)
    rng = synth.matching_rng(5)
    pairs_list = np.stack([synth.random_perfect_matching(w.n, rng) for _ in range(T)]).astype(np.int32)
    ctx = sb.saps_create_ld(w.n, w.N, ld, w.seed)
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.zeros(w.n, cap, dtype=torch.float32, device="cuda")
    idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
    counts = torch.zeros(T, dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    # first use outside the capture: the context allocates its scratch here
    scratch_x = dx.view.clone()
    with torch.cuda.stream(side):
        sb.saps_run_rounds_pack(ctx, scratch_x, dg.ptr, w.lr, 1, 2, p, vals, idx, counts, pairs_list=pairs_list[:2],
                                stream=side)
    side.synchronize()
    assert sb.saps_status(ctx, side) == 0
    sb.saps_set_run_ahead(ctx, True)                      # forget counts taken ahead by the warm-up
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        sb.saps_run_rounds_pack(ctx, dx.ptr, dg.ptr, w.lr, 1, T, p, vals, idx, counts, pairs_list=pairs_list,
                                stream=torch.cuda.current_stream())
    want = x.copy()
    for replay in range(2):
        graph.replay()
        torch.cuda.synchronize()
        assert sb.saps_status(ctx) == 0
        for t in range(1, T + 1):
            oracle.sgd(want, g, w.lr)
            m = oracle.mask(w.seed, t, p, w.N)
            assert int(counts[t - 1]) == int(m.sum())
            if t == T:
                wv, wi, wc = oracle.pack(want, m, cap)
            oracle.pair_average(want, pairs_list[t - 1], m)
        assert (idx.cpu().numpy().view(np.uint32)[:wc] == wi[:wc]).all()
        assert_bits_equal(vals.cpu().numpy()[:, :wc], wv[:, :wc], f"wire buffer after replay {replay}")
        assert_bits_equal(dx.host(), want, f"model after replay {replay}")
    assert dx.canaries_intact()
    del graph
    sb.saps_destroy(ctx)
