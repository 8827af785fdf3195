"""GPU parity of the widened path: Eq. 7 update order, per-round learning rates, the receiving
side of the exchange (unpack-average), the consensus distance, and the bounded wait."""
import numpy as np
import pytest

import oracle
from paper_2002_09692_b200 import synth
from gpu_util import DeviceMatrix, assert_bits_equal, round_up, torch_cuda

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


@pytest.mark.parametrize("N,ld", [(7, 7), (2050, 2052), (40_003, 40_032), (40_003, 40_003), (5 * 2048, 5 * 2048)])
@pytest.mark.parametrize("p", [0.0, 0.1, 1.0])
def test_eq7_order_round_and_emission(sb, N, ld, p):
    torch = torch_cuda()
    n, lr = 6, 0.1
    pairs = [1, 0, 2, 5, 4, 3]
    x = synth.gaussian_matrix(n, N, 1.0, 23, 0)
    g = synth.gaussian_matrix(n, N, 0.05, 23, 1)
    ctx = sb.saps_create_ld(n, N, ld, 23)
    sb.saps_set_update_order(ctx, sb.SAPS_ORDER_GOSSIP_FIRST)
    # plain round
    dx, dg = DeviceMatrix(x, ld), DeviceMatrix(g, ld)
    sb.saps_round(ctx, dx.ptr, dg.ptr, lr, pairs, 3, p)
    want = x.copy()
    m = oracle.gossip_round_eq7(want, g, lr, pairs, 23, 3, p)
    torch.cuda.synchronize()
    assert_bits_equal(dx.host(), want, "Eq. 7 order")
    assert dx.canaries_intact()
    # with emission: the wire buffer holds the current model x (nothing subtracted yet)
    dx2 = DeviceMatrix(x, ld)
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.full((n * cap,), 123.0, dtype=torch.float32, device="cuda")
    idx = torch.full((cap,), -1, dtype=torch.int32, device="cuda")
    count = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    sb.saps_round_pack(ctx, dx2.ptr, dg.ptr, lr, pairs, 3, p, vals, idx, count)
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == 0
    wv, wi, wc = oracle.pack(x, m, cap)
    assert int(count[0]) == wc
    assert_bits_equal(vals.cpu().numpy().reshape(n, cap)[:, :wc], wv[:, :wc], "Eq. 7 wire buffer")
    assert_bits_equal(dx2.host(), want, "Eq. 7 order with emission")
    # switching back restores Algorithm 2's order
    sb.saps_set_update_order(ctx, sb.SAPS_ORDER_SGD_FIRST)
    dx3 = DeviceMatrix(x, ld)
    sb.saps_round(ctx, dx3.ptr, dg.ptr, lr, pairs, 3, p)
    torch.cuda.synchronize()
    want2 = x.copy()
    oracle.gossip_round(want2, g, lr, pairs, 23, 3, p)
    assert_bits_equal(dx3.host(), want2, "Algorithm 2 order")
    sb.saps_destroy(ctx)


def test_run_rounds_with_learning_rate_schedule(sb):
    torch = torch_cuda()
    n, N, T, p = 8, 20_000, 9, 0.2
    x = synth.gaussian_matrix(n, N, 0.05, 24, 0)
    g = synth.gaussian_matrix(n, N, 0.01, 24, 1)
    rng = synth.matching_rng(24)
    plist = np.stack([synth.random_perfect_matching(n, rng) for _ in range(T)]).astype(np.int32)
    lrs = (0.1 / np.sqrt(np.arange(1, T + 1))).astype(np.float32)       # gamma_t = gamma / sqrt(t)
    for order, fn in ((0, oracle.gossip_round), (1, oracle.gossip_round_eq7)):
        dx, dg = DeviceMatrix(x, round_up(N, 32)), DeviceMatrix(g, round_up(N, 32))
        ctx = sb.saps_create_ld(n, N, round_up(N, 32), 24)
        sb.saps_set_update_order(ctx, order)
        sb.saps_run_rounds(ctx, dx.ptr, dg.ptr, 0.0, 1, T, p, pairs_list=plist, lr_list=lrs)
        torch.cuda.synchronize()
        sb.saps_destroy(ctx)
        want = x.copy()
        for t in range(1, T + 1):
            fn(want, g, float(lrs[t - 1]), plist[t - 1], 24, t, p)
        assert_bits_equal(dx.host(), want, f"schedule, order {order}")


@pytest.mark.parametrize("N,p", [(33, 0.5), (70_001, 0.05), (300_000, 0.01), (4096, 1.0), (5000, 0.0),
                                 (70_001, 0.5), (2043, 1.0)])
@pytest.mark.parametrize("align", [4, 8, 32])
def test_wire_path_sgd_pack_exchange_unpack(sb, N, p, align):
    # SGD-only round -> saps_pack -> (buffers travel) -> saps_unpack_avg  ==  fused saps_round,
    # for sparse and dense masks (several kept columns per 32-byte sector) and row strides of
    # every alignment.
    torch = torch_cuda()
    n, lr = 6, 0.05
    pairs = [3, 4, 2, 0, 1, 5]                  # workers 2 and 5 have no peer
    x = synth.gaussian_matrix(n, N, 1.0, 25, 0)
    g = synth.gaussian_matrix(n, N, 0.01, 25, 1)
    ld = round_up(N, align) + (4 if align == 4 and round_up(N, 4) % 8 == 0 else 0)
    ctx = sb.saps_create_ld(n, N, ld, 25)
    fused, dg = DeviceMatrix(x, ld), DeviceMatrix(g, ld)
    sb.saps_round(ctx, fused.ptr, dg.ptr, lr, pairs, 2, p)
    wire = DeviceMatrix(x, ld)
    sb.saps_round(ctx, wire.ptr, dg.ptr, lr, list(range(n)), 2, p)
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.zeros(n, cap, dtype=torch.float32, device="cuda")
    idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
    count = torch.zeros(1, dtype=torch.int32, device="cuda")
    sb.saps_pack(ctx, wire.ptr, 2, p, vals, idx, count)
    sb.saps_unpack_avg(ctx, wire.ptr, vals, idx, count, p, pairs)
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == 0
    assert_bits_equal(wire.host(), fused.host(), "wire path vs fused round")
    assert wire.canaries_intact()
    # against the oracle's receiving side, with an explicitly permuted receive buffer
    a = x.copy()
    oracle.sgd(a, g, lr)
    m = oracle.mask(25, 2, p, N)
    wv, wi, wc = oracle.pack(a, m, cap)
    recv_host = np.ascontiguousarray(wv[pairs])
    want = a.copy()
    oracle.unpack_avg(want, recv_host, wi, min(wc, cap))
    recv_dev = torch.from_numpy(recv_host).cuda()
    wire2 = DeviceMatrix(a, ld)
    sb.saps_unpack_avg(ctx, wire2.ptr, recv_dev, idx, count, p, None)      # row i = what i received
    torch.cuda.synchronize()
    assert_bits_equal(wire2.host(), want, "unpack-average, pairs=None")
    sb.saps_destroy(ctx)


@pytest.mark.parametrize("n,N,ld", [(2, 1, 1), (4, 2049, 2052), (32, 100_003, 100_032), (64, 5000, 5000)])
def test_consensus_distance(sb, n, N, ld):
    torch = torch_cuda()
    x = synth.gaussian_matrix(n, N, 0.05, 26, 0)
    x += np.float32(3.0)                        # a large common offset: deviations are small against it
    dx = DeviceMatrix(x, ld)
    ctx = sb.saps_create_ld(n, N, ld, 26)
    out = torch.zeros(2, dtype=torch.float64, device="cuda")
    sb.saps_consensus_distance(ctx, dx.ptr, out)
    torch.cuda.synchronize()
    want = oracle.consensus_distance(x)
    got = float(out[0])
    assert abs(got - want) <= 1e-10 * want + 1e-300, (got, want)
    assert float(out[1]) == 0.0
    # reproducible: the same bits on a second call
    out2 = torch.zeros(1, dtype=torch.float64, device="cuda")
    sb.saps_consensus_distance(ctx, dx.ptr, out2)
    assert float(out2[0]) == got
    # identical workers: exactly zero
    same = np.repeat(x[:1], n, axis=0)
    ds = DeviceMatrix(same, ld)
    sb.saps_consensus_distance(ctx, ds.ptr, out)
    torch.cuda.synchronize()
    assert float(out[0]) == 0.0
    sb.saps_destroy(ctx)


def test_consensus_distance_follows_lemma_2_on_the_gpu(sb):
    # sparse gossip contracts the consensus distance by q + p * lambda2 per round (Lemma 2)
    torch = torch_cuda()
    n, N, p = 32, 300_000, 0.25
    x = synth.gaussian_matrix(n, N, 1.0, 27, 0)
    dx = DeviceMatrix(x, round_up(N, 32))
    ctx = sb.saps_create_ld(n, N, round_up(N, 32), 27)
    rng = synth.matching_rng(27)
    out = torch.zeros(7, dtype=torch.float64, device="cuda")
    sb.saps_consensus_distance(ctx, dx.ptr, out[0:])
    for t in range(1, 7):
        sb.saps_round(ctx, dx.ptr, None, 0.0, synth.random_perfect_matching(n, rng), t, p)
        sb.saps_consensus_distance(ctx, dx.ptr, out[t:])
    torch.cuda.synchronize()
    sb.saps_destroy(ctx)
    d = out.cpu().numpy()
    phat = oracle.threshold(p) / 2.0 ** 32
    want = (1 - phat) + phat * (n - 2) / (2.0 * (n - 1))
    ratios = d[1:] / d[:-1]
    assert abs(ratios[0] - want) < 0.01 * want and abs(ratios.mean() - want) < 0.01 * want


def test_bounded_wait_reports_a_timeout_instead_of_hanging(sb):
    # one look-back tile never publishes; its successors give up after a short poll budget and the
    # kernel returns with SAPS_ERR_TIMEOUT in the status word; the context stays usable
    torch = torch_cuda()
    n, N, p = 2, 40 * 2048, 0.05
    x = synth.gaussian_matrix(n, N, 1.0, 28, 0)
    dx = DeviceMatrix(x, N)
    ctx = sb.saps_create(n, N, 28)
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.zeros(n, cap, dtype=torch.float32, device="cuda")
    idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
    count = torch.zeros(1, dtype=torch.int32, device="cuda")
    sb.saps_debug_inject(ctx, 3, 200)                       # tile 3 stays silent, 200 polls
    sb.saps_pack(ctx, dx.ptr, 1, p, vals, idx, count)
    assert sb.saps_status(ctx) == sb.SAPS_ERR_TIMEOUT
    sb.saps_debug_inject(ctx, 0xFFFFFFFF, 0)                # hook off, default budget
    sb.saps_pack(ctx, dx.ptr, 1, p, vals, idx, count)
    assert sb.saps_status(ctx) == 0
    wv, wi, wc = oracle.pack(x, oracle.mask(28, 1, p, N), cap)
    assert int(count[0]) == wc
    assert_bits_equal(vals.cpu().numpy()[:, :wc], wv[:, :wc], "pack after a timed-out call")
    sb.saps_destroy(ctx)


@pytest.mark.parametrize("N,ld", [(40_000, 40_000), (6_151, 6_152), (2_048, 2_048)])
def test_staged_round_whose_wait_runs_out_falls_back_to_plain_accesses(sb, N, ld):
    # The staged form of the fused round waits, bounded, for its bulk copies.  The hook makes that
    # wait count as run out in every block: the threads then read and write global memory
    # themselves.  The round, the wire buffer and the next round must still equal the oracle's,
    # the status word must say SAPS_ERR_TIMEOUT, and the context must work normally afterwards.
    torch = torch_cuda()
    n, p, lr, seed = 6, 0.05, 0.1, 41
    x = synth.gaussian_matrix(n, N, 1.0, seed, 0)
    g = synth.gaussian_matrix(n, N, 0.01, seed, 1)
    dx, dg = DeviceMatrix(x, ld), DeviceMatrix(g, ld)
    ctx = sb.saps_create_ld(n, N, ld, seed)
    sb.saps_set_staging(ctx, sb.SAPS_STAGING_BULK)
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.zeros(n, cap, dtype=torch.float32, device="cuda")
    idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
    count = torch.zeros(1, dtype=torch.int32, device="cuda")
    want = x.copy()
    pairs = [1, 0, 3, 2, 4, 5]                      # two pairs and two single workers
    for t, give_up, emit in ((1, True, True), (2, True, False), (3, False, True), (4, False, False)):
        sb.saps_debug_staging_wait(ctx, give_up)
        a = want.copy()
        oracle.sgd(a, g, lr)
        if emit:
            sb.saps_round_pack(ctx, dx.ptr, dg.ptr, lr, pairs, t, p, vals, idx, count)
        else:
            sb.saps_round(ctx, dx.ptr, dg.ptr, lr, pairs, t, p)
        torch.cuda.synchronize()
        assert sb.saps_status(ctx) == (sb.SAPS_ERR_TIMEOUT if give_up else 0), (t, give_up)
        m = oracle.gossip_round(want, g, lr, pairs, seed, t, p)
        assert_bits_equal(dx.host(), want, f"round {t}, wait given up: {give_up}")
        if emit:
            kept = np.nonzero(m)[0]
            c = int(count.cpu().numpy().view(np.uint32)[0])
            assert c == len(kept)
            assert (idx[:c].cpu().numpy().view(np.uint32) == kept.astype(np.uint32)).all()
            assert_bits_equal(vals[:, :c].cpu().numpy(), a[:, kept], f"wire buffer of round {t}")
    assert dx.canaries_intact() and dg.canaries_intact()
    assert_bits_equal(dg.host(), g, "gradient must not change")
    sb.saps_destroy(ctx)


@pytest.mark.parametrize("direct", [False, True])
def test_row_sharded_round_emulated_on_one_gpu(sb, direct):
    # Two "ranks" of 4 workers each, run one after the other on this GPU; the transfer between
    # them is a device copy of the packed rows, or (direct) the fused pass of each rank writes
    # its packed rows straight into the other rank's receive buffer through a table of
    # destinations.  The result must equal the single-context round.
    torch = torch_cuda()
    from paper_2002_09692_b200.row_sharded import RowShardedGossip
    world, per_rank, N, p, lr, seed = 2, 4, 30_000, 0.05, 0.05, 33
    n = world * per_rank
    ld = round_up(N, 32)
    x = synth.gaussian_matrix(n, N, 1.0, 33, 0)
    g = synth.gaussian_matrix(n, N, 0.01, 33, 1)
    rng = synth.matching_rng(33)
    ranks = [RowShardedGossip(r, world, per_rank, N, ld, seed) for r in range(world)]
    dxs = [DeviceMatrix(np.ascontiguousarray(x[r * per_rank:(r + 1) * per_rank]), ld) for r in range(world)]
    dgs = [DeviceMatrix(np.ascontiguousarray(g[r * per_rank:(r + 1) * per_rank]), ld) for r in range(world)]
    cap = sb.saps_pack_capacity(ranks[0].ctx, p)
    bufs = [dict(vals=torch.zeros(per_rank, cap, device="cuda"), recv=torch.zeros(per_rank, cap, device="cuda"),
                 idx=torch.zeros(cap, dtype=torch.int32, device="cuda"),
                 table=torch.zeros(per_rank, dtype=torch.int64, device="cuda"),
                 count=torch.zeros(1, dtype=torch.int32, device="cuda")) for _ in range(world)]
    want = x.copy()
    crossed = 0
    for t in range(1, 6):
        pairs = synth.random_perfect_matching(n, rng)
        if direct:
            bases = [bufs[r]["recv"].data_ptr() for r in range(world)]
            for b in bufs:
                b["recv"].fill_(float("nan"))               # nothing stale may be averaged in
            plans = [ranks[r].local_step_direct(dxs[r].ptr, dgs[r].ptr, lr, pairs, t, p, bases, bufs[r]["table"],
                                                bufs[r]["idx"], bufs[r]["count"]) for r in range(world)]
            torch.cuda.synchronize()                        # "my pass has finished" reaches the peer
            crossed += sum(len(pl.transfers) for pl in plans)
        else:
            plans = [ranks[r].local_step(dxs[r].ptr, dgs[r].ptr, lr, pairs, t, p, bufs[r]["vals"], bufs[r]["idx"],
                                         bufs[r]["count"]) for r in range(world)]
            for r in range(world):                          # the wire: each packed row goes to its peer's rank
                for row, peer, _tag in plans[r].transfers:
                    j = int(pairs[r * per_rank + row])
                    bufs[peer]["recv"][j - peer * per_rank].copy_(bufs[r]["vals"][row])
                    crossed += 1
        for r in range(world):
            ranks[r].merge(dxs[r].ptr, plans[r], bufs[r]["recv"], bufs[r]["idx"], bufs[r]["count"], p)
        oracle.gossip_round(want, g, lr, pairs, seed, t, p)
    torch.cuda.synchronize()
    assert crossed > 0
    got = np.concatenate([d.host() for d in dxs], axis=0)
    assert_bits_equal(got, want, "row-sharded round")
    assert all(d.canaries_intact() for d in dxs)
    for rk in ranks:
        rk.close()
    # the explicit row map refuses rows outside the context
    ctx = sb.saps_create(4, 100, 0)
    assert sb._lib.saps_unpack_avg_rows(ctx, 0x1000, 0x1000, 0x1000, 0x1000, 0.5, sb._pairs([0, 1, 2, 4]), None) \
        == sb.SAPS_ERR_INVALID
    sb.saps_destroy(ctx)
