"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times
(row stride rounded up to 32, saps_select_peers + saps_round_pack on the current stream).

vgg16-sized: every element of two whole rounds against the oracle.
resnet50- and gpt2s-sized: inputs are drawn on the device; the rows of a few sampled pairs
are checked element by element against the oracle (the mask depends on the column only, so
the oracle can run on a row subset), and properties that hold at any size are checked on
all rows with device arithmetic.
"""
import numpy as np
import pytest

import oracle
from paper_2002_09692_b200 import synth
from gpu_util import assert_bits_equal, round_up, torch_cuda
from helpers import golden_records

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sb():
    torch_cuda()
    from paper_2002_09692_b200 import binding
    return binding


def _golden_count(seed, t, N, p):
    for r in golden_records("mask_hash.txt"):
        if r[0] == "count" and (int(r[1]), int(r[2]), int(r[3]), float(r[4])) == (seed, t, N, p):
            return int(r[5])
    return None


def _oracle_round_with_pack(x, g, w, pairs, t, p, cap):
    """One round of the oracle in Algorithm 2's order, in place on x; returns the wire buffer."""
    oracle.sgd(x, g, w.lr)
    m = oracle.mask(w.seed, t, p, w.N)
    wv, wi, wc = oracle.pack(x, m, cap)
    oracle.pair_average(x, np.asarray(pairs, dtype=np.int32), m)
    return wv, wi, wc


def test_vgg16_consecutive_rounds_every_element(sb):
    # The mode the benchmark times, at the size it times it: one context, keep_frac fixed at
    # 0.01, saps_select_peers + saps_round_pack on consecutive rounds, so that from the second
    # round on the per-tile counts (7,192 tiles) are the ones the previous fused kernel counted
    # ahead.  Every element of x, the count, the index list and the packed values are compared
    # with the oracle after every round.  A fourth round at keep_frac 0.001 then takes the
    # other route (counts from a kernel of their own).  The same first three rounds are then
    # repeated from the initial model through the C-side loop saps_run_rounds_pack.
    torch = torch_cuda()
    w = synth.WORKLOADS["vgg16"]
    n, N, ld = w.n, w.N, round_up(w.N, 32)
    x, g = synth.model_and_grad(w)
    x0 = x.copy()
    B = synth.bandwidth_matrix(n, *w.bw_range, seed=w.seed)
    dx = torch.zeros(n, ld, dtype=torch.float32, device="cuda")
    dg = torch.zeros(n, ld, dtype=torch.float32, device="cuda")
    dx[:, :N].copy_(torch.from_numpy(x))
    dg[:, :N].copy_(torch.from_numpy(g))
    ctx = sb.saps_create_ld(n, N, ld, w.seed)
    schedule = [(1, 0.01), (2, 0.01), (3, 0.01), (4, 0.001)]
    used_pairs, counts3 = [], []
    last3 = None
    for t, p in schedule:
        cap = sb.saps_pack_capacity(ctx, p)
        vals = torch.zeros(n, cap, dtype=torch.float32, device="cuda")
        idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
        count = torch.zeros(1, dtype=torch.int32, device="cuda")
        pairs = sb.saps_select_peers(ctx, B, t, n)
        sb.saps_round_pack(ctx, dx, dg, w.lr, pairs, t, p, vals, idx, count)
        torch.cuda.synchronize()
        assert sb.saps_status(ctx) == 0
        wv, wi, wc = _oracle_round_with_pack(x, g, w, pairs, t, p, cap)
        if (t, p) == (1, 0.01):
            assert wc == _golden_count(0, 1, N, p) == 147_227
        assert int(count[0]) == wc, f"count of round {t}"
        assert (idx[:wc].cpu().numpy().view(np.uint32) == wi[:wc]).all(), f"index list of round {t}"
        assert_bits_equal(vals[:, :wc].cpu().numpy(), wv[:, :wc], f"wire buffer of round {t}")
        assert_bits_equal(dx[:, :N].cpu().numpy(), x, f"model after round {t}")
        assert float(dx[:, N:].abs().max()) == 0.0       # padding columns untouched
        if p == 0.01:
            used_pairs.append(pairs)
            counts3.append(wc)
            if t == 3:
                last3 = (x.copy(), wv[:, :wc].copy(), wi[:wc].copy())
    sb.saps_destroy(ctx)
    del x

    # the same three rounds through the scheduler loop, selection included, in one call
    want_x, want_v, want_i = last3
    dx[:, :N].copy_(torch.from_numpy(x0))
    ctx = sb.saps_create_ld(n, N, ld, w.seed)
    cap = sb.saps_pack_capacity(ctx, 0.01)
    vals = torch.zeros(n, cap, dtype=torch.float32, device="cuda")
    idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
    counts = torch.zeros(3, dtype=torch.int32, device="cuda")
    log = np.zeros((3, n), dtype=np.int32)
    sb.saps_run_rounds_pack(ctx, dx, dg, w.lr, 1, 3, 0.01, vals, idx, counts, bandwidth=B, out_pairs_log=log)
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == 0
    sb.saps_destroy(ctx)
    assert log.tolist() == [list(p) for p in used_pairs]          # same matchings as call by call
    assert counts.cpu().numpy().view(np.uint32).tolist() == counts3
    c = counts3[-1]
    assert (idx[:c].cpu().numpy().view(np.uint32) == want_i).all()
    assert_bits_equal(vals[:, :c].cpu().numpy(), want_v, "wire buffer of round 3 from the scheduler loop")
    assert_bits_equal(dx[:, :N].cpu().numpy(), want_x, "model after three scheduled rounds")
    assert float(dx[:, N:].abs().max()) == 0.0


def test_vgg16_host_pipeline_every_element(sb):
    # The end-to-end entry point at the size and in the configuration bench.py times it: pinned
    # host matrices in, 15 column chunks over three lanes, model and wire buffer out; two
    # consecutive rounds (the second one uses counts taken ahead by the first one's chunk kernels),
    # every element against the oracle.
    torch = torch_cuda()
    w = synth.WORKLOADS["vgg16"]
    n, N, ld, p = w.n, w.N, round_up(w.N, 32), 0.01
    x, g = synth.model_and_grad(w)
    B = synth.bandwidth_matrix(n, *w.bw_range, seed=w.seed)
    hx = torch.from_numpy(x.copy()).pin_memory()
    hg = torch.from_numpy(g).pin_memory()
    d_x = torch.zeros(n, ld, dtype=torch.float32, device="cuda")
    d_g = torch.zeros(n, ld, dtype=torch.float32, device="cuda")
    ctx = sb.saps_create_ld(n, N, ld, w.seed)
    cap = sb.saps_pack_capacity(ctx, p)
    hv = torch.zeros(n, cap, dtype=torch.float32).pin_memory()
    hi = torch.zeros(cap, dtype=torch.int32).pin_memory()
    hc = torch.zeros(1, dtype=torch.int32).pin_memory()
    d_v = torch.zeros(n, cap, dtype=torch.float32, device="cuda")
    d_i = torch.zeros(cap, dtype=torch.int32, device="cuda")
    d_c = torch.zeros(1, dtype=torch.int32, device="cuda")
    for t in (1, 2):
        pairs = sb.saps_select_peers(ctx, B, t, n)
        sb.saps_round_pack_host(ctx, hx, hg, w.lr, pairs, t, p, d_x, d_g, hv, hi, hc, d_v, d_i, d_c)
        assert sb.saps_status(ctx) == 0
        wv, wi, wc = _oracle_round_with_pack(x, g, w, pairs, t, p, cap)
        assert int(hc[0]) == wc
        assert (hi.numpy().view(np.uint32)[:wc] == wi[:wc]).all()
        assert_bits_equal(hv.numpy()[:, :wc], wv[:, :wc], f"host wire buffer, round {t}")
        assert_bits_equal(hx.numpy(), x, f"host model after round {t}")
    assert float(d_x[:, N:].abs().max()) == 0.0 and float(d_g[:, N:].abs().max()) == 0.0
    sb.saps_destroy(ctx)


def _sampled_rounds(sb, torch, w, p, pairs_of_round, rows_of_round, golden=None):
    """Bench-style consecutive rounds t = 1, 2, ... on one context (fixed keep_frac, so every
    round after the first uses the counts the previous kernel took ahead) on device-drawn
    inputs.  After every round: the sampled rows against the oracle element by element, the
    index list and the count against the oracle's mask, and properties that hold at any size
    on all rows with device arithmetic.  rows_of_round[t-1] is closed under round t's matching
    and contains rows_of_round[t]: the oracle follows exactly the rows whose whole history it
    has seen."""
    n, N, ld = w.n, w.N, round_up(w.N, 32)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(99 + int(p * 1e6))
    dx = torch.empty(n, ld, dtype=torch.float32, device="cuda").normal_(0.0, w.x_std, generator=gen)
    dg = torch.empty(n, ld, dtype=torch.float32, device="cuda").normal_(0.0, w.g_std, generator=gen)
    first = sorted(rows_of_round[0])
    state = {r: dx[r, :N].cpu().numpy() for r in first}              # the oracle's copy of the rows
    grad = {r: dg[r, :N].cpu().numpy() for r in first}
    ctx = sb.saps_create_ld(n, N, ld, w.seed)
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.zeros(n, cap, dtype=torch.float32, device="cuda")
    idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
    count = torch.zeros(1, dtype=torch.int32, device="cuda")
    bits = torch.zeros(round_up(N, 32) // 32, dtype=torch.int32, device="cuda")
    shifts = torch.arange(32, device="cuda", dtype=torch.int32)
    for t, pairs in enumerate(pairs_of_round, start=1):
        rows = sorted(rows_of_round[t - 1])
        local = {r: i for i, r in enumerate(rows)}
        assert all(int(pairs[r]) in local for r in rows) and all(r in state for r in rows)
        a = (dx - w.lr * dg)[:, :N]                       # two roundings per element, like the round
        sb.saps_mask(ctx, t, p, bits)
        sb.saps_round_pack(ctx, dx, dg, w.lr, pairs, t, p, vals, idx, count)
        torch.cuda.synchronize()
        assert sb.saps_status(ctx) == 0

        # -- element by element on the sampled rows --
        x_s = np.stack([state[r] for r in rows])
        g_s = np.stack([grad[r] for r in rows])
        m = oracle.gossip_round(x_s, g_s, w.lr, [local[int(pairs[r])] for r in rows], w.seed, t, p)
        for i, r in enumerate(rows):
            state[r] = x_s[i]
        c = int(count[0])
        assert c == int(m.sum(dtype=np.int64)), f"count of round {t}"
        if golden is not None and t == 1:
            assert c == golden
        assert_bits_equal(dx[rows, :N].cpu().numpy(), x_s, f"sampled rows {rows}, round {t}")
        kept = np.nonzero(m)[0]
        assert (idx[:c].cpu().numpy().view(np.uint32) == kept.astype(np.uint32)).all(), f"index list, round {t}"
        del x_s, g_s

        # -- properties on every row, on the device --
        mdev = ((bits[:, None] >> shifts[None, :]) & 1).bool().reshape(-1)[:N]
        assert int(mdev.sum()) == c
        out = dx[:, :N]
        peer = torch.as_tensor(np.asarray(pairs), device="cuda", dtype=torch.long)
        assert torch.equal(torch.where(mdev[None, :], a, out), a)               # unmasked: SGD step only
        om, am = out[:, mdev], a[:, mdev]
        assert torch.equal(om, om[peer])                                        # peers agree bitwise
        assert torch.equal(om + om[peer], am + am[peer])                        # pair sums to one rounding
        assert torch.equal(vals[:, :c], am)                                     # wire buffer = a o m
        del a, mdev, out, om, am
    sb.saps_destroy(ctx)


def _history_cone(pairs_of_round, last_rows):
    """rows[t]: the workers whose values influence `last_rows` from round t+1 on, i.e. the set to
    follow in round t+1: rows[T-1] = last_rows + their peers in round T, rows[t-1] = rows[t] +
    their peers in round t."""
    rows = [None] * len(pairs_of_round)
    cur = set(last_rows)
    for t in range(len(pairs_of_round) - 1, -1, -1):
        cur = cur | {int(pairs_of_round[t][r]) for r in cur}
        rows[t] = set(cur)
    return rows


def test_resnet50_keep_frac_sweep_sampled_rows(sb):
    # uniformly random perfect matchings; three consecutive rounds per keep_frac on one context;
    # the oracle follows workers 0 and 17 and everyone whose values reach them (at most 16 rows
    # at t = 1, 8 at t = 2, 4 at t = 3)
    torch = torch_cuda()
    w = synth.WORKLOADS["resnet50"]
    rng = synth.matching_rng(w.seed)
    for p in w.keep_fracs:
        rounds = [synth.random_perfect_matching(w.n, rng) for _ in range(3)]
        _sampled_rounds(sb, torch, w, p, rounds, _history_cone(rounds, {0, 17}),
                        golden=_golden_count(2, 1, w.N, p))
        torch.cuda.empty_cache()


def test_gpt2s_sampled_rows(sb):
    # adaptive peer selection (Algorithm 3) for three consecutive rounds; the oracle follows
    # worker 5 and everyone whose values reach it (8 rows at t = 1, 4 at t = 2, 2 at t = 3)
    torch = torch_cuda()
    w = synth.WORKLOADS["gpt2s"]
    B = synth.bandwidth_matrix(w.n, *w.bw_range, seed=w.seed)
    ctx = sb.saps_create(w.n, 16, w.seed)
    rounds = [sb.saps_select_peers(ctx, B, t, w.n) for t in (1, 2, 3)]
    sb.saps_destroy(ctx)
    rows = _history_cone(rounds, {5})
    assert len(rows[0]) <= 8 and len(rows[2]) == 2
    _sampled_rounds(sb, torch, w, 0.01, rounds, rows, golden=_golden_count(0, 1, w.N, 0.01))
    torch.cuda.empty_cache()


def _many_rounds_on_column_windows(sb, torch, w, p, T, windows, bandwidth=None, pairs_list=None):
    """The configured number of rounds at full size in ONE scheduler call (saps_run_rounds_pack),
    followed on the CPU by the oracle on a few column windows of ALL workers: the mask depends on
    the column only and the update acts column by column, so a window can be replayed on its own
    (SGD step, that window of the full-length oracle mask, pair average).  Checked: every round's
    count against the oracle's mask, the final model on the windows, the last round's index list
    and the windows' part of the last wire buffer."""
    n, N, ld = w.n, w.N, round_up(w.N, 32)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(4321 + T)
    dx = torch.empty(n, ld, dtype=torch.float32, device="cuda").normal_(0.0, w.x_std, generator=gen)
    dg = torch.empty(n, ld, dtype=torch.float32, device="cuda").normal_(0.0, w.g_std, generator=gen)
    xs = [np.ascontiguousarray(dx[:, c0:c1].cpu().numpy()) for c0, c1 in windows]
    gs = [np.ascontiguousarray(dg[:, c0:c1].cpu().numpy()) for c0, c1 in windows]
    padding = dx[:, N:].clone()
    ctx = sb.saps_create_ld(n, N, ld, w.seed)
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.zeros(n, cap, dtype=torch.float32, device="cuda")
    idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
    counts = torch.zeros(T, dtype=torch.int32, device="cuda")
    log = np.zeros((T, n), dtype=np.int32)
    sb.saps_run_rounds_pack(ctx, dx, dg, w.lr, 1, T, p, vals, idx, counts, pairs_list=pairs_list,
                            bandwidth=bandwidth, out_pairs_log=log)
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == 0
    sb.saps_destroy(ctx)
    got_counts = counts.cpu().numpy().view(np.uint32)
    for t in range(1, T + 1):
        m = oracle.mask(w.seed, t, p, N)
        assert int(got_counts[t - 1]) == int(m.sum(dtype=np.int64)), f"count of round {t}"
        for (c0, c1), xw, gw in zip(windows, xs, gs):
            oracle.sgd(xw, gw, w.lr)
            if t == T:
                kept = np.nonzero(m)[0]
                c = len(kept)
                assert (idx[:c].cpu().numpy().view(np.uint32) == kept.astype(np.uint32)).all()
                lo, hi = np.searchsorted(kept, [c0, c1])
                assert_bits_equal(vals[:, lo:hi].cpu().numpy(), xw[:, kept[lo:hi] - c0],
                                  f"last wire buffer, columns [{c0}, {c1})")
            oracle.pair_average(xw, log[t - 1], np.ascontiguousarray(m[c0:c1]))
    for (c0, c1), xw in zip(windows, xs):
        assert_bits_equal(dx[:, c0:c1].cpu().numpy(), xw, f"model after {T} rounds, columns [{c0}, {c1})")
    assert torch.equal(dx[:, N:], padding)                 # columns beyond N are never written
    return log


def _windows(N):
    # the first tiles, an unaligned stretch in the middle, and the ragged end of the rows
    mid = (N // 2) | 1
    return [(0, 150_000), (mid, mid + 100_001), (N - 150_003, N)]


def test_vgg16_fifty_rounds_adaptive_selection(sb):
    # 50 rounds at each keep_frac with Algorithm 3 choosing the peers, as the workload is specified
    torch = torch_cuda()
    w = synth.WORKLOADS["vgg16"]
    B = synth.bandwidth_matrix(w.n, *w.bw_range, seed=w.seed)
    for p in w.keep_fracs:
        log = _many_rounds_on_column_windows(sb, torch, w, p, w.rounds, _windows(w.N), bandwidth=B)
        assert len({tuple(r) for r in log}) > 25            # the matching keeps changing
        torch.cuda.empty_cache()


def test_resnet50_twenty_rounds_per_keep_frac(sb):
    # uniformly random perfect matching per round, 20 rounds for each keep_frac of the sweep
    torch = torch_cuda()
    w = synth.WORKLOADS["resnet50"]
    rng = synth.matching_rng(w.seed)
    for p in w.keep_fracs:
        pairs_list = np.stack([synth.random_perfect_matching(w.n, rng) for _ in range(w.rounds)]).astype(np.int32)
        _many_rounds_on_column_windows(sb, torch, w, p, w.rounds, _windows(w.N), pairs_list=pairs_list)
        torch.cuda.empty_cache()


def test_gpt2s_ten_rounds_adaptive_selection(sb):
    torch = torch_cuda()
    w = synth.WORKLOADS["gpt2s"]
    B = synth.bandwidth_matrix(w.n, *w.bw_range, seed=w.seed)
    _many_rounds_on_column_windows(sb, torch, w, w.keep_fracs[0], w.rounds, _windows(w.N), bandwidth=B)
    torch.cuda.empty_cache()


def test_largest_column_count(sb):
    # N just below 2^32 (the largest the 32-bit column index allows), ragged (N mod 4 = 3),
    # two workers, pure gossip with emission.  Checked against the oracle's hash on sampled and
    # on the very last columns, and by device-side invariants on all 8.6e9 elements.
    torch = torch_cuda()
    free, _ = torch.cuda.mem_get_info()
    if free < 100 * 2 ** 30:
        pytest.skip("needs about 100 GB of free device memory")
    n, N, ld, seed, t, p = 2, 2 ** 32 - 5, 2 ** 32, 7, 3, 1e-4
    x = torch.empty(n, ld, dtype=torch.float32, device="cuda").normal_(0.0, 1.0)
    x0 = x.clone()
    ctx = sb.saps_create_ld(n, N, ld, seed)
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.zeros(n, cap, dtype=torch.float32, device="cuda")
    idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
    count = torch.zeros(1, dtype=torch.int32, device="cuda")
    bits = torch.zeros(2 ** 27, dtype=torch.int32, device="cuda")
    sb.saps_mask(ctx, t, p, bits)
    sb.saps_round_pack(ctx, x, None, 0.0, [1, 0], t, p, vals, idx, count)
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == 0
    c = int(count.cpu().numpy().view(np.uint32)[0])
    thr = oracle.threshold(p)
    phat = thr / 2.0 ** 32
    assert abs(c - N * phat) < 5 * np.sqrt(N * phat * (1 - phat))
    # the bitmap agrees with the count, and has nothing at or beyond N
    words = bits.cpu().numpy().view(np.uint32)
    assert int(np.unpackbits(words.view(np.uint8)).sum(dtype=np.int64)) == c
    assert words[-1] >> 27 == 0                                   # columns 2^32-5 .. 2^32-1 do not exist
    # index list: strictly ascending, every sampled entry is a kept column by the oracle's hash
    cols = idx[:c].cpu().numpy().view(np.uint32).astype(np.int64)
    assert (np.diff(cols) > 0).all() and cols[-1] < N
    k0, k1 = oracle.round_key(seed, t)
    rng = np.random.default_rng(0)
    for r in list(rng.integers(0, c, 300)) + [0, c - 1]:
        assert oracle.hash_k(int(cols[r]), k0, k1) < thr
    # the last 2^17 columns, one by one: exactly the oracle's kept set (32-bit wrap would show here)
    lo = N - 2 ** 17
    want_tail = [k for k in range(lo, N) if oracle.hash_k(k, k0, k1) < thr]
    assert list(cols[cols >= lo]) == want_tail
    # wire buffer = the senders' values at the kept columns
    gather = torch.from_numpy(cols).cuda()
    assert torch.equal(vals[:, :c], x0[:, gather])
    # the model: kept columns hold the pair mean on both workers, everything else is untouched
    mean = 0.5 * (x0[0, gather] + x0[1, gather])
    assert torch.equal(x[0, gather], mean) and torch.equal(x[1, gather], mean)
    x0[:, gather] = x[:, gather]
    assert torch.equal(x, x0)                                     # includes the padding columns
    # the standalone compaction (two million look-back tiles) finds the same columns
    vals2 = torch.zeros(n, cap, dtype=torch.float32, device="cuda")
    idx2 = torch.zeros(cap, dtype=torch.int32, device="cuda")
    count2 = torch.zeros(1, dtype=torch.int32, device="cuda")
    sb.saps_pack(ctx, x, t, p, vals2, idx2, count2)
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == 0
    assert int(count2.cpu().numpy().view(np.uint32)[0]) == c and torch.equal(idx2[:c], idx[:c])
    assert torch.equal(vals2[:, :c], x[:, gather])
    del vals, idx, vals2, idx2, gather, mean, x0
    torch.cuda.empty_cache()
    # Two more rounds at a dense keep_frac: the second one takes its per-tile counts from the
    # first one's kernel, which counted them ahead; with N mod 4 = 3 the three leftover columns
    # are counted one thread each, and nfull + thread index must not wrap past 2^32 (a wrap
    # would count columns 0..247 a second time: 12 spurious hits expected at this density).
    p2 = 0.05
    cap2 = sb.saps_pack_capacity(ctx, p2)
    vals = torch.zeros(n, cap2, dtype=torch.float32, device="cuda")
    idx = torch.zeros(cap2, dtype=torch.int32, device="cuda")
    for t2 in (t + 1, t + 2):
        sb.saps_round_pack(ctx, x, None, 0.0, [1, 0], t2, p2, vals, idx, count)
        sb.saps_mask(ctx, t2, p2, bits)
        torch.cuda.synchronize()
        assert sb.saps_status(ctx) == 0
        c2 = int(count.cpu().numpy().view(np.uint32)[0])
        words = bits.cpu().numpy().view(np.uint32)
        assert c2 == int(np.bitwise_count(words).sum(dtype=np.int64)), f"count of round {t2}"
        cols = idx[:c2].cpu().numpy().view(np.uint32)
        assert int(cols[-1]) < N and int(cols[0]) >= 0
        lo = N - 2 ** 12
        k0, k1 = oracle.round_key(seed, t2)
        thr2 = oracle.threshold(p2)
        assert [int(k) for k in cols[cols >= lo]] == [k for k in range(lo, N) if oracle.hash_k(k, k0, k1) < thr2]
    del vals, idx
    torch.cuda.empty_cache()
    # consensus distance at this size: both workers identical (the keep_frac = 1 round makes them
    # so) except for one column that differs by exactly 1: || X - mean ||_F^2 = 2 * (1/2)^2
    sb.saps_round(ctx, x, None, 0.0, [1, 0], t + 3, 1.0)
    x[0, 0] = 0.25
    x[1, 0] = 1.25
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    sb.saps_consensus_distance(ctx, x, out)
    torch.cuda.synchronize()
    assert float(out[0]) == 0.5
    x[1, 0] = 0.25
    x[0, N - 1] = 0.5                                    # the very last column, served by the leftover path
    x[1, N - 1] = 2.5
    sb.saps_consensus_distance(ctx, x, out)
    torch.cuda.synchronize()
    assert float(out[0]) == 2.0                          # 2 * (2/2)^2
    sb.saps_destroy(ctx)
    del x
    torch.cuda.empty_cache()
