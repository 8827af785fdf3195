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


def test_vgg16_two_whole_rounds(sb):
    torch = torch_cuda()
    w = synth.WORKLOADS["vgg16"]
    n, N, ld = w.n, w.N, round_up(w.N, 32)
    x, g = synth.model_and_grad(w)
    B = synth.bandwidth_matrix(n, *w.bw_range, seed=w.seed)
    dx = torch.zeros(n, ld, dtype=torch.float32, device="cuda")
    dg = torch.zeros(n, ld, dtype=torch.float32, device="cuda")
    dx[:, :N].copy_(torch.from_numpy(x))
    dg[:, :N].copy_(torch.from_numpy(g))
    ctx = sb.saps_create_ld(n, N, ld, w.seed)
    for p in w.keep_fracs:                               # 0.01, then 0.001
        cap = sb.saps_pack_capacity(ctx, p)
        vals = torch.zeros(n, cap, dtype=torch.float32, device="cuda")
        idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
        count = torch.zeros(1, dtype=torch.int32, device="cuda")
        t = 1 if p == 0.01 else 2
        pairs = sb.saps_select_peers(ctx, B, t, n)
        sb.saps_round_pack(ctx, dx, dg, w.lr, pairs, t, p, vals, idx, count)
        torch.cuda.synchronize()
        assert sb.saps_status(ctx) == 0
        oracle.sgd(x, g, w.lr)
        m = oracle.mask(w.seed, t, p, N)
        wv, wi, wc = oracle.pack(x, m, cap)
        oracle.pair_average(x, pairs, m)
        if t == 1:
            assert wc == _golden_count(0, 1, N, p) == 147_227
        assert int(count[0]) == wc
        assert (idx[:wc].cpu().numpy().view(np.uint32) == wi[:wc]).all()
        assert_bits_equal(vals[:, :wc].cpu().numpy(), wv[:, :wc], f"wire buffer, keep_frac {p}")
        assert_bits_equal(dx[:, :N].cpu().numpy(), x, f"model after round {t}")
        assert float(dx[:, N:].abs().max()) == 0.0       # padding columns untouched
    sb.saps_destroy(ctx)


def _sampled_round(sb, torch, w, p, t, pairs, sample_rows, golden=None):
    """One bench-style round on device-drawn inputs; returns nothing, asserts parity."""
    n, N, ld = w.n, w.N, round_up(w.N, 32)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(99 + t)
    dx = torch.empty(n, ld, dtype=torch.float32, device="cuda").normal_(0.0, w.x_std, generator=gen)
    dg = torch.empty(n, ld, dtype=torch.float32, device="cuda").normal_(0.0, w.g_std, generator=gen)
    rows = sorted(sample_rows)
    x_s = dx[rows, :N].cpu().numpy()
    g_s = dg[rows, :N].cpu().numpy()
    a_dev = dx - w.lr * dg                              # two roundings per element, like the round
    ctx = sb.saps_create_ld(n, N, ld, w.seed)
    cap = sb.saps_pack_capacity(ctx, p)
    vals = torch.zeros(n, cap, dtype=torch.float32, device="cuda")
    idx = torch.zeros(cap, dtype=torch.int32, device="cuda")
    count = torch.zeros(1, dtype=torch.int32, device="cuda")
    bits = torch.zeros(round_up(N, 32) // 32, dtype=torch.int32, device="cuda")
    sb.saps_mask(ctx, t, p, bits)
    sb.saps_round_pack(ctx, dx, dg, w.lr, pairs, t, p, vals, idx, count)
    torch.cuda.synchronize()
    assert sb.saps_status(ctx) == 0
    sb.saps_destroy(ctx)

    # -- element by element on the sampled rows --
    local = {r: i for i, r in enumerate(rows)}
    sub_pairs = [local[int(pairs[r])] for r in rows]
    m = oracle.gossip_round(x_s, g_s, w.lr, sub_pairs, w.seed, t, p)
    c = int(count[0])
    assert c == int(m.sum(dtype=np.int64))
    if golden is not None:
        assert c == golden
    assert_bits_equal(dx[rows, :N].cpu().numpy(), x_s, f"sampled rows {rows}")
    kept = np.nonzero(m)[0]
    assert (idx[:c].cpu().numpy().view(np.uint32) == kept.astype(np.uint32)).all()

    # -- properties on every row, on the device --
    shifts = torch.arange(32, device="cuda", dtype=torch.int32)
    mdev = ((bits[:, None] >> shifts[None, :]) & 1).bool().reshape(-1)[:N]
    assert int(mdev.sum()) == c
    out = dx[:, :N]
    a = a_dev[:, :N]
    peer = torch.as_tensor(np.asarray(pairs), device="cuda", dtype=torch.long)
    assert torch.equal(torch.where(mdev[None, :], a, out), a)                  # unmasked: SGD step only
    assert torch.equal(out[:, mdev], out[peer][:, mdev])                        # peers agree bitwise
    assert torch.equal(out[:, mdev] + out[peer][:, mdev], a[:, mdev] + a[peer][:, mdev])  # pair sums
    assert torch.equal(vals[:, :c], a[:, mdev])                                 # wire buffer = a o m


def test_resnet50_keep_frac_sweep_sampled_rows(sb):
    torch = torch_cuda()
    w = synth.WORKLOADS["resnet50"]
    rng = synth.matching_rng(w.seed)
    for p in w.keep_fracs:
        pairs = synth.random_perfect_matching(w.n, rng)
        rows = {0, int(pairs[0]), 17, int(pairs[17])}
        _sampled_round(sb, torch, w, p, 1, pairs, rows, golden=_golden_count(2, 1, w.N, p))
        torch.cuda.empty_cache()


def test_gpt2s_sampled_rows(sb):
    torch = torch_cuda()
    w = synth.WORKLOADS["gpt2s"]
    B = synth.bandwidth_matrix(w.n, *w.bw_range, seed=w.seed)
    ctx = sb.saps_create(w.n, 16, w.seed)
    pairs = sb.saps_select_peers(ctx, B, 1, w.n)
    sb.saps_destroy(ctx)
    rows = {5, int(pairs[5])}
    _sampled_round(sb, torch, w, 0.01, 1, pairs, rows, golden=_golden_count(0, 1, w.N, 0.01))
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
    sb.saps_destroy(ctx)
    del x, x0
    torch.cuda.empty_cache()
