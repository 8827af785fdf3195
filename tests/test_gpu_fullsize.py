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
