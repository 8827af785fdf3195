"""Randomised GPU parity sweep: random shapes, strides, alignments, matchings, keep fractions,
update orders and entry points, each compared bit for bit with the CPU oracle."""
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


def _random_pairs(n, rng):
    perm = list(rng.permutation(n))
    singles = int(rng.integers(0, 3)) if n > 2 else 0
    pairs = list(range(n))
    free = perm[singles:]
    for a in range(0, len(free) - 1, 2):
        i, j = int(free[a]), int(free[a + 1])
        pairs[i], pairs[j] = j, i
    return pairs


@pytest.mark.parametrize("case", range(80))
def test_random_case(sb, case):
    torch = torch_cuda()
    rng = np.random.default_rng(1000 + case)
    n = int(rng.choice([1, 2, 3, 4, 7, 8, 16, 31, 32, 64]))
    N = int(rng.choice([rng.integers(1, 70), rng.integers(2000, 2100), rng.integers(4000, 30_000)]))
    ld = int(rng.choice([N, round_up(N, 4), round_up(N, 32), N + int(rng.integers(1, 9))]))
    lead = int(rng.choice([0, 0, 1, 2, 3, 4]))
    p = float(rng.choice([0.0, 1.0, rng.uniform(0.0005, 0.02), rng.uniform(0.05, 0.6)]))
    has_g = bool(rng.integers(0, 2))
    lr = float(rng.choice([0.0, 0.05, 0.5])) if has_g else 0.0
    order = int(rng.integers(0, 2))
    emit = bool(rng.integers(0, 2))
    seed = int(rng.integers(0, 2 ** 63))
    t0 = int(rng.choice([1, 7, 2 ** 32 - 1, 2 ** 40]))
    # cases beyond the first 60 also draw: per-worker destinations for the wire buffer, and the
    # hook that makes the staged form's wait for its copies count as run out (plain accesses then)
    rows_form = case >= 60 and bool(rng.integers(0, 2))
    give_up = case >= 60 and bool(rng.integers(0, 2))
    x = synth.gaussian_matrix(n, N, 1.0, case, 0)
    g = synth.gaussian_matrix(n, N, 0.1, case, 1) if has_g else None
    dx = DeviceMatrix(x, ld, lead)
    dg = DeviceMatrix(g, ld, lead) if has_g else None
    ctx = sb.saps_create_ld(n, N, ld, seed)
    sb.saps_set_update_order(ctx, order)
    sb.saps_debug_staging_wait(ctx, give_up)
    want = x.copy()
    fn = oracle.gossip_round_eq7 if order else oracle.gossip_round
    for t in (t0, t0 + 1, t0 + 2):                       # consecutive rounds exercise the run-ahead
        pairs = _random_pairs(n, rng)
        if emit:
            cap = sb.saps_pack_capacity(ctx, p)
            vals = torch.full((n, max(cap, 1)), 123.0, dtype=torch.float32, device="cuda")
            idx = torch.full((max(cap, 1),), -1, dtype=torch.int32, device="cuda")
            count = torch.full((1,), -1, dtype=torch.int32, device="cuda")
            if rows_form:
                table = torch.tensor([vals.data_ptr() + 4 * vals.shape[1] * i for i in range(n)], dtype=torch.int64,
                                     device="cuda")
                sb.saps_round_pack_rows(ctx, dx.ptr, dg.ptr if has_g else None, lr, pairs, t, p, table, idx, count)
            else:
                sb.saps_round_pack(ctx, dx.ptr, dg.ptr if has_g else None, lr, pairs, t, p, vals, idx, count)
            sent = want.copy()
            if not order:
                oracle.sgd(sent, g, lr)
            m = oracle.mask(seed, t, p, N)
            wv, wi, wc = oracle.pack(sent, m, cap)
            torch.cuda.synchronize()
            assert int(count.cpu().numpy().view(np.uint32)[0]) == wc
            assert (idx.cpu().numpy().view(np.uint32)[:wc] == wi[:wc]).all()
            assert_bits_equal(vals.cpu().numpy()[:, :wc], wv[:, :wc], f"case {case} wire buffer t={t}")
        else:
            sb.saps_round(ctx, dx.ptr, dg.ptr if has_g else None, lr, pairs, t, p)
        fn(want, g, lr, pairs, seed, t, p)
        torch.cuda.synchronize()
        assert_bits_equal(dx.host(), want, f"case {case}: n={n} N={N} ld={ld} lead={lead} p={p} g={has_g} "
                                           f"order={order} emit={emit} t={t}")
    assert sb.saps_status(ctx) in ((0, sb.SAPS_ERR_TIMEOUT) if give_up else (0,))
    assert dx.canaries_intact()
    if has_g:
        assert_bits_equal(dg.host(), g, "gradient untouched")
    sb.saps_destroy(ctx)
