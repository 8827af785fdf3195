"""Pins for the oracle's round (Algorithm 2 with the averaging merge of GenerateW / Eq. 7)."""
import numpy as np
import pytest

import oracle
from oracle import peer_selection as ps
from paper_2002_09692_b200 import synth
from helpers import golden_records


def _inputs(n, N, seed=3, x_std=1.0, g_std=0.01):
    return (synth.gaussian_matrix(n, N, x_std, seed, 0),
            synth.gaussian_matrix(n, N, g_std, seed, 1))


def test_worked_example():
    recs = list(golden_records("worked_example.txt"))
    want_mask = np.array([int(v) for v in next(r for r in recs if r[0] == "mask")[1:]], np.uint8)
    want_rows = {int(r[1]): np.array(r[2:], np.float32) for r in recs if r[0] == "row"}
    want_pack = {int(r[1]): np.array(r[2:], np.float32) for r in recs if r[0] == "pack"}
    n, N = 4, 8
    x = np.array([[8 * i + k for k in range(N)] for i in range(n)], np.float32)
    g = np.array([[i + 1] * N for i in range(n)], np.float32)
    pairs = [1, 0, 3, 2]
    # pack sees the post-SGD model
    a = x.copy()
    oracle.sgd(a, g, 0.5)
    m = oracle.mask(0, 1, 0.5, N)
    assert (m == want_mask).all()
    vals, idx, count = oracle.pack(a, m)
    assert count == 3 and list(idx) == [2, 3, 5]
    for i in range(n):
        assert (vals[i] == want_pack[i]).all()
    m2 = oracle.gossip_round(x, g, 0.5, pairs, 0, 1, 0.5)
    assert (m2 == want_mask).all()
    for i in range(n):
        assert (x[i] == want_rows[i]).all(), i


def test_full_mask_no_gradient_is_dense_product_with_W():
    # keep_frac = 1, no SGD: X' = W X with the doubly stochastic W of GenerateW (Eq. 4 / Eq. 7)
    n, N = 8, 3001
    x, _ = _inputs(n, N)
    pairs = synth.random_perfect_matching(n, synth.matching_rng(5))
    W = ps.generate_W(list(pairs))
    want = W @ x.astype(np.float64)
    oracle.gossip_round(x, None, 0.0, pairs, 1, 1, 1.0)
    err = np.abs(x.astype(np.float64) - want)
    assert (err <= np.abs(want) * 2.0 ** -24 + 1e-45).all()
    # one rounding only: casting the exact product gives the same bits
    assert (want.astype(np.float32) == x).all()


def test_empty_mask_is_axpy():
    # keep_frac = 0: X' = X - lr G, nothing exchanged
    from scipy.linalg.blas import saxpy
    n, N = 4, 5003
    x, g = _inputs(n, N)
    want = saxpy(g.ravel(), x.ravel().copy(), a=-0.1).reshape(n, N)
    x0 = x.copy()
    oracle.gossip_round(x, g, 0.1, [1, 0, 3, 2], 1, 1, 0.0)
    # a BLAS may fuse the multiply-add: that skips the rounding of lr*g (half a unit in the
    # last place of the product) and can move the result by one unit in its last place
    assert (np.abs(x - want) <= 2.0 ** -23 * np.abs(want) + 2.0 ** -24 * np.abs(0.1 * g)).all()
    assert (x == x0 - np.float32(0.1) * g).all()


def test_unmasked_coordinates_untouched_bit_for_bit():
    # the "x o not m" term of Algorithm 2: with no gradient an unkept coordinate keeps its bits
    n, N = 6, 10_007
    x, g = _inputs(n, N)
    x0 = x.copy()
    pairs = [1, 0, 3, 2, 5, 4]
    m = oracle.gossip_round(x, None, 0.0, pairs, 2, 7, 0.1)
    keep = m.astype(bool)
    assert 0 < keep.sum() < N
    assert (x[:, ~keep].view(np.uint32) == x0[:, ~keep].view(np.uint32)).all()
    # with lr = 0 and a gradient present, likewise
    x1 = x0.copy()
    oracle.gossip_round(x1, g, 0.0, pairs, 2, 7, 0.1)
    assert (x1[:, ~keep] == x0[:, ~keep]).all()
    # with a gradient they hold exactly the SGD step
    x2 = x0.copy()
    oracle.gossip_round(x2, g, 0.05, pairs, 2, 7, 0.1)
    assert (x2[:, ~keep] == (x0 - np.float32(0.05) * g)[:, ~keep]).all()


def test_pair_sum_preserved_to_one_rounding():
    # W doubly stochastic: a matched pair's kept coordinates keep their sum, and both get the same bits
    n, N = 8, 20_011
    x, g = _inputs(n, N)
    pairs = synth.random_perfect_matching(n, synth.matching_rng(1))
    a = x - np.float32(0.05) * g
    m = oracle.gossip_round(x, g, 0.05, pairs, 0, 3, 0.3).astype(bool)
    for i in range(n):
        j = int(pairs[i])
        assert (x[i, m].view(np.uint32) == x[j, m].view(np.uint32)).all()
        assert (x[i, m] + x[j, m] == a[i, m] + a[j, m]).all()
        exact = a[i, m].astype(np.float64) + a[j, m].astype(np.float64)
        got = x[i, m].astype(np.float64) + x[j, m].astype(np.float64)
        assert (np.abs(got - exact) <= np.abs(exact) * 2.0 ** -24).all()


def test_column_sums_over_workers_preserved():
    # sum_i x_i[k] is invariant under the exchange (W 1 = 1)
    n, N = 16, 4099
    x, _ = _inputs(n, N)
    s0 = x.astype(np.float64).sum(axis=0)
    pairs = synth.random_perfect_matching(n, synth.matching_rng(2))
    oracle.gossip_round(x, None, 0.0, pairs, 4, 9, 0.5)
    s1 = x.astype(np.float64).sum(axis=0)
    assert np.allclose(s0, s1, rtol=0, atol=n * 2.0 ** -24 * 8)


def test_unmatched_worker_only_takes_its_sgd_step():
    n, N = 5, 1003
    x, g = _inputs(n, N)
    x0 = x.copy()
    pairs = [1, 0, 2, 4, 3]              # worker 2 has no peer
    oracle.gossip_round(x, g, 0.1, pairs, 0, 1, 0.5)
    assert (x[2] == x0[2] - np.float32(0.1) * g[2]).all()


def test_lemma_1_mask_and_gossip_commute():
    # (A o M) W = (A W) o M: average every column first, then select by the mask
    n, N = 8, 6007
    x, g = _inputs(n, N)
    pairs = synth.random_perfect_matching(n, synth.matching_rng(3))
    a = x.copy()
    oracle.sgd(a, g, 0.05)
    everything = a.copy()
    oracle.pair_average(everything, pairs, np.ones(N, np.uint8))
    m = oracle.gossip_round(x, g, 0.05, pairs, 5, 2, 0.2).astype(bool)
    want = np.where(m[None, :], everything, a)
    assert (x.view(np.uint32) == want.view(np.uint32)).all()


@pytest.mark.parametrize("n", [2, 8, 32])
def test_hypercube_consensus(n):
    # keep_frac 1, no gradient, connected schedule: after log2 n rounds every worker holds the mean
    N = 2003
    x, _ = _inputs(n, N, seed=n)
    mean = x.astype(np.float64).mean(axis=0)
    d = n.bit_length() - 1
    for r in range(d):
        oracle.gossip_round(x, None, 0.0, synth.hypercube_pairs(n, r), 0, r + 1, 1.0)
    assert (x.view(np.uint32) == x[0].view(np.uint32)[None, :]).all()
    scale = np.abs(x).max()
    assert np.abs(x[0] - mean).max() <= d * 2.0 ** -24 * max(scale, 4.0)


def test_lemma_2_contraction_factor():
    # Uniformly random perfect matchings: W is a projection, E[W^T W] = E[W] has second
    # eigenvalue (n-2)/(2(n-1)); with the mask the squared consensus distance shrinks by
    # q + p * lambda2 per round in expectation (Lemma 2).
    n, N, p = 32, 250_000, 0.25
    lam2 = (n - 2) / (2.0 * (n - 1))
    phat = oracle.threshold(p) / 2.0 ** 32
    want = (1 - phat) + phat * lam2
    x, _ = _inputs(n, N, seed=8)
    rng = synth.matching_rng(8)

    def dist(x):
        x64 = x.astype(np.float64)
        return ((x64 - x64.mean(axis=0, keepdims=True)) ** 2).sum()

    ratios = []
    d0 = dist(x)
    for t in range(1, 7):
        oracle.gossip_round(x, None, 0.0, synth.random_perfect_matching(n, rng), 8, t, p)
        d1 = dist(x)
        ratios.append(d1 / d0)
        d0 = d1
    assert abs(ratios[0] - want) < 0.01 * want          # iid start: holds for any matching
    assert abs(np.mean(ratios) - want) < 0.01 * want
    # a wrong reading (replace instead of average, or factor 1) would not contract like this
    assert all(r < 1.0 for r in ratios)


def test_pack_definition():
    n, N = 4, 9001
    x, _ = _inputs(n, N)
    m = oracle.mask(3, 2, 0.1, N)
    vals, idx, count = oracle.pack(x, m)
    assert count == int(m.sum()) == len(idx)
    assert (np.diff(idx.astype(np.int64)) > 0).all()
    assert (idx == np.nonzero(m)[0]).all()
    assert (vals == x[:, np.nonzero(m)[0]]).all()
    # a kept coordinate that is exactly zero is still sent
    x[:, idx[0]] = 0.0
    vals2, _, count2 = oracle.pack(x, m)
    assert count2 == count and (vals2[:, 0] == 0).all()
    # capacity clamp: count stays exact, only cap entries are written
    vals3, idx3, count3 = oracle.pack(x, m, cap=10)
    assert count3 == count and (idx3 == idx[:10]).all() and (vals3 == vals2[:, :10]).all()


def test_unfused_wire_path_equals_the_round():
    # SGD -> pack -> swap buffers -> average from the two packed buffers -> scatter == round
    n, N = 6, 7001
    x, g = _inputs(n, N)
    pairs = [3, 2, 1, 0, 5, 4]
    a = x.copy()
    oracle.sgd(a, g, 0.05)
    m = oracle.mask(6, 4, 0.15, N)
    vals, idx, count = oracle.pack(a, m)
    merged = a.copy()
    for i in range(n):
        merged[i, idx] = np.float32(0.5) * (vals[i] + vals[pairs[i]])
    oracle.gossip_round(x, g, 0.05, pairs, 6, 4, 0.15)
    assert (x.view(np.uint32) == merged.view(np.uint32)).all()
    # after the round a worker and its peer would send identical buffers
    v2, _, _ = oracle.pack(x, m)
    for i in range(n):
        assert (v2[i] == v2[pairs[i]]).all()


def test_rejects_bad_pairs():
    x, _ = _inputs(4, 16)
    with pytest.raises(ValueError):
        oracle.gossip_round(x, None, 0.0, [1, 2, 0, 3], 0, 1, 0.5)
    with pytest.raises(ValueError):
        oracle.gossip_round(x, None, 0.0, [1, 0, 4, 2], 0, 1, 0.5)


# ---- Eq. 7 ordering, receiving side, consensus distance ---------------------------------------

def test_eq7_order_is_the_matrix_form():
    # X' = X o not M + (X o M) W - gamma G, evaluated densely in double precision
    n, N, lr, p = 8, 4001, 0.05, 0.3
    x, g = _inputs(n, N, seed=12)
    pairs = synth.random_perfect_matching(n, synth.matching_rng(12))
    W = ps.generate_W(list(pairs))
    m = oracle.mask(4, 6, p, N).astype(np.float64)
    X, G = x.astype(np.float64), g.astype(np.float64)
    want = X * (1 - m)[None, :] + W @ (X * m[None, :]) - np.float64(np.float32(lr)) * G
    got = x.copy()
    m2 = oracle.gossip_round_eq7(got, g, lr, pairs, 4, 6, p)
    assert (m2 == m).all()
    # three fp32 roundings (sum, product lr*g, difference) against the exact value
    tol = 2.0 ** -23 * (np.abs(want) + np.abs(X) + np.abs(lr * G)) + 1e-45
    assert (np.abs(got.astype(np.float64) - want) <= tol).all()
    # and it is NOT the Algorithm 2 order: there the gradient step is averaged too
    alg2 = x.copy()
    oracle.gossip_round(alg2, g, lr, pairs, 4, 6, p)
    kept = m.astype(bool)
    assert (alg2[:, ~kept] == got[:, ~kept]).all()
    assert not np.array_equal(alg2[:, kept], got[:, kept])
    diff = got.astype(np.float64) - alg2.astype(np.float64)
    # difference on kept coordinates = -lr (g_i - (g_i + g_j)/2) up to rounding
    want_diff = -lr * (G - W @ G)
    assert np.allclose(diff[:, kept], want_diff[:, kept], rtol=0, atol=1e-6)


def test_eq7_order_reductions():
    n, N = 6, 3001
    x, g = _inputs(n, N, seed=13)
    pairs = [1, 0, 3, 2, 5, 4]
    # without a gradient the two orders coincide bit for bit
    a, b = x.copy(), x.copy()
    oracle.gossip_round(a, None, 0.0, pairs, 1, 2, 0.4)
    oracle.gossip_round_eq7(b, None, 0.0, pairs, 1, 2, 0.4)
    assert (a.view(np.uint32) == b.view(np.uint32)).all()
    # empty mask: plain SGD in both orders
    a, b = x.copy(), x.copy()
    oracle.gossip_round(a, g, 0.1, pairs, 1, 2, 0.0)
    oracle.gossip_round_eq7(b, g, 0.1, pairs, 1, 2, 0.0)
    assert (a == b).all() and (a == x - np.float32(0.1) * g).all()
    # column sums move by exactly the summed gradient step (W is doubly stochastic)
    c = x.copy()
    oracle.gossip_round_eq7(c, g, 0.1, pairs, 1, 2, 0.5)
    want = x.astype(np.float64).sum(0) - 0.1 * g.astype(np.float64).sum(0)
    assert np.allclose(c.astype(np.float64).sum(0), want, rtol=0, atol=1e-5)


def test_unpack_avg_is_the_receiving_side_of_the_round():
    n, N = 6, 7001
    x, g = _inputs(n, N, seed=14)
    pairs = [3, 2, 1, 0, 5, 4]
    a = x.copy()
    oracle.sgd(a, g, 0.05)
    m = oracle.mask(6, 4, 0.15, N)
    vals, idx, count = oracle.pack(a, m)
    recv = np.ascontiguousarray(vals[pairs])             # what each worker gets from its peer
    oracle.unpack_avg(a, recv, idx, count)
    oracle.gossip_round(x, g, 0.05, pairs, 6, 4, 0.15)
    assert (x.view(np.uint32) == a.view(np.uint32)).all()
    # hand-checkable: one worker, two kept columns
    y = np.array([[1.0, 2.0, 3.0, 4.0]], np.float32)
    oracle.unpack_avg(y, np.array([[10.0, 20.0]], np.float32), np.array([1, 3], np.uint32), 2)
    assert (y == np.array([[1.0, 6.0, 3.0, 12.0]], np.float32)).all()
    # count smaller than the buffer: the rest is ignored
    y = np.array([[1.0, 2.0, 3.0, 4.0]], np.float32)
    oracle.unpack_avg(y, np.array([[10.0, 20.0]], np.float32), np.array([1, 3], np.uint32), 1)
    assert (y == np.array([[1.0, 6.0, 3.0, 4.0]], np.float32)).all()


def test_consensus_distance_closed_forms():
    rng = np.random.default_rng(5)
    a = rng.standard_normal(1000).astype(np.float32)
    # identical workers: zero; two opposite workers: 2 sum a^2
    assert oracle.consensus_distance(np.stack([a, a, a])) == 0.0
    assert np.isclose(oracle.consensus_distance(np.stack([a, -a])), 2 * (a.astype(np.float64) ** 2).sum(),
                      rtol=1e-14)
    # n * (population variance over workers), summed over coordinates: a library routine
    x, _ = _inputs(16, 5000, seed=15)
    want = 16 * np.var(x.astype(np.float64), axis=0).sum()
    assert np.isclose(oracle.consensus_distance(x), want, rtol=1e-12)
    # adding the same vector to every worker changes nothing (up to the fp32 rounding of the inputs)
    shifted = (x.astype(np.float64) + 3.0).astype(np.float32)
    assert np.isclose(oracle.consensus_distance(shifted), want, rtol=1e-5)
    # hand-checkable: workers (0, 2) and (4, 6): means 2 and 4, deviations +-2 -> 4 * 4
    assert oracle.consensus_distance(np.array([[0.0, 2.0], [4.0, 6.0]], np.float32)) == 16.0
    # full gossip with a connected schedule drives it to (numerically) zero
    y, _ = _inputs(8, 500, seed=16)
    d0 = oracle.consensus_distance(y)
    for r in range(3):
        oracle.gossip_round(y, None, 0.0, synth.hypercube_pairs(8, r), 0, r + 1, 1.0)
    assert oracle.consensus_distance(y) == 0.0 < d0
