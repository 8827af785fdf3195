"""Pins for the oracle's mask: golden hash values and the Bernoulli law of Eq. 3."""
import math

import numpy as np
import pytest

import oracle
from helpers import golden_records, parse_int


def _records(kind):
    return [r[1:] for r in golden_records("mask_hash.txt") if r[0] == kind]


def test_golden_mix():
    for v, want in _records("mix"):
        assert oracle.mix(parse_int(v)) == parse_int(want)


def test_golden_round_key():
    for seed, t, k0, k1 in _records("key"):
        assert oracle.round_key(parse_int(seed), parse_int(t)) == (parse_int(k0), parse_int(k1))


def test_golden_hash():
    recs = _records("hash")
    assert len(recs) >= 40
    for seed, t, k, want in recs:
        k0, k1 = oracle.round_key(parse_int(seed), parse_int(t))
        assert oracle.hash_k(parse_int(k), k0, k1) == parse_int(want), (seed, t, k)


def test_golden_threshold():
    for p, want in _records("thr"):
        assert oracle.threshold(float(p)) == int(want)
    assert oracle.threshold(-0.5) == 0
    assert oracle.threshold(2.0) == 1 << 32
    assert oracle.threshold(float("nan")) == 0


@pytest.mark.parametrize("rec", _records("count"), ids=lambda r: "-".join(r[:4]))
def test_golden_counts(rec):
    seed, t, N, p, want = rec
    m = oracle.mask(int(seed), int(t), float(p), int(N))
    assert int(m.sum(dtype=np.int64)) == int(want)


def test_golden_first_and_last_columns():
    for seed, t, N, p, *cols in _records("first"):
        idx = np.nonzero(oracle.mask(int(seed), int(t), float(p), int(N)))[0]
        assert list(idx[:len(cols)]) == [int(c) for c in cols]
    for seed, t, N, p, col in _records("last"):
        idx = np.nonzero(oracle.mask(int(seed), int(t), float(p), int(N)))[0]
        assert int(idx[-1]) == int(col)


def test_mask_matches_hash_and_threshold():
    # the mask is exactly "hash below threshold", including both extremes
    N = 5000
    for p in (0.0, 1e-3, 0.37, 1.0):
        m = oracle.mask(9, 4, p, N)
        k0, k1 = oracle.round_key(9, 4)
        thr = oracle.threshold(p)
        for k in range(0, N, 97):
            assert m[k] == (oracle.hash_k(k, k0, k1) < thr)
    assert oracle.mask(3, 3, 1.0, 1000).all()
    assert not oracle.mask(3, 3, 0.0, 1000).any()


def test_hash_is_injective_on_windows():
    # for a fixed key the hash permutes the 32-bit integers, so no two columns collide
    k0, k1 = oracle.round_key(5, 17)
    for start in (0, (1 << 32) - (1 << 18), 0x7FFF0000):
        vals = {oracle.hash_k(start + k, k0, k1) for k in range(1 << 16)}
        assert len(vals) == 1 << 16


@pytest.mark.parametrize("N,p", [(65_536, 0.1), (272_474, 0.01), (1 << 20, 0.25),
                                 (1 << 20, 0.001), (3_000_000, 0.03)])
def test_density_within_binomial_5_sigma(N, p):
    # Eq. 3: each coordinate is kept with probability p, so count ~ Binomial(N, p)
    phat = oracle.threshold(p) / 2.0 ** 32
    sigma = math.sqrt(N * phat * (1 - phat))
    zs = []
    for seed in (0, 1, 2):
        for t in (1, 2, 3, 50, 1 << 33):
            c = int(oracle.mask(seed, t, p, N).sum(dtype=np.int64))
            zs.append((c - N * phat) / sigma)
    assert max(abs(z) for z in zs) < 5.0
    # the z-scores themselves must look standard normal, not all on one side
    assert abs(np.mean(zs)) < 5.0 / math.sqrt(len(zs))


def test_rounds_are_independent():
    # overlap of two rounds' masks ~ Binomial(N, p^2)
    N, p = 1 << 21, 0.1
    phat = oracle.threshold(p) / 2.0 ** 32
    for seed, t in ((0, 1), (0, 2), (7, 100)):
        a = oracle.mask(seed, t, p, N)
        b = oracle.mask(seed, t + 1, p, N)
        c = oracle.mask(seed + 1, t, p, N)
        for other in (b, c):
            ov = int((a & other).sum(dtype=np.int64))
            q = phat * phat
            assert abs(ov - N * q) < 5.0 * math.sqrt(N * q * (1 - q))


def test_neighbouring_columns_are_independent():
    # P(m[k] and m[k+1]) = p^2 : no short-range structure in k
    N, p = 1 << 21, 0.2
    phat = oracle.threshold(p) / 2.0 ** 32
    m = oracle.mask(11, 5, p, N)
    for lag in (1, 2, 4, 32, 1024):
        both = int((m[:-lag] & m[lag:]).sum(dtype=np.int64))
        q = phat * phat
        assert abs(both - (N - lag) * q) < 5.0 * math.sqrt(N * q * (1 - q))


def test_each_column_is_chosen_binomially_over_rounds():
    # over T rounds a column is kept Binomial(T, p) times: mean T p, variance T p (1-p)
    N, T, p = 20_000, 400, 0.1
    phat = oracle.threshold(p) / 2.0 ** 32
    hits = np.zeros(N, dtype=np.int64)
    for t in range(1, T + 1):
        hits += oracle.mask(0, t, p, N)
    assert abs(hits.mean() - T * phat) < 5.0 * math.sqrt(T * phat * (1 - phat) / N)
    var = hits.var()
    assert abs(var / (T * phat * (1 - phat)) - 1.0) < 0.05


def test_traffic_closed_form():
    # Table 1: a worker sends and receives 2 (N/c) T values in T rounds
    N, T, p = 272_474, 100, 0.01
    phat = oracle.threshold(p) / 2.0 ** 32
    total = sum(int(oracle.mask(1, t, p, N).sum(dtype=np.int64)) for t in range(1, T + 1))
    sigma = math.sqrt(T * N * phat * (1 - phat))
    assert abs(2 * total - 2 * T * N * phat) < 2 * 5.0 * sigma


def test_threshold_comparison_is_strict():
    # keep(k) is "hash < threshold": with the threshold set to a column's own hash value that
    # column is dropped, one more and it is kept (floor(keep_frac 2^32) is exact for h / 2^32)
    seed, t = 12, 34
    k0, k1 = oracle.round_key(seed, t)
    for k in (0, 1, 77, 4095, 100_000):
        h = oracle.hash_k(k, k0, k1)
        assert oracle.threshold(h / 2.0 ** 32) == h
        assert oracle.mask(seed, t, h / 2.0 ** 32, k + 1)[k] == 0
        if h + 1 <= 2 ** 32:
            assert oracle.mask(seed, t, (h + 1) / 2.0 ** 32, k + 1)[k] == 1
