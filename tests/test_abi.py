"""CPU-side checks of the C-ABI library: it loads, exports what include/saps.h declares,
validates arguments without touching a GPU, and its host-side peer selection agrees with
the oracle and with brute force."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from oracle import peer_selection as ps
from paper_2002_09692_b200 import binding as sb
from paper_2002_09692_b200 import synth
from helpers import all_perfect_matchings, check_involution, golden_records, max_matching_size_dp, parse_int

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "saps.h")).read()
    return sorted(set(re.findall(r"SAPS_API[^;(]*?\b(saps_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared()
    assert len(names) >= 20 and "saps_round" in names and "saps_select_peers" in names
    lib = ctypes.CDLL(str(sb._LIB_PATH))
    for name in names:
        assert hasattr(lib, name), f"{name} declared in saps.h but not exported"
    assert sorted(sb.EXPORTS) == names, "binding and header disagree"


def test_header_is_plain_c():
    # the boundary is a C ABI: the header must compile as C99 without warnings
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    out = subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-x", "c",
                          os.path.join(ROOT, "include", "saps.h")], capture_output=True, text=True)
    assert out.returncode == 0, out.stderr


def test_round_key_and_threshold_golden():
    for rec in golden_records("mask_hash.txt"):
        if rec[0] == "key":
            assert sb.saps_round_key(parse_int(rec[1]), parse_int(rec[2])) == (parse_int(rec[3]), parse_int(rec[4]))
        elif rec[0] == "thr":
            assert sb.saps_threshold(float(rec[1])) == int(rec[2])
    assert sb.saps_threshold(float("nan")) == 0 and sb.saps_threshold(7.0) == 1 << 32
    # the library's host key and the oracle's agree on arbitrary inputs too
    rng = np.random.default_rng(0)
    for _ in range(200):
        seed, t = int(rng.integers(0, 2 ** 63)), int(rng.integers(1, 2 ** 40))
        assert sb.saps_round_key(seed, t) == oracle.round_key(seed, t)


def test_create_validates():
    for n, N, ld in ((0, 10, 10), (65, 10, 10), (4, 0, 0), (4, 1 << 32, 1 << 32), (4, 10, 9)):
        with pytest.raises(sb.SapsError) as e:
            sb.saps_create_ld(n, N, ld, 0)
        assert e.value.status == sb.SAPS_ERR_INVALID
    ctx = sb.saps_create_ld(64, (1 << 32) - 1, 1 << 32, 5)
    sb.saps_destroy(ctx)
    assert sb._lib.saps_destroy(None) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_create(4, 10, 0, None) == sb.SAPS_ERR_INVALID


def test_round_rejects_bad_arguments_before_any_launch():
    # all of these fail on the host; no CUDA call is reached, so this runs without a GPU
    ctx = sb.saps_create(4, 100, 0)
    fake = 0x1000  # never dereferenced
    good = [1, 0, 3, 2]

    def status(**kw):
        a = dict(x=fake, g=fake, lr=0.1, pairs=good, t=1, p=0.5)
        a.update(kw)
        return sb._lib.saps_round(ctx, a["x"], a["g"], a["lr"], sb._pairs(a["pairs"]), a["t"], a["p"], None)

    assert status(x=None) == sb.SAPS_ERR_INVALID
    assert status(t=0) == sb.SAPS_ERR_INVALID
    assert status(p=-0.1) == sb.SAPS_ERR_INVALID
    assert status(p=1.5) == sb.SAPS_ERR_INVALID
    assert status(p=float("nan")) == sb.SAPS_ERR_INVALID
    assert status(g=None, lr=0.1) == sb.SAPS_ERR_INVALID
    assert status(lr=float("nan")) == sb.SAPS_ERR_INVALID
    assert status(pairs=[1, 2, 0, 3]) == sb.SAPS_ERR_PAIRS
    assert status(pairs=[1, 0, 4, 2]) == sb.SAPS_ERR_PAIRS
    assert status(pairs=[-1, 0, 3, 2]) == sb.SAPS_ERR_PAIRS
    assert sb._lib.saps_round(ctx, fake, fake, 0.1, None, 1, 0.5, None) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_pack(ctx, None, 1, 0.5, fake, fake, fake, None) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_pack(ctx, fake, 1, 0.5, None, fake, fake, None) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_pack(ctx, fake, 1, 2.0, fake, fake, fake, None) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_mask(ctx, 0, 0.5, fake, None) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_run_rounds(ctx, fake, fake, 0.1, 1, 3, 0.5, None, None, None, None, None) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_set_update_order(ctx, 2) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_set_update_order(ctx, sb.SAPS_ORDER_GOSSIP_FIRST) == sb.SAPS_OK
    assert sb._lib.saps_unpack_avg(ctx, fake, None, fake, fake, 0.5, None, None) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_unpack_avg(ctx, fake, fake, fake, fake, 0.5, sb._pairs([1, 2, 0, 3]), None) == sb.SAPS_ERR_PAIRS
    assert sb._lib.saps_consensus_distance(ctx, fake, None, None) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_debug_staging_wait(None, 1) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_debug_staging_wait(ctx, 1) == sb.SAPS_OK
    assert sb._lib.saps_debug_staging_wait(ctx, 0) == sb.SAPS_OK
    assert sb._lib.saps_set_staging(ctx, 3) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_set_staging(ctx, -1) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_set_staging(ctx, sb.SAPS_STAGING_BULK) == sb.SAPS_OK
    assert sb._lib.saps_set_host_pipeline(ctx, 0, 7) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_set_host_pipeline(ctx, 0, -1) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_set_host_pipeline(None, 0, 2) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_set_host_pipeline(ctx, 1 << 40, 6) == sb.SAPS_OK
    assert sb._lib.saps_set_host_pipeline(ctx, 0, 0) == sb.SAPS_OK          # 0 = leave as it is
    assert sb._lib.saps_round_host(ctx, fake, fake, 0.1, sb._pairs(good), 1, 0.5, None, fake) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_round_host(ctx, fake, fake, 0.1, sb._pairs(good), 1, 0.5, fake, None) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_set_column_offset(ctx, (1 << 32) - 50) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_set_column_offset(ctx, (1 << 32) - 100) == sb.SAPS_OK
    sb.saps_destroy(ctx)
    for code in range(-7, 1):
        assert sb.saps_strerror(code) not in ("", "unknown status")
    assert sb.saps_strerror(-99) == "unknown status"


def test_selection_round_numbers_stay_inside_the_signed_timestamp_range():
    # round numbers become signed 64-bit timestamps in R; anything that could wrap, or collide
    # with the "never" marker, is refused on the host
    n = 4
    B = np.ones((n, n)) - np.eye(n)
    ctx = sb.saps_create(n, 100, 0)
    out = (ctypes.c_int32 * n)()
    big = sb.SAPS_SELECT_MAX_T
    assert sb._lib.saps_select_peers(ctx, B.ctypes.data, big + 1, out) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_select_peers(ctx, B.ctypes.data, 1 << 63, out) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_select_peers(ctx, B.ctypes.data, (1 << 64) - 1, out) == sb.SAPS_ERR_INVALID
    assert sb.saps_get_select_state(ctx, n)[1] == 0                       # nothing was recorded
    fake = 0x1000
    # the scheduler refuses before it launches anything when a later round would cross the limit
    assert sb._lib.saps_run_rounds(ctx, fake, fake, 0.1, big, 2, 0.5, None, None, B.ctypes.data, None,
                                   None) == sb.SAPS_ERR_INVALID
    R_ok = (ctypes.c_int64 * (n * n))(*([sb.SAPS_NEVER] * (n * n)))
    assert sb._lib.saps_set_select_state(ctx, R_ok, big + 1) == sb.SAPS_ERR_INVALID
    for bad in (-1, big + 1, -(1 << 63)):
        R_bad = (ctypes.c_int64 * (n * n))(*([sb.SAPS_NEVER] * (n * n)))
        R_bad[1] = bad
        assert sb._lib.saps_set_select_state(ctx, R_bad, 5) == sb.SAPS_ERR_INVALID
    assert sb._lib.saps_set_select_state(ctx, R_ok, big - 1) == sb.SAPS_OK
    # the largest allowed round still works and is recorded as it is
    pairs = sb.saps_select_peers(ctx, B, big, n)
    check_involution(pairs)
    R, last = sb.saps_get_select_state(ctx, n)
    assert last == big and R[0][pairs[0]] == big
    sb.saps_destroy(ctx)


def test_pack_capacity_formula():
    ctx = sb.saps_create(32, 14_728_266, 0)
    for p in (0.1, 0.01, 0.001):
        phat = oracle.threshold(p) / 2.0 ** 32
        N = 14_728_266
        want = int(np.ceil(N * phat + 8 * np.sqrt(N * phat * (1 - phat)))) + 64
        want = (want + 31) // 32 * 32
        assert sb.saps_pack_capacity(ctx, p) == want
        count = int(oracle.mask(0, 1, p, N).sum(dtype=np.int64))
        assert count <= want
    assert sb.saps_pack_capacity(ctx, 1.0) == 14_728_266
    assert sb.saps_pack_capacity(ctx, 0.0) == 64
    assert sb.saps_pack_capacity(ctx, float("nan")) == 0
    sb.saps_set_pack_capacity(ctx, 1000)
    assert sb.saps_pack_capacity(ctx, 0.5) == 1000
    sb.saps_set_pack_capacity(ctx, 0)
    assert sb.saps_pack_capacity(ctx, 1.0) == 14_728_266
    sb.saps_destroy(ctx)


# ---- host-side peer selection (Algorithm 3) against the oracle and brute force -------------

def _candidate_edges(B, R, t, b_thres, t_thres):
    E, mode = ps.candidate_edges(B, R, t, b_thres, t_thres)
    return E, mode


@pytest.mark.parametrize("n", [4, 6, 8])
def test_select_peers_agrees_with_brute_force(n):
    matchings = list(all_perfect_matchings(n))
    for trial in range(20):
        B = synth.bandwidth_matrix(n, 1.0, 100.0, seed=50 * n + trial)
        ctx = sb.saps_create(n, 16, trial)
        b_thres = ps.default_b_thres(B)
        t_thres = ps.default_t_thres(n)
        if trial % 2:
            b_thres = 40.0 + trial
            sb.saps_set_select_params(ctx, b_thres, 3)
            t_thres = 3
        R = ps.new_timestamps(n)                  # the oracle's copy of the state
        for t in range(1, 14):
            E, mode = _candidate_edges(B, R, t, b_thres, t_thres)
            pairs = sb.saps_select_peers(ctx, B, t, n)
            check_involution(pairs)
            assert all(pairs[i] != i for i in range(n))
            chosen = sum(1 for i in range(n) if pairs[i] > i and E[i, pairs[i]])
            best = max(sum(1 for (a, b) in m if E[a, b]) for m in matchings)
            assert chosen == best, (trial, t, mode)
            # the oracle finds a matching of the same quality from the same state
            _, info = ps.generate_gossip_matrix(B, R, t, b_thres, t_thres)
            assert len(info["match"]) == chosen
            ps.record_round(R, pairs, t)          # both sides continue from the library's choice
            libR, last = sb.saps_get_select_state(ctx, n)
            assert last == t
            want = [[ps.NEVER if v == ps.NEVER else int(v) for v in row] for row in R]
            assert [[sb.SAPS_NEVER if v == sb.SAPS_NEVER else v for v in row] for row in libR] == want
        sb.saps_destroy(ctx)


@pytest.mark.parametrize("n", [4, 6, 8])
def test_select_peers_finds_planted_unique_optimum(n):
    rng = np.random.default_rng(n)
    for trial in range(8):
        perm = rng.permutation(n)
        planted = {(min(perm[a], perm[a + 1]), max(perm[a], perm[a + 1])) for a in range(0, n, 2)}
        B = synth.bandwidth_matrix(n, 1.0, 10.0, seed=trial)
        for i, j in planted:
            B[i, j] = B[j, i] = 60.0
        ctx = sb.saps_create(n, 16, trial)
        sb.saps_set_select_params(ctx, 20.0, 5)
        sb.saps_set_select_state(ctx, [[10 ** 6] * n for _ in range(n)], 10 ** 6)   # all recent
        pairs = sb.saps_select_peers(ctx, B, 10 ** 6, n)
        assert {(i, pairs[i]) for i in range(n) if pairs[i] > i} == planted
        sb.saps_destroy(ctx)


@pytest.mark.parametrize("n", [10, 14, 16, 32, 64])
def test_select_peers_matching_size_against_independent_matchers(n):
    # bandwidth mode on a sparse B*: compare the number of B* pairs with the subset DP (small n)
    # and with the oracle's blossom (all n)
    rng = np.random.default_rng(n)
    for trial in range(6):
        B = synth.bandwidth_matrix(n, 1.0, 100.0, seed=900 + trial)
        b_thres = float(rng.choice([80.0, 90.0, 95.0]))
        ctx = sb.saps_create(n, 16, trial)
        sb.saps_set_select_params(ctx, b_thres, 4)
        sb.saps_set_select_state(ctx, [[500] * n for _ in range(n)], 500)
        R = np.full((n, n), 500, dtype=np.int64)
        E, mode = _candidate_edges(B, R, 500, b_thres, 4)
        assert mode == "bandwidth"
        pairs = sb.saps_select_peers(ctx, B, 500, n)
        check_involution(pairs)
        assert all(pairs[i] != i for i in range(n))
        chosen = sum(1 for i in range(n) if pairs[i] > i and E[i, pairs[i]])
        assert chosen == len(ps.maximum_matching(E, rng.permutation(n)))
        if n <= 16:
            assert chosen == max_matching_size_dp(E.tolist())
        sb.saps_destroy(ctx)


def test_select_peers_schedule_invariants():
    n = 32
    B = synth.bandwidth_matrix(n, 1.0, 100.0, seed=1)
    ctx = sb.saps_create(n, 16, 1)
    b_thres, t_thres = ps.default_b_thres(B), ps.default_t_thres(n)
    R = ps.new_timestamps(n)
    S = ps.symmetrise(B)
    connected_at, seen = [], set()
    for t in range(1, 101):
        label = ps.components(ps.recent_graph(R, t, t_thres))
        pairs = sb.saps_select_peers(ctx, B, t, n)
        check_involution(pairs)
        assert all(pairs[i] != i for i in range(n))
        seen.add(tuple(pairs))
        if max(label) == 0:
            connected_at.append(t)
        else:
            # merge mode: at least one pair joins two components, and as many as possible do
            E, _ = ps.candidate_edges(B, R, t, b_thres, t_thres)
            cross = sum(1 for i in range(n) if pairs[i] > i and label[i] != label[pairs[i]])
            assert cross == len(ps.maximum_matching(E)) >= 1
        ps.record_round(R, pairs, t)
    later = [t for t in connected_at if t > 2 * t_thres]
    assert later and np.diff([2 * t_thres] + later + [100]).max() <= t_thres
    assert len(seen) > 50                      # the matching changes from round to round
    # bandwidth mode prefers fast links: mean chosen bandwidth beats a random matching's mean
    sb.saps_destroy(ctx)


def test_select_peers_is_a_pure_function_of_seed_t_and_state():
    n = 16
    B = synth.bandwidth_matrix(n, 1.0, 100.0, seed=3)
    a, b = sb.saps_create(n, 8, 7), sb.saps_create(n, 999, 7)
    log_a = [sb.saps_select_peers(a, B, t, n) for t in range(1, 30)]
    log_b = [sb.saps_select_peers(b, B, t, n) for t in range(1, 30)]
    assert log_a == log_b
    # checkpoint / resume reproduces the continuation
    R, last = sb.saps_get_select_state(a, n)
    cont = [sb.saps_select_peers(a, B, t, n) for t in range(30, 40)]
    c = sb.saps_create(n, 8, 7)
    sb.saps_set_select_state(c, R, last)
    assert [sb.saps_select_peers(c, B, t, n) for t in range(30, 40)] == cont
    # reset forgets
    sb.saps_select_reset(a)
    assert sb.saps_select_peers(a, B, 1, n) == log_a[0]
    with pytest.raises(sb.SapsError):
        sb.saps_select_peers(c, B, 5, n)       # t went backwards
    for h in (a, b, c):
        sb.saps_destroy(h)


def test_select_peers_remembers_nothing_wrong_about_an_earlier_matrix():
    # The library keeps what it derived from the last bandwidth matrix (symmetrised links,
    # threshold, link masks) for as long as the caller passes the same matrix and threshold
    # setting.  A context that sees the matrices and settings change from call to call must
    # choose exactly what contexts do that never saw another matrix (same seed, same R history).
    n = 16
    mats = [synth.bandwidth_matrix(n, 1.0, 100.0, seed=s) for s in (1, 2, 3)]
    mats[2][4, 9] = 0.0                                   # an asymmetric, partly missing link
    settings = [(float("nan"), 0), (40.0, 0), (float("inf"), 0)]
    mixed = sb.saps_create(n, 8, 5)
    for t in range(1, 61):
        B = mats[(t * 7) % 3]
        b_thres, t_thres = settings[(t // 3) % 3]
        # control: a fresh context brought to the same state, which has never derived anything
        R, last = sb.saps_get_select_state(mixed, n)
        fresh = sb.saps_create(n, 8, 5)
        sb.saps_set_select_state(fresh, R, last)
        sb.saps_set_select_params(fresh, b_thres, t_thres)
        sb.saps_set_select_params(mixed, b_thres, t_thres)
        want = sb.saps_select_peers(fresh, B, t, n)
        got = sb.saps_select_peers(mixed, B.copy(), t, n)  # another buffer with the same values
        assert got == want, t
        sb.saps_destroy(fresh)
    # an edit in place of the caller's buffer is seen
    B = mats[0].copy()
    sb.saps_set_select_params(mixed, 50.0, 0)
    sb.saps_select_peers(mixed, B, 61, n)
    B[:, :] = 0.0
    assert sb.saps_select_peers(mixed, B, 62, n) == list(range(n))   # no links left: nobody is paired
    sb.saps_destroy(mixed)


def test_select_peers_odd_n_missing_links_and_bad_input():
    ctx = sb.saps_create(5, 8, 0)
    B = synth.bandwidth_matrix(5, 1.0, 100.0, seed=4)
    pairs = sb.saps_select_peers(ctx, B, 1, 5)
    check_involution(pairs)
    assert sum(1 for i in range(5) if pairs[i] == i) == 1
    B[0, 1] = float("nan")
    with pytest.raises(sb.SapsError):
        sb.saps_select_peers(ctx, B, 2, 5)
    sb.saps_destroy(ctx)
    ctx = sb.saps_create(4, 8, 0)
    B = synth.bandwidth_matrix(4, 1.0, 100.0, seed=4)
    B[3, :] = B[:, 3] = 0.0
    pairs = sb.saps_select_peers(ctx, B, 1, 4)
    assert pairs[3] == 3 and sum(1 for i in range(4) if pairs[i] == i) == 2
    # asymmetric input is symmetrised by the minimum
    B2 = synth.bandwidth_matrix(4, 50.0, 100.0, seed=5)
    B2[0, 1] = 1.0          # one direction slow: the link counts as slow
    sb.saps_set_select_params(ctx, 40.0, 5)
    sb.saps_set_select_state(ctx, [[9] * 4 for _ in range(4)], 9)
    pairs = sb.saps_select_peers(ctx, B2, 9, 4)
    assert pairs[0] != 1
    sb.saps_destroy(ctx)


def test_comm_stats_table_1_and_bottleneck_bandwidth():
    # Table 1: a worker moves 2 N/c values per round; Section IV-D: the round is as fast as
    # the slowest chosen link
    n = 4
    B = np.array([[0, 10, 3, 4], [12, 0, 5, 6], [3, 5, 0, 2], [4, 6, 8, 0]], dtype=np.float64)
    ctx = sb.saps_create(n, 100, 0)
    st = sb.saps_comm_stats(ctx, B, [1, 0, 3, 2], 1000, 1e6)
    assert st["values_per_worker"] == 2000 and st["bytes_per_worker"] == 8000
    assert st["bottleneck_bandwidth"] == 2.0          # min(2, 8) on link (2,3); link (0,1) is min(10,12)
    assert st["mean_bandwidth"] == 6.0
    assert st["comm_time_s"] == 32 * 1000 / 2e6
    st = sb.saps_comm_stats(ctx, B, [0, 1, 2, 3], 1000, 1e6)
    assert st["bottleneck_bandwidth"] == 0.0 and st["comm_time_s"] == 0.0
    with pytest.raises(sb.SapsError):
        sb.saps_comm_stats(ctx, B, [1, 1, 3, 2], 10, 1e6)
    sb.saps_destroy(ctx)


def test_adaptive_selection_beats_random_matching_on_bottleneck_bandwidth():
    # the point of Algorithm 3 (Fig. 5): the chosen pairs sit on faster links than random ones
    n = 32
    B = synth.bandwidth_matrix(n, 0.01, 5.0, seed=11)          # U(0, 5] MB/s as in Section IV-D
    ctx = sb.saps_create(n, 100, 11)
    rng = synth.matching_rng(11)
    ours, rand = [], []
    for t in range(1, 201):
        pairs = sb.saps_select_peers(ctx, B, t, n)
        ours.append(sb.saps_comm_stats(ctx, B, pairs, 1, 8e6)["mean_bandwidth"])
        rand.append(sb.saps_comm_stats(ctx, B, synth.random_perfect_matching(n, rng), 1, 8e6)["mean_bandwidth"])
    sb.saps_destroy(ctx)
    assert np.mean(ours) > 1.25 * np.mean(rand)


@pytest.mark.parametrize("n", [4, 6, 8])
def test_select_peers_bottleneck_mode_against_brute_force(n):
    # b_thres = +inf: the chosen matching's slowest link is the best any perfect matching can do
    for trial in range(12):
        B = synth.bandwidth_matrix(n, 0.01, 5.0, seed=700 + 10 * n + trial)
        S = ps.symmetrise(B)
        best = max(min(S[a, b] for a, b in m) for m in all_perfect_matchings(n))
        ctx = sb.saps_create(n, 16, trial)
        sb.saps_set_select_params(ctx, float("inf"), 4)
        sb.saps_set_select_state(ctx, [[90] * n for _ in range(n)], 90)      # bandwidth mode
        pairs = sb.saps_select_peers(ctx, B, 90, n)
        check_involution(pairs)
        st = sb.saps_comm_stats(ctx, B, pairs, 1, 8e6)
        assert st["bottleneck_bandwidth"] == best == ps.bottleneck_threshold(B)
        sb.saps_destroy(ctx)


def test_select_peers_bottleneck_mode_at_32_workers_matches_the_oracle():
    n = 32
    for trial in range(3):
        B = synth.bandwidth_matrix(n, 0.01, 5.0, seed=40 + trial)
        ctx = sb.saps_create(n, 16, trial)
        sb.saps_set_select_params(ctx, float("inf"), 0)
        sb.saps_set_select_state(ctx, [[7] * n for _ in range(n)], 7)
        pairs = sb.saps_select_peers(ctx, B, 7, n)
        check_involution(pairs)
        assert all(pairs[i] != i for i in range(n))
        st = sb.saps_comm_stats(ctx, B, pairs, 1, 8e6)
        assert st["bottleneck_bandwidth"] == ps.bottleneck_threshold(B)
        sb.saps_destroy(ctx)


def test_bandwidth_study_orders_the_topologies():
    # Section IV-D, Fig. 5: adaptive selection uses faster links than random matching or a ring
    from paper_2002_09692_b200 import bandwidth_study
    r = bandwidth_study.study(16, 8, 30, 1e-3, 5.0)
    assert r["adaptive_bottleneck"]["slowest_link_mean"] > r["adaptive_median"]["slowest_link_mean"]
    assert r["adaptive_median"]["slowest_link_mean"] > 2 * r["random_matching"]["slowest_link_mean"]
    assert r["adaptive_median"]["mean_link_mean"] > r["random_matching"]["mean_link_mean"]
    assert r["random_matching"]["slowest_link_mean"] > r["ring"]["slowest_link_mean"]
