"""Pins for the oracle's peer selection (Algorithm 3) and its blossom matcher."""
import itertools

import numpy as np
import pytest
from scipy.sparse import csr_matrix
from scipy.sparse.csgraph import maximum_bipartite_matching

from oracle import peer_selection as ps
from paper_2002_09692_b200 import synth
from helpers import (all_perfect_matchings, check_involution, check_matching,
                     max_matching_size_dp)


def _random_graph(n, density, rng):
    E = np.zeros((n, n), dtype=bool)
    for i in range(n):
        for j in range(i + 1, n):
            if rng.random() < density:
                E[i, j] = E[j, i] = True
    return E


def _graph(n, edges):
    E = np.zeros((n, n), dtype=bool)
    for i, j in edges:
        E[i, j] = E[j, i] = True
    return E


# ---- the matcher --------------------------------------------------------------

def test_textbook_graphs():
    c5 = _graph(5, [(i, (i + 1) % 5) for i in range(5)])
    assert len(ps.maximum_matching(c5)) == 2
    petersen = _graph(10, [(i, (i + 1) % 5) for i in range(5)] + [(i, i + 5) for i in range(5)]
                      + [(5 + i, 5 + (i + 2) % 5) for i in range(5)])
    assert len(ps.maximum_matching(petersen)) == 5
    star = _graph(7, [(0, i) for i in range(1, 7)])
    assert len(ps.maximum_matching(star)) == 1
    # two triangles joined by a bridge: needs a blossom to see the perfect matching
    tri2 = _graph(6, [(0, 1), (1, 2), (2, 0), (2, 3), (3, 4), (4, 5), (5, 3)])
    assert len(ps.maximum_matching(tri2)) == 3
    # a triangle hanging off a path, started from the far end
    flower = _graph(6, [(0, 1), (1, 2), (2, 3), (3, 4), (4, 2), (4, 5)])
    for order in itertools.permutations(range(6)):
        assert len(ps.maximum_matching(flower, order)) == 3
    for n in (1, 2, 3, 8, 9):
        K = ~np.eye(n, dtype=bool)
        assert len(ps.maximum_matching(K)) == n // 2
    assert ps.maximum_matching(np.zeros((4, 4), dtype=bool)) == []


@pytest.mark.parametrize("n", [4, 5, 6, 7, 8, 10, 12, 14])
def test_matcher_against_subset_dp(n):
    rng = np.random.default_rng(n)
    for trial in range(40):
        E = _random_graph(n, rng.choice([0.15, 0.3, 0.5, 0.8]), rng)
        order = rng.permutation(n)
        match = ps.maximum_matching(E, order)
        check_matching(E, match)
        assert len(match) == max_matching_size_dp(E.tolist()), (n, trial)


def test_matcher_against_subset_dp_sparse_16():
    rng = np.random.default_rng(160)
    for trial in range(6):
        E = _random_graph(16, 0.12, rng)
        match = ps.maximum_matching(E, rng.permutation(16))
        check_matching(E, match)
        assert len(match) == max_matching_size_dp(E.tolist())


@pytest.mark.parametrize("n", [32, 64])
def test_matcher_on_bipartite_graphs_against_hopcroft_karp(n):
    # a bipartite graph is a special case where a library routine gives the optimum
    rng = np.random.default_rng(n + 1)
    h = n // 2
    for density in (0.03, 0.08, 0.3):
        Bi = rng.random((h, h)) < density
        E = np.zeros((n, n), dtype=bool)
        E[:h, h:] = Bi
        E[h:, :h] = Bi.T
        lib = maximum_bipartite_matching(csr_matrix(Bi), perm_type="column")
        want = int((lib >= 0).sum())
        match = ps.maximum_matching(E, rng.permutation(n))
        check_matching(E, match)
        assert len(match) == want


def test_matcher_order_changes_the_matching_not_its_size():
    rng = np.random.default_rng(3)
    E = _random_graph(12, 0.4, rng)
    seen = set()
    for _ in range(30):
        m = ps.maximum_matching(E, rng.permutation(12))
        seen.add(tuple(m))
        assert len(m) == max_matching_size_dp(E.tolist())
    assert len(seen) > 1


# ---- Algorithm 3 --------------------------------------------------------------

def test_symmetrise_and_threshold():
    B = np.array([[9, 5, 1], [7, 9, 4], [3, 2, 9]], dtype=float)
    S = ps.symmetrise(B)
    assert (S == np.array([[0, 5, 1], [5, 0, 2], [1, 2, 0]])).all()
    Bs = ps.connected_graph(B, 2.0)
    assert (Bs == np.array([[0, 1, 0], [1, 0, 1], [0, 1, 0]], dtype=bool)).all()
    assert ps.default_b_thres(B) == 2.0
    assert ps.default_t_thres(32) == 10 and ps.default_t_thres(4) == 4 and ps.default_t_thres(2) == 2


def test_generate_W_is_doubly_stochastic():
    pairs = [1, 0, 3, 2, 4]
    W = ps.generate_W(pairs)
    assert np.allclose(W.sum(axis=0), 1) and np.allclose(W.sum(axis=1), 1)
    assert (W == W.T).all()
    assert W[0, 0] == W[0, 1] == 0.5 and W[4, 4] == 1.0
    assert ((W != 0).sum(axis=1)[:4] == 2).all()


def test_recent_graph_window():
    R = ps.new_timestamps(3)
    assert not ps.recent_graph(R, 1, 10).any()          # "never" is not recent, even at t = 1
    R[0, 1] = R[1, 0] = 5
    assert ps.recent_graph(R, 14, 10)[0, 1]             # 5 > 14 - 10
    assert not ps.recent_graph(R, 15, 10)[0, 1]         # 5 > 15 - 10 fails
    assert ps.components(ps.recent_graph(R, 14, 10)) == [0, 0, 1]


@pytest.mark.parametrize("n", [4, 6, 8])
def test_selection_agrees_with_brute_force_over_all_perfect_matchings(n):
    # Among all (n-1)!! perfect matchings, the selected one uses as many candidate edges
    # (B* edges, or cross-component edges) as any.
    rng = np.random.default_rng(100 + n)
    matchings = list(all_perfect_matchings(n))
    assert len(matchings) == {4: 3, 6: 15, 8: 105}[n]
    for trial in range(25):
        B = synth.bandwidth_matrix(n, 1.0, 100.0, seed=1000 * n + trial)
        R = ps.new_timestamps(n)
        b_thres = ps.default_b_thres(B) if trial % 2 else float(rng.uniform(20, 90))
        t_thres = ps.default_t_thres(n)
        for t in range(1, 12):
            pairs, info = ps.generate_gossip_matrix(B, R, t, b_thres, t_thres,
                                                    rng.permutation(n), rng.permutation(n))
            check_involution(pairs)
            assert all(pairs[i] != i for i in range(n))       # every worker is matched
            E = info["E"]
            chosen = sum(1 for i in range(n) if pairs[i] > i and E[i, pairs[i]])
            best = max(sum(1 for (a, b) in m if E[a, b]) for m in matchings)
            assert chosen == best == len(info["match"])
            ps.record_round(R, pairs, t)


@pytest.mark.parametrize("n", [4, 6, 8])
def test_planted_unique_optimum_is_found(n):
    # one perfect matching above the threshold, every other link below it: the answer is unique
    rng = np.random.default_rng(n)
    for trial in range(10):
        perm = rng.permutation(n)
        planted = {(min(perm[a], perm[a + 1]), max(perm[a], perm[a + 1])) for a in range(0, n, 2)}
        B = synth.bandwidth_matrix(n, 1.0, 10.0, seed=trial)
        for i, j in planted:
            B[i, j] = B[j, i] = 50.0 + trial
        R = np.full((n, n), 10**6, dtype=np.int64)            # everything recent: bandwidth mode
        pairs, info = ps.generate_gossip_matrix(B, R, 10**6, 20.0, 5, rng.permutation(n))
        assert info["mode"] == "bandwidth"
        assert {(i, pairs[i]) for i in range(n) if pairs[i] > i} == planted


def test_first_round_is_merge_mode_on_all_links():
    n = 8
    B = synth.bandwidth_matrix(n, 1.0, 100.0, seed=0)
    R = ps.new_timestamps(n)
    pairs, info = ps.generate_gossip_matrix(B, R, 1, 50.0, 6)
    assert info["mode"] == "merge"
    assert info["E"].sum() == n * (n - 1)                      # all singletons: every link crosses
    assert len(info["match"]) == n // 2 and info["match2"] == []


def test_second_stage_ignores_bandwidth():
    # B* is a star: the first matching has one edge, the rest is paired regardless of speed
    n = 6
    B = np.full((n, n), 1.0)
    B[0, :] = B[:, 0] = 90.0
    R = np.full((n, n), 100, dtype=np.int64)
    pairs, info = ps.generate_gossip_matrix(B, R, 100, 50.0, 5)
    assert info["mode"] == "bandwidth" and len(info["match"]) == 1 and len(info["match2"]) == 2
    check_involution(pairs)
    assert all(pairs[i] != i for i in range(n))


def test_missing_links_and_odd_n_leave_identity_rows():
    n = 5
    B = synth.bandwidth_matrix(n, 1.0, 100.0, seed=4)
    R = ps.new_timestamps(n)
    pairs, _ = ps.generate_gossip_matrix(B, R, 1, 50.0, 6)
    check_involution(pairs)
    assert sum(1 for i in range(n) if pairs[i] == i) == 1
    B2 = synth.bandwidth_matrix(4, 1.0, 100.0, seed=4)
    B2[3, :] = B2[:, 3] = 0.0                                  # worker 3 has left
    pairs, _ = ps.generate_gossip_matrix(B2, ps.new_timestamps(4), 1, 50.0, 4)
    assert pairs[3] == 3 and sum(1 for i in range(4) if pairs[i] == i) == 2


@pytest.mark.parametrize("n", [8, 32])
def test_recent_edges_stay_connected(n):
    # Section II-C: the edges that have a chance to be chosen must form a connected graph.
    # After the warm-up the recent graph is connected at least once in every window of
    # T_thres rounds, and whenever it is not, every first-stage pair joins two components.
    rng = np.random.default_rng(n)
    B = synth.bandwidth_matrix(n, 1.0, 100.0, seed=n)
    b_thres, t_thres = ps.default_b_thres(B), ps.default_t_thres(n)
    R = ps.new_timestamps(n)
    connected_at = []
    modes = []
    for t in range(1, 8 * t_thres + 1):
        Q = ps.recent_graph(R, t, t_thres)
        label = ps.components(Q)
        pairs, info = ps.generate_gossip_matrix(B, R, t, b_thres, t_thres,
                                                rng.permutation(n), rng.permutation(n))
        check_involution(pairs)
        assert all(pairs[i] != i for i in range(n))
        modes.append(info["mode"])
        if max(label) == 0:
            connected_at.append(t)
            assert info["mode"] == "bandwidth"
            for i, j in info["match"]:
                assert ps.symmetrise(B)[i, j] >= b_thres
        else:
            assert info["mode"] == "merge"
            for i, j in info["match"]:
                assert label[i] != label[j]
        ps.record_round(R, pairs, t)
    assert "bandwidth" in modes and "merge" in modes
    warm = 2 * t_thres
    later = [t for t in connected_at if t > warm]
    assert later
    gaps = np.diff([warm] + later + [8 * t_thres])
    assert gaps.max() <= t_thres


@pytest.mark.parametrize("n", [4, 6, 8])
def test_bottleneck_threshold_against_brute_force(n):
    # max over all perfect matchings of the slowest chosen link
    for trial in range(15):
        B = synth.bandwidth_matrix(n, 0.01, 5.0, seed=300 + 10 * n + trial)
        S = ps.symmetrise(B)
        best = max(min(S[a, b] for a, b in m) for m in all_perfect_matchings(n))
        assert ps.bottleneck_threshold(B) == best
        R = np.full((n, n), 50, dtype=np.int64)
        pairs, info = ps.generate_gossip_matrix(B, R, 50, float("inf"), 5)
        assert info["mode"] == "bandwidth" and len(info["match"]) == n // 2
        assert min(S[i, pairs[i]] for i in range(n)) == best


def test_bottleneck_threshold_with_missing_links_and_odd_n():
    B = synth.bandwidth_matrix(5, 1.0, 9.0, seed=2)
    S = ps.symmetrise(B)
    theta = ps.bottleneck_threshold(B)
    assert len(ps.maximum_matching(S >= theta)) == 2
    bigger = [v for v in np.unique(S) if v > theta]
    assert all(len(ps.maximum_matching(S >= v)) < 2 for v in bigger)
    assert ps.bottleneck_threshold(np.zeros((4, 4))) == 0.0


def test_record_round_stamps_the_round():
    # the timestamp matrix records the exchange of round t (Section II-C): an edge used in
    # round t stays "recently connected" for exactly T_thres rounds
    R = ps.new_timestamps(4)
    ps.record_round(R, [1, 0, 3, 2], 7)
    assert R[0, 1] == R[1, 0] == R[2, 3] == R[3, 2] == 7
    assert R[0, 2] == ps.NEVER and R[0, 0] == ps.NEVER
    T = 5
    assert ps.recent_graph(R, 7 + T - 1, T)[0, 1] and not ps.recent_graph(R, 7 + T, T)[0, 1]
    ps.record_round(R, [0, 2, 1, 3], 9)                  # workers 0 and 3 sit this round out
    assert R[1, 2] == R[2, 1] == 9 and R[0, 1] == 7 and R[0, 0] == ps.NEVER
