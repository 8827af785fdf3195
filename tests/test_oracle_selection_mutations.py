"""The same sharpness check for the peer-selection oracle: plant mistakes in a copy of its
Python source and require at least one pin of tests/test_oracle_peer_selection.py to fail."""
import importlib.util
import os
import signal
import sys

import pytest

import test_oracle_peer_selection as pins
from oracle import peer_selection as real

SRC = real.__file__

PINS = [
    pins.test_textbook_graphs,
    lambda: pins.test_matcher_against_subset_dp(8),
    lambda: pins.test_matcher_against_subset_dp(12),
    pins.test_symmetrise_and_threshold, pins.test_generate_W_is_doubly_stochastic, pins.test_recent_graph_window,
    pins.test_record_round_stamps_the_round,
    lambda: pins.test_selection_agrees_with_brute_force_over_all_perfect_matchings(6),
    lambda: pins.test_planted_unique_optimum_is_found(6),
    pins.test_first_round_is_merge_mode_on_all_links, pins.test_second_stage_ignores_bandwidth,
    pins.test_missing_links_and_odd_n_leave_identity_rows,
    lambda: pins.test_recent_edges_stay_connected(8),
    lambda: pins.test_bottleneck_threshold_against_brute_force(6),
]

MUTATIONS = [
    ("symmetrise by max instead of min", "S = np.minimum(B, B.T).copy()", "S = np.maximum(B, B.T).copy()"),
    ("B* uses a strict threshold", "Bs = (S >= b_thres) & (S > 0.0)", "Bs = (S > b_thres) & (S > 0.0)"),
    ("recent window off by one", "int(R[i, j]) > t - t_thres", "int(R[i, j]) >= t - t_thres"),
    ("never-used links count as recent", "R[i, j] != NEVER and int(R[i, j]) > t - t_thres", "int(R[i, j]) > t - t_thres - (1 << 62)"),
    ("merge mode keeps same-component pairs", "label[i] != label[j] and S[i, j] > 0.0", "S[i, j] > 0.0"),
    ("second stage skipped", "    if 2 * len(match) != n:", "    if False:"),
    ("second stage can re-use matched workers", "i not in taken and j not in taken and S[i, j] > 0.0", "S[i, j] > 0.0"),
    ("blossom lifted the wrong way round", "    if i % 2 == 0:\n        walk = cyc[:i + 1]", "    if i % 2 == 1:\n        walk = cyc[:i + 1]"),
    ("contracted blossom loses its stem", "    mate2[b] = mate[base]", "    mate2[b] = None"),
    ("blossom test mistakes odd tree vertices for even ones", "            elif level[w] % 2 == 1:\n                continue", "            elif level[w] % 2 == 0 and root[v] == root[w]:\n                continue"),
    ("W without the diagonal half", "            W[i, i] = 0.5\n            W[i, j] = 0.5", "            W[i, j] = 0.5"),
    ("timestamps recorded one round late", "            R[i, j] = t\n            R[j, i] = t", "            R[i, j] = t - 1\n            R[j, i] = t - 1"),
    ("bottleneck bisection keeps the lower half", "            lo = mid\n        else:\n            hi = mid - 1", "            hi = mid - 1\n        else:\n            lo = mid"),
]


def _load(source: str, name: str):
    spec = importlib.util.spec_from_loader(name, loader=None)
    mod = importlib.util.module_from_spec(spec)
    mod.__file__ = SRC
    sys.modules[name] = mod          # dataclasses / typing look modules up by name
    exec(compile(source, SRC, "exec"), mod.__dict__)
    return mod


class _TooLong(Exception):
    pass


def _alarm(signum, frame):
    raise _TooLong()


def _failures(mod, monkeypatch, stop_at_first=False) -> int:
    """Number of pins that fail (or crash, or do not come back within a few seconds: a mutated
    matcher may walk in circles) against the module `mod`."""
    monkeypatch.setattr(pins, "ps", mod)
    failed = 0
    old = signal.signal(signal.SIGALRM, _alarm)
    try:
        for pin in PINS:
            signal.setitimer(signal.ITIMER_REAL, 10.0)
            try:
                pin()
            except (AssertionError, StopIteration, KeyError, IndexError, TypeError, RecursionError, _TooLong):
                failed += 1
            finally:
                signal.setitimer(signal.ITIMER_REAL, 0.0)
            if failed and stop_at_first:
                break
    finally:
        signal.signal(signal.SIGALRM, old)
    return failed


def test_unmodified_source_passes_every_pin(monkeypatch):
    assert _failures(_load(open(SRC).read(), "ps_copy"), monkeypatch) == 0


@pytest.mark.parametrize("what,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(what, old, new, monkeypatch):
    source = open(SRC).read()
    assert source.count(old) >= 1, f"mutation target not found: {what}"
    assert _failures(_load(source.replace(old, new, 1), "ps_mutant"), monkeypatch, stop_at_first=True) >= 1, \
        f"no pin noticed: {what}"
