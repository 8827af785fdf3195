"""Shared test helpers: golden-file reader and brute-force matching checkers.

The brute-force routines are deliberately independent of both the oracle's and
the library's matcher: plain enumeration / subset dynamic programming.
"""
from __future__ import annotations

import os
from functools import lru_cache

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def golden_records(name):
    """Yield whitespace-split records of a golden text file, comments skipped."""
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if line:
                yield line.split()


def parse_int(s):
    return int(s, 0)


def all_perfect_matchings(n):
    """Every perfect matching of the complete graph on n (even) vertices: (n-1)!! of them."""
    def rec(free):
        if not free:
            yield []
            return
        a = free[0]
        for b in free[1:]:
            rest = [v for v in free if v != a and v != b]
            for m in rec(rest):
                yield [(a, b)] + m
    yield from rec(list(range(n)))


def max_matching_size_dp(E):
    """Maximum matching size by dynamic programming over vertex subsets (n <= ~18)."""
    n = len(E)
    nbr = [sum(1 << w for w in range(n) if w != v and (E[v][w] or E[w][v])) for v in range(n)]

    @lru_cache(maxsize=None)
    def best(mask):
        if mask == 0:
            return 0
        v = (mask & -mask).bit_length() - 1
        rest = mask & ~(1 << v)
        r = best(rest)                      # v stays unmatched
        cand = rest & nbr[v]
        while cand:
            w = (cand & -cand).bit_length() - 1
            cand &= cand - 1
            r = max(r, 1 + best(rest & ~(1 << w)))
        return r

    return best((1 << n) - 1)


def check_matching(E, match):
    """match is a set of vertex-disjoint edges of E."""
    seen = set()
    for i, j in match:
        assert i != j and (E[i][j] or E[j][i]), f"({i},{j}) is not an edge"
        assert i not in seen and j not in seen, "vertex used twice"
        seen.update((i, j))


def check_involution(pairs):
    n = len(pairs)
    for i in range(n):
        j = int(pairs[i])
        assert 0 <= j < n and int(pairs[j]) == i, f"pairs[{i}]={j} breaks the involution"
