"""Bandwidth utilisation of the peer-selection rule (host only; protocol of Section IV-D).

For M random bandwidth matrices (32 workers, link speeds uniform on (0, 5] MB/s) run T rounds of
saps_select_peers and record, per round, the slowest and the mean bandwidth over the chosen
pairs.  Compared with a uniformly random perfect matching per round and with a fixed ring
(every worker talks to both ring neighbours, so its round is as slow as the slowest ring link),
the two topologies the paper plots beside its own.

    python -m paper_2002_09692_b200.bandwidth_study [--matrices 200] [--rounds 100] [--n 32]
"""
from __future__ import annotations

import argparse
import json

import numpy as np

from . import binding as sb
from . import synth


def study(n: int, matrices: int, rounds: int, lo: float, hi: float, seed: int = 0):
    keys = ("adaptive_median", "adaptive_bottleneck", "random_matching", "ring")
    slow = {k: [] for k in keys}
    mean = {k: [] for k in keys}
    rng = synth.matching_rng(seed)
    for m in range(matrices):
        B = synth.bandwidth_matrix(n, lo, hi, seed=seed * 100_003 + m)
        ring = [B[i, (i + 1) % n] for i in range(n)]
        slow["ring"].append(min(ring))
        mean["ring"].append(float(np.mean(ring)))
        for key, b_thres in (("adaptive_median", float("nan")), ("adaptive_bottleneck", float("inf"))):
            ctx = sb.saps_create(n, 1, seed + m)
            sb.saps_set_select_params(ctx, b_thres, 0)
            for t in range(1, rounds + 1):
                st = sb.saps_comm_stats(ctx, B, sb.saps_select_peers(ctx, B, t, n), 1, 8e6)
                slow[key].append(st["bottleneck_bandwidth"])
                mean[key].append(st["mean_bandwidth"])
            sb.saps_destroy(ctx)
        ctx = sb.saps_create(n, 1, 0)
        for t in range(rounds):
            st = sb.saps_comm_stats(ctx, B, synth.random_perfect_matching(n, rng), 1, 8e6)
            slow["random_matching"].append(st["bottleneck_bandwidth"])
            mean["random_matching"].append(st["mean_bandwidth"])
        sb.saps_destroy(ctx)
    return {k: {"slowest_link_mean": float(np.mean(slow[k])), "mean_link_mean": float(np.mean(mean[k]))}
            for k in keys}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--n", type=int, default=32)
    ap.add_argument("--matrices", type=int, default=200)
    ap.add_argument("--rounds", type=int, default=100)
    ap.add_argument("--lo", type=float, default=1e-3)
    ap.add_argument("--hi", type=float, default=5.0)
    a = ap.parse_args()
    out = study(a.n, a.matrices, a.rounds, a.lo, a.hi)
    print(json.dumps({"n": a.n, "matrices": a.matrices, "rounds": a.rounds, "unit": "MB/s", **out}, indent=1))


if __name__ == "__main__":
    main()
