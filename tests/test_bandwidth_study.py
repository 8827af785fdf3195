"""Host-only checks of the bandwidth study (protocol of Section IV-D: 32 workers, link speeds
drawn uniformly at random, the slowest chosen link per round as the figure of merit).

The two reference topologies have closed forms, which pin the study's bookkeeping: the slowest
of m independent U(lo, hi) links has expectation lo + (hi - lo) / (m + 1).  A ring uses n links,
a perfect matching n / 2.  The adaptive rule has no closed form; it must beat both and its
bottleneck-threshold mode must beat its median-threshold mode.
"""
import math

from paper_2002_09692_b200 import bandwidth_study


def test_ring_and_random_matching_follow_their_closed_forms():
    n, lo, hi, M, T = 32, 1e-3, 5.0, 400, 4
    out = bandwidth_study.study(n, M, T, lo, hi, seed=3)

    def check(key, links, samples):
        want = lo + (hi - lo) / (links + 1)
        sd = (hi - lo) * math.sqrt(links / ((links + 1) ** 2 * (links + 2)))   # of the minimum of `links` uniforms
        got = out[key]["slowest_link_mean"]
        assert abs(got - want) < 5 * sd / math.sqrt(samples), (key, got, want)

    check("ring", n, M)                       # 5/33 MB/s for links on (0, 5]
    check("random_matching", n // 2, M * T)   # 5/17 MB/s
    mid = 0.5 * (lo + hi)
    sd_link = (hi - lo) / math.sqrt(12.0)
    assert abs(out["ring"]["mean_link_mean"] - mid) < 5 * sd_link / math.sqrt(M * n)
    assert abs(out["random_matching"]["mean_link_mean"] - mid) < 5 * sd_link / math.sqrt(M * T * n / 2)
    # the paper's ordering (Fig. 5): adaptive selection keeps the slowest chosen link far above
    # what a random matching or a ring gets
    a, b = out["adaptive_median"]["slowest_link_mean"], out["adaptive_bottleneck"]["slowest_link_mean"]
    assert b > a > 2 * out["random_matching"]["slowest_link_mean"] > 2 * out["ring"]["slowest_link_mean"]
