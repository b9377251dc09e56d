"""The threshold bisection against a synthetic monotone density curve (no GPU)."""
import math

from paper_2609_20971_b200.calibrate import bisect_alpha


def test_bisection_hits_a_monotone_curve():
    calls = []

    def density(ab, ar):                       # non-increasing in both thresholds, floor at 2 % (forced blocks)
        calls.append((ab, ar))
        return 0.02 + 0.98 * math.exp(-6.0 * ab - 2.0 * ar)
    for target in (0.03, 0.05, 0.10, 0.15):
        ab, ar, d = bisect_alpha(density, target, ratio=0.18 / 0.22, tol=1e-5, iters=40)
        assert abs(d - target) < 1e-4 and abs(ar - ab * 0.18 / 0.22) < 1e-12
    assert len(calls) < 4 * 45


def test_targets_outside_the_reachable_range_clamp():
    def density(ab, ar):
        return 0.02 + 0.5 * (1 - ab)
    assert bisect_alpha(density, 0.9)[0] == 1e-4          # loosest thresholds
    assert bisect_alpha(density, 0.001)[0] == 1.0         # tightest thresholds
