"""Pins of the oracle's router calibration (threshold = (1 - rho) quantile of the calibration scores, Sec. 4.2
"Inference-time calibration") against things other than itself: numpy's own quantile routine, closed forms on
evenly spaced pools, a brute-force order-statistic count, and the budget property the threshold exists for."""
import numpy as np
import pytest

import oracle


def test_matches_numpys_linear_quantile():
    rng = np.random.default_rng(0)
    for n in (1, 2, 3, 17, 64, 1000, 3200):
        x = rng.random(n).astype(np.float32)
        for rho in (0.0, 0.2, 0.4, 0.7, 1.0, 0.123):
            want = np.quantile(x.astype(np.float64), 1.0 - rho)      # numpy's default rule is the linear one
            assert oracle.router_threshold(x, rho) == pytest.approx(want, rel=1e-13, abs=1e-15)


def test_closed_forms_on_an_evenly_spaced_pool():
    x = np.arange(11, dtype=np.float32) / 10.0          # 0.0, 0.1, ..., 1.0 (as float32)
    assert oracle.router_threshold(x, 1.0) == 0.0       # budget 1: everything is high precision
    assert oracle.router_threshold(x, 0.0) == 1.0       # budget 0: only the top score reaches the threshold
    assert oracle.router_threshold(x, 0.5) == float(x[5])
    # between two order statistics: h = 10 * 0.75 = 7.5 -> halfway between x[7] and x[8]
    assert oracle.router_threshold(x, 0.25) == pytest.approx(0.5 * (float(x[7]) + float(x[8])), rel=1e-15)
    # a swapped budget (rho instead of 1 - rho) would give the mirror image
    assert oracle.router_threshold(x, 0.2) == pytest.approx(0.8, rel=1e-6)
    assert oracle.router_threshold(x[::-1].copy(), 0.2) == oracle.router_threshold(x, 0.2)   # order of the pool is irrelevant


def test_order_statistics_by_brute_force_counting():
    rng = np.random.default_rng(1)
    x = rng.standard_normal(200).astype(np.float32)
    x[10:20] = x[5]                                      # ties
    n = len(x)
    for rho in (0.2, 0.4, 0.7):
        h = (n - 1) * (1.0 - rho)
        lo = int(np.floor(h))
        # the element with exactly `lo` elements sorting before it (ties broken by index)
        def kth(k):
            for i in range(n):
                r = sum(1 for j in range(n) if x[j] < x[i] or (x[j] == x[i] and j < i))
                if r == k:
                    return float(x[i])
        a, b = kth(lo), kth(min(lo + 1, n - 1))
        assert oracle.router_threshold(x, rho) == a + (h - lo) * (b - a)


def test_threshold_realises_the_budget_on_the_calibration_pool():
    rng = np.random.default_rng(2)
    x = rng.random(3200).astype(np.float32)              # 64 tasks x 50 steps, the size of the paper's pool
    for rho in (0.2, 0.4, 0.7):
        tau = oracle.router_threshold(x, rho)
        frac_high = oracle.router_mask(x, tau).mean()
        assert abs(frac_high - rho) <= 1.0 / len(x) + 1e-12
    m = oracle.router_mask(np.array([0.1, 0.5, 0.5, 0.9], np.float32), 0.5)
    assert m.tolist() == [0, 1, 1, 1] and m.dtype == np.uint8   # p >= tau, ties go to high precision


def test_bad_arguments():
    with pytest.raises(ValueError):
        oracle.router_threshold(np.zeros(0, np.float32), 0.5)
    with pytest.raises(ValueError):
        oracle.router_threshold(np.ones(3, np.float32), 1.5)
