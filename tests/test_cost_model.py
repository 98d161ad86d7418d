"""The latency cost of Sec. 4.3 (C = T_router N_steps + T_high N_high + T_low N_low) as a host function, pinned by
the numbers the paper prints in App. "Latency calibration" and by closed forms."""
import os

import pytest

from paper_2602_02711_b200 import cost

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "latency_coefficients.txt")


def rows():
    out = {"coef": [], "speedup": {}, "w3": None}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        if f[0] == "projected_w3":
            out["w3"] = (float(f[1]), float(f[2]))
        elif f[0] == "speedup":
            out["speedup"][f[1]] = float(f[2])
        else:
            out["coef"].append((f[0], f[1], float(f[2]), float(f[3]), float(f[4])))
    return out


def test_projected_three_bit_coefficient_matches_the_printed_value():
    t_w4, printed = rows()["w3"]
    assert round(cost.projected_w3_time(t_w4), 2) == printed


def test_printed_speedups_follow_from_the_printed_coefficients():
    r = rows()
    for bench, model, th, tl, _ in r["coef"]:
        if bench == "WebShop" and model in r["speedup"]:
            assert round(th / tl, 2) == r["speedup"][model]
            # all steps on the low-precision model, no router: relative cost = T_low / T_high
            assert cost.relative_cost_at_budget(0.0, th, tl) == pytest.approx(tl / th)


def test_cost_equation_terms():
    # each term alone, then linearity in the counts
    assert cost.episode_cost(2.0, 5, 0.0, 0, 0.0, 0) == 10.0
    assert cost.episode_cost(0.0, 0, 3.0, 7, 0.0, 0) == 21.0
    assert cost.episode_cost(0.0, 0, 0.0, 0, 0.5, 8) == 4.0
    a = cost.episode_cost(22.81, 30, 12.64, 400, 10.29, 900)
    b = cost.episode_cost(22.81, 60, 12.64, 800, 10.29, 1800)
    assert b == pytest.approx(2 * a)
    assert a == pytest.approx(22.81 * 30 + 12.64 * 400 + 10.29 * 900)


def test_budget_endpoints_and_router_term():
    th, tl, tr = 25.02, 16.77, 19.90
    assert cost.relative_cost_at_budget(1.0, th, tl) == pytest.approx(1.0)
    assert cost.relative_cost_at_budget(0.4, th, tl) == pytest.approx(0.4 + 0.6 * tl / th)
    # a router call per step of 100 tokens adds T_router / (100 T_high)
    with_router = cost.relative_cost_at_budget(0.4, th, tl, t_router=tr, tokens_per_step=100)
    assert with_router == pytest.approx(0.4 + 0.6 * tl / th + tr / (100 * th))
    with pytest.raises(ValueError):
        cost.relative_cost_at_budget(1.2, th, tl)
    with pytest.raises(ValueError):
        cost.episode_cost(-1.0, 1, 1.0, 1, 1.0, 1)
