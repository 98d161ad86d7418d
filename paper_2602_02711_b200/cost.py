"""Latency-based cost of a routed episode (Sec. 4.3, the cost inside the reward R = 1[success] - lambda * C):

    C = T_router * N_steps + T_high * N_high_tokens + T_low * N_low_tokens

with per-call router time T_router and per-token times T_high / T_low of the high- and the low-precision
model (App. "Latency calibration": T_prec = 1000 * sum(wall seconds) / sum(completion tokens), in ms per token).
Host arithmetic only; bench.py feeds it the per-token layer times it measures.
"""
from __future__ import annotations


def episode_cost(t_router: float, n_steps: int, t_high: float, n_high_tokens: float, t_low: float,
                 n_low_tokens: float) -> float:
    """C of Sec. 4.3 for one trajectory; any consistent time unit."""
    if min(t_router, t_high, t_low) < 0 or min(n_steps, n_high_tokens, n_low_tokens) < 0:
        raise ValueError("times and counts must be non-negative")
    return t_router * n_steps + t_high * n_high_tokens + t_low * n_low_tokens


def relative_cost_at_budget(rho: float, t_high: float, t_low: float, t_router: float = 0.0,
                            tokens_per_step: float = 1.0) -> float:
    """C(routed at high-precision budget rho) / C(every step on the high-precision model, no router), for steps
    of equal length: a fraction rho of the steps (Sec. 4.2 "Inference-time calibration": rho in {0.2, 0.4, 0.7})
    runs on the high-precision model.  t_router = 0 leaves the router's own cost out (say so where the number is
    reported)."""
    if not 0.0 <= rho <= 1.0:
        raise ValueError("rho must lie in [0, 1]")
    if t_high <= 0 or tokens_per_step <= 0:
        raise ValueError("t_high and tokens_per_step must be positive")
    routed = episode_cost(t_router, 1, t_high, rho * tokens_per_step, t_low, (1.0 - rho) * tokens_per_step)
    return routed / (t_high * tokens_per_step)


def projected_w3_time(t_w4: float, speedup: float = 1.15) -> float:
    """App. "Latency calibration": the 3-bit model's per-token time is projected as T_W4 / 1.15."""
    return t_w4 / speedup
