"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU checker.

This module only *draws* tensors: normal weights and activations rounded to bf16 bit
patterns, Bernoulli precision masks, outlier channels. It holds none of the method's
arithmetic (no quantization, no packing, no matmul) so that it can feed the CUDA path
and the CPU oracle alike without coupling them.

The layers are stand-ins for the decoder checkpoints the paper evaluates (Sec. 5,
"Experimental Models and Precision"): weights ~ N(0, 0.02^2), activations ~ N(0, 1),
both rounded to nearest-even bf16.
"""
from __future__ import annotations

import numpy as np

WEIGHT_SIGMA = 0.02
ACT_SIGMA = 1.0

# tensor ids inside one seed's stream family
TID_WEIGHT = 0
TID_ACT = 1
TID_MASK = 2
TID_OUTLIER = 3
TID_SAMPLE = 4


def f64_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bf16 (ties to even); returns uint16 bit patterns.

    One rounding step straight from the float64 bit fields (never through float32), so no
    double rounding. Inputs must be zero or finite with a magnitude inside bf16's normal range.
    """
    a = np.ascontiguousarray(a, dtype=np.float64)
    u = a.view(np.uint64)
    sign = (u >> np.uint64(63)).astype(np.uint32)
    exp = ((u >> np.uint64(52)) & np.uint64(0x7FF)).astype(np.int64)
    man = u & np.uint64((1 << 52) - 1)
    is_zero = (exp == 0) & (man == 0)
    e = exp - 1023 + 127
    if not np.all(is_zero | ((e >= 1) & (e <= 254))):
        raise ValueError("value outside bf16 normal range")
    m7 = (man >> np.uint64(45)).astype(np.uint32)
    rem = man & np.uint64((1 << 45) - 1)
    half = np.uint64(1 << 44)
    round_up = (rem > half) | ((rem == half) & ((m7 & 1) == 1))
    mag = (e.astype(np.uint32) << 7 | m7) + round_up.astype(np.uint32)  # carry may bump the exponent
    if np.any(mag[~is_zero] >= 0x7F80):
        raise ValueError("value rounds to bf16 infinity")
    mag = np.where(is_zero, 0, mag).astype(np.uint32)
    return ((sign << 15) | mag).astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _rng(seed: int, tensor_id: int, index: int = 0) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(tensor_id), int(index)])


def normal_bf16(shape, sigma: float, seed: int, tensor_id: int, index: int = 0) -> np.ndarray:
    """N(0, sigma^2) samples as bf16 bit patterns (uint16 array of `shape`)."""
    g = _rng(seed, tensor_id, index)
    x = g.standard_normal(size=shape, dtype=np.float64) * sigma
    return f64_to_bf16_bits(x)


def weights(N: int, K: int, seed: int = 0, index: int = 0) -> np.ndarray:
    """W [N][K] bf16 bits, ~N(0, 0.02^2)."""
    return normal_bf16((N, K), WEIGHT_SIGMA, seed, TID_WEIGHT, index)


def activations(M: int, K: int, seed: int = 0, index: int = 0,
                outlier_frac: float = 0.0, outlier_scale: float = 20.0) -> np.ndarray:
    """X [M][K] bf16 bits, ~N(0, 1); optionally floor(outlier_frac*K) seeded channels x outlier_scale."""
    g = _rng(seed, TID_ACT, index)
    x = g.standard_normal(size=(M, K), dtype=np.float64) * ACT_SIGMA
    n_out = int(np.floor(outlier_frac * K))
    if n_out > 0:
        cols = _rng(seed, TID_OUTLIER, index).permutation(K)[:n_out]
        x[:, cols] *= outlier_scale
    return f64_to_bf16_bits(x)


def precision_mask(M: int, p_high: float = 0.3, seed: int = 0, index: int = 0) -> np.ndarray:
    """mask [M] uint8; 1 = the step needs the high-precision (bf16) weights, drawn Bernoulli(p_high)."""
    g = _rng(seed, TID_MASK, index)
    return (g.random(M) < p_high).astype(np.uint8)


def sample_outputs(M: int, N: int, count: int, seed: int = 0, index: int = 0):
    """`count` seeded (m, n) output coordinates plus the corners and edges of the output."""
    g = _rng(seed, TID_SAMPLE, index)
    ms = g.integers(0, M, size=count, dtype=np.int64)
    ns = g.integers(0, N, size=count, dtype=np.int64)
    edge_m = np.array([0, 0, M - 1, M - 1, M // 2], dtype=np.int64)
    edge_n = np.array([0, N - 1, 0, N - 1, N // 2], dtype=np.int64)
    return (np.concatenate([edge_m, ms]).astype(np.int32),
            np.concatenate([edge_n, ns]).astype(np.int32))


# Decoder layer shapes (N = out features, K = in features) used by tests and bench.
LAYER_7B = {
    "qkv": (12288, 4096),
    "o": (4096, 4096),
    "gate_up": (22016, 4096),
    "down": (4096, 11008),
}
LAYER_14B = {
    "q": (5120, 5120),
    "k": (1024, 5120),
    "v": (1024, 5120),
    "o": (5120, 5120),
    "gate": (13824, 5120),
    "up": (13824, 5120),
    "down": (5120, 13824),
}
LAYER_32B = {
    "gate": (27648, 5120),
    "down": (5120, 27648),
}


TID_LOGIT = 71
TID_LOGIT_NOISE = 72
TID_STEP_LEN = 73


def logit_pair(T: int, V: int, seed: int = 0, index: int = 0, critical_frac: float = 0.1):
    """Two [T][V] float64 logit matrices standing in for the high- and the low-precision model on the
    same action tokens: high ~ N(0, 2.5^2) with a few strongly preferred entries per token; low =
    high + N(0, 0.1^2) for most tokens and + N(0, 1.5^2) for a `critical_frac` of them (most steps
    agree closely, a few deviate a lot)."""
    g = _rng(seed, TID_LOGIT, index)
    high = g.standard_normal(size=(T, V), dtype=np.float64) * 2.5
    for i in range(T):
        top = g.integers(0, V, size=3)
        high[i, top] += np.array([9.0, 7.0, 6.0])
    gn = _rng(seed, TID_LOGIT_NOISE, index)
    sigma = np.where(gn.random(T) < critical_frac, 1.5, 0.1)
    low = high + gn.standard_normal(size=(T, V), dtype=np.float64) * sigma[:, None]
    return high, low


def step_offsets(T: int, mean_len: int = 12, seed: int = 0, index: int = 0) -> np.ndarray:
    """int32 [S + 1] token offsets of consecutive steps whose action blocks have 0 .. 2 mean_len tokens."""
    g = _rng(seed, TID_STEP_LEN, index)
    offs = [0]
    while offs[-1] < T:
        offs.append(min(T, offs[-1] + int(g.integers(0, 2 * mean_len + 1))))
    return np.asarray(offs, dtype=np.int32)


# ---- the step-level router (Sec. 4.1): random-init parameters and synthetic step embeddings ----
TID_ROUTER_PARAM = 81
TID_ROUTER_EMB = 82
TID_ROUTER_LEN = 83


def router_params(d: int, heads: int, ffn: int, layers: int, l_max: int, classes: int, seed: int = 0) -> dict:
    """Random-init parameters of the router's encoder as float32 arrays (the paper times its router with random weights
    too, App. "Per-call router coefficient").  Matrices ~ N(0, 1/fan_in), biases and positional embeddings small,
    layer-norm gains near one.  Shapes: see the oracle's router_forward."""
    g = _rng(seed, TID_ROUTER_PARAM, d * 131 + layers)

    def mat(rows, cols):
        return (g.standard_normal((rows, cols)) / np.sqrt(cols)).astype(np.float32)

    def vec(n, scale=0.05, base=0.0):
        return (base + scale * g.standard_normal(n)).astype(np.float32)

    del heads  # the head count does not change any shape
    p = {"pos": (0.1 * g.standard_normal((l_max, d))).astype(np.float32), "layers": []}
    for _ in range(layers):
        p["layers"].append({
            "wqkv": mat(3 * d, d), "bqkv": vec(3 * d), "wo": mat(d, d), "bo": vec(d),
            "ln1_g": vec(d, 0.05, 1.0), "ln1_b": vec(d),
            "w1": mat(ffn, d), "b1": vec(ffn), "w2": mat(d, ffn), "b2": vec(d),
            "ln2_g": vec(d, 0.05, 1.0), "ln2_b": vec(d),
        })
    p["wc"] = mat(classes, d)
    p["bc"] = vec(classes)
    return p


def router_embeddings(B: int, L: int, d: int, seed: int = 0, index: int = 0) -> np.ndarray:
    """Z [B][L][d] float32: stand-ins for the frozen sentence encoder's step embeddings (unit-scale normal rows)."""
    return _rng(seed, TID_ROUTER_EMB, index).standard_normal((B, L, d)).astype(np.float32)


def router_lengths(B: int, L: int, seed: int = 0, index: int = 0) -> np.ndarray:
    """Valid entries per sequence (task embedding + steps so far), uniform in [1, L]; the first and last sequence take
    the extremes 1 and L."""
    n = _rng(seed, TID_ROUTER_LEN, index).integers(1, L + 1, size=B, dtype=np.int64).astype(np.int32)
    n[0] = 1
    n[-1] = L
    return n
