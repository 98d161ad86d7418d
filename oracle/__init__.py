"""ctypes front end of the CPU oracle (`dmr_oracle.c`).

TEST INFRASTRUCTURE ONLY. The product path never imports this package; only the tests, the
smoke check and the benchmark's CPU-baseline leg do. It shares nothing with the CUDA
library: it compiles its own C file with gcc and works on numpy arrays.

All tensors are numpy arrays: bf16 tensors are uint16 bit patterns, outputs are float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dmr_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

OK = 0
ERR_ARG = 1
ERR_NONFINITE = 5


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no FMA contraction, OpenMP). Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_bf16_to_f64.restype = ctypes.c_double
        _lib.oracle_bf16_to_f64.argtypes = [ctypes.c_uint16]
        _lib.oracle_f64_to_bf16_rne.restype = ctypes.c_uint16
        _lib.oracle_f64_to_bf16_rne.argtypes = [ctypes.c_double]
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__(f"oracle error code {code}")
        self.code = code


def _check(code):
    if code != OK:
        raise OracleError(code)


def num_threads() -> int:
    return int(_L().oracle_num_threads())


def group_of(K: int, group: int) -> int:
    return K if group == 0 else group


def f64_to_bf16_rne(x: float) -> int:
    return int(_L().oracle_f64_to_bf16_rne(float(x)))


def bf16_to_f64(b: int) -> float:
    return float(_L().oracle_bf16_to_f64(int(b)))


def pack(codes: np.ndarray, bits: int) -> np.ndarray:
    codes = _c(codes, np.uint8)
    N, K = codes.shape
    out = np.zeros((N, K * bits // 32), dtype=np.uint32)
    _check(_L().oracle_pack(_p(codes), N, K, bits, _p(out)))
    return out


def unpack(qweight: np.ndarray, K: int, bits: int) -> np.ndarray:
    qweight = _c(qweight, np.uint32)
    N = qweight.shape[0]
    out = np.zeros((N, K), dtype=np.uint8)
    _check(_L().oracle_unpack(_p(qweight), N, K, bits, _p(out)))
    return out


def quantize(W: np.ndarray, bits: int = 4, group: int = 128, return_codes: bool = False):
    """W [N][K] bf16 bits -> (qweight u32 [N][K*bits/32], scales u16 [N][G], zeros u8 [N][G])."""
    W = _c(W, np.uint16)
    N, K = W.shape
    g = group_of(K, group)
    if K % g != 0 or K % (32 if bits == 3 else 32 // bits) != 0:
        raise OracleError(ERR_ARG)
    G = K // g
    qweight = np.zeros((N, K * bits // 32), dtype=np.uint32)
    scales = np.zeros((N, G), dtype=np.uint16)
    zeros = np.zeros((N, G), dtype=np.uint8)
    codes = np.zeros((N, K), dtype=np.uint8) if return_codes else None
    _check(_L().oracle_quantize(_p(W), N, K, bits, group, _p(qweight), _p(scales), _p(zeros), _p(codes)))
    if return_codes:
        return qweight, scales, zeros, codes
    return qweight, scales, zeros


def dequantize(qweight, scales, zeros, K: int, bits: int = 4, group: int = 128):
    """-> (What float64 [N][K] exact s*(q-z), What_bf16 u16 [N][K] nearest bf16)."""
    qweight = _c(qweight, np.uint32)
    scales = _c(scales, np.uint16)
    zeros = _c(zeros, np.uint8)
    N = qweight.shape[0]
    What = np.zeros((N, K), dtype=np.float64)
    Wb = np.zeros((N, K), dtype=np.uint16)
    _check(_L().oracle_dequantize(_p(qweight), _p(scales), _p(zeros), N, K, bits, group, _p(What), _p(Wb)))
    return What, Wb


def lowbit_linear(X, qweight, scales, zeros, bits: int = 4, group: int = 128, rounded: bool = False):
    """Y [M][N] float64 = X . dequant(Wq)^T (rounded=True uses the nearest-bf16 dequantized weights)."""
    X = _c(X, np.uint16)
    qweight = _c(qweight, np.uint32)
    scales = _c(scales, np.uint16)
    zeros = _c(zeros, np.uint8)
    M, K = X.shape
    N = qweight.shape[0]
    Y = np.zeros((M, N), dtype=np.float64)
    _check(_L().oracle_lowbit_linear(_p(X), M, _p(qweight), _p(scales), _p(zeros), N, K, bits, group,
                                     int(rounded), _p(Y)))
    return Y


def dense_linear(X, W):
    X = _c(X, np.uint16)
    W = _c(W, np.uint16)
    M, K = X.shape
    N = W.shape[0]
    Y = np.zeros((M, N), dtype=np.float64)
    _check(_L().oracle_dense_linear(_p(X), M, _p(W), N, K, _p(Y)))
    return Y


def routed_linear(X, mask, W, qweight, scales, zeros, bits: int = 4, group: int = 128):
    X = _c(X, np.uint16)
    mask = _c(mask, np.uint8)
    W = _c(W, np.uint16)
    qweight = _c(qweight, np.uint32)
    scales = _c(scales, np.uint16)
    zeros = _c(zeros, np.uint8)
    M, K = X.shape
    N = W.shape[0]
    Y = np.zeros((M, N), dtype=np.float64)
    _check(_L().oracle_routed_linear(_p(X), M, _p(mask), _p(W), _p(qweight), _p(scales), _p(zeros),
                                     N, K, bits, group, _p(Y)))
    return Y


def sampled_linear(X, ms, ns, *, mask=None, W=None, qweight=None, scales=None, zeros=None,
                   bits: int = 4, group: int = 128, rounded: bool = False):
    """Values of the (routed / low-bit / dense) linear at the output coordinates (ms[i], ns[i])."""
    X = _c(X, np.uint16)
    M, K = X.shape
    ms = _c(ms, np.int32)
    ns = _c(ns, np.int32)
    if W is not None:
        W = _c(W, np.uint16)
        N = W.shape[0]
    if qweight is not None:
        qweight = _c(qweight, np.uint32)
        scales = _c(scales, np.uint16)
        zeros = _c(zeros, np.uint8)
        N = qweight.shape[0]
    if mask is not None:
        mask = _c(mask, np.uint8)
    out = np.zeros(len(ms), dtype=np.float64)
    _check(_L().oracle_sampled_linear(_p(X), M, _p(mask), _p(W), _p(qweight), _p(scales), _p(zeros),
                                      N, K, bits, group, int(rounded), _p(ms), _p(ns), len(ms), _p(out)))
    return out


def route_partition(mask):
    mask = _c(mask, np.uint8)
    M = mask.shape[0]
    ih = np.zeros(max(M, 1), dtype=np.int32)
    il = np.zeros(max(M, 1), dtype=np.int32)
    nh = ctypes.c_int32(0)
    nl = ctypes.c_int32(0)
    _check(_L().oracle_route_partition(_p(mask), M, _p(ih), _p(il), ctypes.byref(nh), ctypes.byref(nl)))
    return ih[:nh.value].copy(), il[:nl.value].copy()


def stepwise_kl(logits_high: np.ndarray, logits_low: np.ndarray, step_offsets):
    """Step-wise KL divergence (Sec. "KL-ST Stage"; App. on search and click steps):
    KL_t = mean over the action tokens i of step t of KL(pi_high(x_i) || pi_low(x_i)), pi = softmax(logits).

    `logits_high`, `logits_low`: [T][V] arrays, uint16 (bf16 bit patterns) or floating point; everything is
    computed in float64 from the definition: log-softmax of each row, p = exp(log-softmax of the high
    row), KL = sum_v p_v (log p_v - log q_v) with the convention that p_v = 0 contributes 0.
    `step_offsets`: S + 1 non-decreasing token indices. Returns (kl_step [S], kl_token [T]) in nats;
    a step without tokens has KL 0.
    """
    def as_f64(a):
        a = np.asarray(a)
        if a.dtype == np.uint16:
            return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        return a.astype(np.float64)

    A, B = as_f64(logits_high), as_f64(logits_low)
    T = A.shape[0]
    kl_token = np.zeros(T, dtype=np.float64)
    for i in range(T):
        a, b = A[i], B[i]
        log_p = a - (a.max() + np.log(np.sum(np.exp(a - a.max()))))
        log_q = b - (b.max() + np.log(np.sum(np.exp(b - b.max()))))
        p = np.exp(log_p)
        with np.errstate(invalid="ignore"):
            terms = np.where(p > 0.0, p * (log_p - log_q), 0.0)
        kl_token[i] = np.sum(terms)
    off = np.asarray(step_offsets, dtype=np.int64)
    kl_step = np.zeros(max(len(off) - 1, 0), dtype=np.float64)
    for s in range(len(kl_step)):
        seg = kl_token[off[s]:off[s + 1]]
        kl_step[s] = seg.mean() if len(seg) else 0.0
    return kl_step, kl_token


def router_threshold(cal_scores, rho: float) -> float:
    """tau(rho) = Quantile(D_cal, 1 - rho) (Sec. 4.2 "Inference-time calibration"), in float64.

    The paper names no quantile rule; the reading taken is linear interpolation between order statistics: sort
    the scores ascending, h = (n - 1)(1 - rho), lo = floor(h), tau = x[lo] + (h - lo) * (x[lo + 1] - x[lo])
    (x[n - 1] when lo is the last index). Scores are widened exactly to float64 first.
    """
    x = np.sort(np.asarray(cal_scores).astype(np.float64))
    n = len(x)
    if n < 1 or not (0.0 <= rho <= 1.0):
        raise ValueError("need at least one score and 0 <= rho <= 1")
    h = float(n - 1) * (1.0 - float(rho))
    lo = min(int(np.floor(h)), n - 1)
    hi = min(lo + 1, n - 1)
    gamma = h - float(lo)
    return float(x[lo] + gamma * (x[hi] - x[lo]))


def router_mask(scores, tau: float) -> np.ndarray:
    """mask[m] = 1 where the step's router score reaches the threshold (p_t >= tau: high precision), else 0."""
    return (np.asarray(scores).astype(np.float64) >= float(tau)).astype(np.uint8)


def router_forward(Z, lengths, params, heads: int):
    """Forward pass of the step-level router (Sec. 4.1 "Router Architecture"), in float64:

        H_t = TransformerEnc_theta(X_t + P_t, m_t),   pi_theta(r_t | s_t) = Softmax(W h_t*),

    X_t = [z_task, z_1, ..., z_t] (one row of Z per sequence, `lengths[b]` valid entries first: the valid-step mask m_t),
    P_t learned positional embeddings, h_t* the encoder's output at the last valid step.

    The paper fixes neither width, heads, feed-forward size, normalisation placement nor activation.  Reading taken: the
    encoder layer of "Attention is all you need" - post-layer-norm, x <- LN(x + MHA(x)), x <- LN(x + W2 relu(W1 x + b1) + b2),
    scaled dot-product attention over the valid steps only (padded steps are never keys; attention among valid steps is
    not causal: the sequence already ends at the step being decided), LN with eps = 1e-5 over the feature axis, no dropout.

    Z [B][L][d]; lengths [B] (1 <= len <= L); params: dict with
      "pos" [L_max][d]; "layers": list of dicts with "wqkv" [3d][d] (rows: queries, keys, values), "bqkv" [3d], "wo" [d][d],
      "bo" [d], "ln1_g", "ln1_b" [d], "w1" [f][d], "b1" [f], "w2" [d][f], "b2" [d], "ln2_g", "ln2_b" [d];
      "wc" [C][d], "bc" [C].
    Returns probabilities [B][C].
    """
    Z = np.asarray(Z, dtype=np.float64)
    B, L, d = Z.shape
    dh = d // heads
    if dh * heads != d:
        raise ValueError("heads must divide d")
    pos = np.asarray(params["pos"], dtype=np.float64)
    out = np.zeros((B, np.asarray(params["wc"]).shape[0]), dtype=np.float64)

    def layer_norm(x, g, b):
        mu = x.mean(axis=-1, keepdims=True)
        var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
        return (x - mu) / np.sqrt(var + 1e-5) * g + b

    for b in range(B):
        n = int(lengths[b])
        if not 1 <= n <= L:
            raise ValueError("lengths must lie in [1, L]")
        x = Z[b, :n, :] + pos[:n, :]                      # X_t + P_t, valid steps only
        for lay in params["layers"]:
            wqkv = np.asarray(lay["wqkv"], dtype=np.float64)
            qkv = x @ wqkv.T + np.asarray(lay["bqkv"], dtype=np.float64)
            q, k, v = qkv[:, :d], qkv[:, d:2 * d], qkv[:, 2 * d:]
            att = np.zeros_like(x)
            for h in range(heads):
                sl = slice(h * dh, (h + 1) * dh)
                s = (q[:, sl] @ k[:, sl].T) / np.sqrt(float(dh))
                s = s - s.max(axis=-1, keepdims=True)
                p = np.exp(s)
                p = p / p.sum(axis=-1, keepdims=True)
                att[:, sl] = p @ v[:, sl]
            y = att @ np.asarray(lay["wo"], dtype=np.float64).T + np.asarray(lay["bo"], dtype=np.float64)
            x = layer_norm(x + y, np.asarray(lay["ln1_g"], dtype=np.float64), np.asarray(lay["ln1_b"], dtype=np.float64))
            hdn = np.maximum(x @ np.asarray(lay["w1"], dtype=np.float64).T + np.asarray(lay["b1"], dtype=np.float64), 0.0)
            y = hdn @ np.asarray(lay["w2"], dtype=np.float64).T + np.asarray(lay["b2"], dtype=np.float64)
            x = layer_norm(x + y, np.asarray(lay["ln2_g"], dtype=np.float64), np.asarray(lay["ln2_b"], dtype=np.float64))
        hstar = x[n - 1]                                   # last-valid-step pooling
        logits = np.asarray(params["wc"], dtype=np.float64) @ hstar + np.asarray(params["bc"], dtype=np.float64)
        e = np.exp(logits - logits.max())
        out[b] = e / e.sum()
    return out
