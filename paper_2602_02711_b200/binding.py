"""ctypes binding of libdmr.so: argument marshalling only, every step runs in the CUDA kernels.

Functions carry the names of the C entry points (include/dmr.h) and take torch CUDA tensors
(or, for the *_host call, pinned host tensors). There is no CPU fallback: if the library is
missing or a call fails, a DmrError is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libdmr.so")

OUT_BF16 = 0
OUT_F32 = 1
OP_LOWBIT, OP_DENSE, OP_ROUTED = 0, 1, 2


class DmrError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"libdmr: {msg} (status {code})")
        self.code = code


class QFormat(ctypes.Structure):
    """dmr_qformat_t: bits in {3, 4, 8}; group_size 0 = one group per output row."""
    _fields_ = [("bits", ctypes.c_int32), ("group_size", ctypes.c_int32)]

    def group(self, K: int) -> int:
        return K if self.group_size == 0 else self.group_size


_lib = None


class RouterCfg(ctypes.Structure):
    """dmr_router_cfg_t: sizes of the step-level router's encoder (Sec. 4.1)."""
    _fields_ = [("d", ctypes.c_int32), ("heads", ctypes.c_int32), ("ffn", ctypes.c_int32), ("layers", ctypes.c_int32),
                ("l_max", ctypes.c_int32), ("classes", ctypes.c_int32)]


def lib_path() -> str:
    return _LIB_PATH


def lib() -> ctypes.CDLL:
    """Loads libdmr.so (built in-tree by paper_2602_02711_b200.build). Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise DmrError(-1, f"{_LIB_PATH} not found: run `python -m paper_2602_02711_b200.build`")
    L = ctypes.CDLL(_LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    for name in ("dmr_qweight_bytes", "dmr_scales_bytes", "dmr_zeros_bytes"):
        getattr(L, name).restype = sz
        getattr(L, name).argtypes = [i32, i32, QFormat]
    L.dmr_workspace_bytes.restype = sz
    L.dmr_workspace_bytes.argtypes = [i32, i32, i32, i32, QFormat]
    L.dmr_stepwise_kl.restype = i32
    L.dmr_stepwise_kl.argtypes = [vp, vp, i32, i32, i32, vp, i32, vp, vp, vp]
    L.dmr_quantize.restype = i32
    L.dmr_quantize.argtypes = [vp, i32, i32, QFormat, vp, vp, vp, vp, vp]
    L.dmr_dequantize.restype = i32
    L.dmr_dequantize.argtypes = [vp, vp, vp, i32, i32, QFormat, vp, i32, vp]
    L.dmr_lowbit_linear.restype = i32
    L.dmr_lowbit_linear.argtypes = [vp, i32, vp, vp, vp, i32, i32, QFormat, vp, i32, vp, sz, vp]
    L.dmr_dense_linear.restype = i32
    L.dmr_dense_linear.argtypes = [vp, i32, vp, i32, i32, vp, i32, vp, sz, vp]
    L.dmr_routed_linear.restype = i32
    L.dmr_routed_linear.argtypes = [vp, i32, vp, vp, vp, vp, vp, i32, i32, QFormat, vp, i32, vp, sz, vp]
    L.dmr_route_partition.restype = i32
    L.dmr_route_partition.argtypes = [vp, i32, vp, vp, vp, vp]
    L.dmr_host_staging_bytes.restype = sz
    L.dmr_host_staging_bytes.argtypes = [i32, i32, i32, i32]
    L.dmr_lowbit_linear_host.restype = i32
    L.dmr_lowbit_linear_host.argtypes = [vp, i32, vp, vp, vp, i32, i32, QFormat, vp, i32, vp, sz, vp, sz, vp]
    L.dmr_noalloc_max_n.restype = i32
    L.dmr_lowbit_linear_noalloc.restype = i32
    L.dmr_lowbit_linear_noalloc.argtypes = [vp, i32, vp, vp, vp, i32, i32, QFormat, vp, i32, vp]
    L.dmr_router_calibrate.restype = i32
    L.dmr_router_calibrate.argtypes = [vp, i32, ctypes.c_double, vp, vp]
    L.dmr_router_mask.restype = i32
    L.dmr_router_mask.argtypes = [vp, i32, vp, vp, vp]
    L.dmr_router_param_floats.restype = sz
    L.dmr_router_param_floats.argtypes = [RouterCfg]
    L.dmr_router_workspace_bytes.restype = sz
    L.dmr_router_workspace_bytes.argtypes = [RouterCfg, i32, i32]
    L.dmr_router_forward.restype = i32
    L.dmr_router_forward.argtypes = [vp, RouterCfg, vp, vp, i32, i32, vp, vp, i32, vp, sz, vp]
    L.dmr_selftest_wait_timeout.restype = i32
    L.dmr_selftest_wait_timeout.argtypes = [vp, sz, vp]
    L.dmr_workspace_status.restype = i32
    L.dmr_workspace_status.argtypes = [vp, vp]
    L.dmr_describe_dispatch.restype = i32
    L.dmr_describe_dispatch.argtypes = [i32, i32, i32, i32, QFormat, ctypes.c_char_p, sz]
    L.dmr_status_string.restype = ctypes.c_char_p
    L.dmr_status_string.argtypes = [i32]
    L.dmr_last_cuda_error.restype = i32
    L.dmr_launch_count.restype = ctypes.c_uint64
    _lib = L
    return L


def _check(code: int):
    if code != 0:
        L = lib()
        msg = L.dmr_status_string(code).decode()
        if code == 7:
            msg += f" (cudaError {L.dmr_last_cuda_error()})"
        raise DmrError(code, msg)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _dev(t: torch.Tensor, dtype, name: str):
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise DmrError(1, f"{name} must be a contiguous CUDA tensor of {dtype}")
    return t


def dmr_launch_count() -> int:
    return int(lib().dmr_launch_count())


def dmr_describe_dispatch(op: int, M: int, N: int, K: int, fmt: QFormat = None) -> dict:
    """Which kernel family and launch shape the library would use, as a dict such as
    {"kernel": "prefill", "bits": 4, "bn": 256, "tiles": 3072, "ctas": 148}."""
    buf = ctypes.create_string_buffer(256)
    n = lib().dmr_describe_dispatch(op, M, N, K, fmt if fmt is not None else QFormat(4, 0), buf, 256)
    if n < 0:
        raise DmrError(1, "invalid arguments")
    words = buf.value.decode().split()
    out = {"kernel": words[0]}
    for w in words[1:]:
        k, v = w.split("=")
        out[k] = int(v)
    return out


def dmr_workspace_bytes(op: int, M: int, N: int, K: int, fmt: QFormat) -> int:
    return int(lib().dmr_workspace_bytes(op, M, N, K, fmt))


def new_workspace(op: int, M: int, N: int, K: int, fmt: QFormat, device="cuda") -> torch.Tensor:
    """A zeroed scratch buffer of the size `op` needs (torch owns the memory)."""
    return torch.zeros(dmr_workspace_bytes(op, M, N, K, fmt), dtype=torch.uint8, device=device)


@dataclass
class QuantizedLinear:
    """Packed weights of one Linear layer as dmr_quantize lays them out."""
    qweight: torch.Tensor  # int32 [N][K*bits/32]
    scales: torch.Tensor   # bf16  [N][G]
    zeros: torch.Tensor    # uint8 [N][G]
    N: int
    K: int
    fmt: QFormat

    def weight_bytes(self) -> int:
        return self.qweight.numel() * 4 + self.scales.numel() * 2 + self.zeros.numel()


def dmr_quantize(W: torch.Tensor, fmt: QFormat, stream=None, check: bool = True) -> QuantizedLinear:
    """bf16 W [N][K] -> packed codes + per-group scale / zero. check=True synchronises to read the status."""
    _dev(W, torch.bfloat16, "W")
    N, K = W.shape
    L = lib()
    qb = L.dmr_qweight_bytes(N, K, fmt)
    if qb == 0:
        raise DmrError(1, "invalid quantization format for this K")
    G = K // fmt.group(K)
    qweight = torch.empty((N, K * fmt.bits // 32), dtype=torch.int32, device=W.device)
    scales = torch.empty((N, G), dtype=torch.bfloat16, device=W.device)
    zeros = torch.empty((N, G), dtype=torch.uint8, device=W.device)
    status = torch.zeros(1, dtype=torch.int32, device=W.device)
    _check(L.dmr_quantize(_ptr(W), N, K, fmt, _ptr(qweight), _ptr(scales), _ptr(zeros), _ptr(status), _stream(stream)))
    if check:
        code = int(status.item())
        if code != 0:
            _check(code)
    return QuantizedLinear(qweight, scales, zeros, N, K, fmt)


def quantize_layer(W: torch.Tensor, bits: int = 4, group_size: int = 128) -> QuantizedLinear:
    return dmr_quantize(W, QFormat(bits, group_size))


def dmr_dequantize(q: QuantizedLinear, out: int = OUT_F32, stream=None) -> torch.Tensor:
    W = torch.empty((q.N, q.K), dtype=torch.float32 if out == OUT_F32 else torch.bfloat16, device=q.qweight.device)
    _check(lib().dmr_dequantize(_ptr(q.qweight), _ptr(q.scales), _ptr(q.zeros), q.N, q.K, q.fmt, _ptr(W), out,
                                _stream(stream)))
    return W


def _out_tensor(M, N, out, device, Y):
    dt = torch.float32 if out == OUT_F32 else torch.bfloat16
    if Y is None:
        return torch.empty((M, N), dtype=dt, device=device)
    return _dev(Y, dt, "Y")


def dmr_lowbit_linear(X: torch.Tensor, q: QuantizedLinear, out: int = OUT_BF16, Y=None, workspace=None,
                      stream=None) -> torch.Tensor:
    """Y = X . dequant(Wq)^T."""
    _dev(X, torch.bfloat16, "X")
    M, K = X.shape
    if K != q.K:
        raise DmrError(1, "X and the quantized weights disagree on K")
    Y = _out_tensor(M, q.N, out, X.device, Y)
    if workspace is None:
        workspace = new_workspace(OP_LOWBIT, M, q.N, K, q.fmt, X.device)
    _check(lib().dmr_lowbit_linear(_ptr(X), M, _ptr(q.qweight), _ptr(q.scales), _ptr(q.zeros), q.N, K, q.fmt,
                                   _ptr(Y), out, _ptr(workspace), workspace.numel(), _stream(stream)))
    return Y


def dmr_dense_linear(X: torch.Tensor, W: torch.Tensor, out: int = OUT_BF16, Y=None, workspace=None,
                     stream=None) -> torch.Tensor:
    """Y = X . W^T with bf16 weights."""
    _dev(X, torch.bfloat16, "X")
    _dev(W, torch.bfloat16, "W")
    M, K = X.shape
    N = W.shape[0]
    if W.shape[1] != K:
        raise DmrError(1, "X and W disagree on K")
    Y = _out_tensor(M, N, out, X.device, Y)
    if workspace is None:
        workspace = new_workspace(OP_DENSE, M, N, K, QFormat(4, 0), X.device)
    _check(lib().dmr_dense_linear(_ptr(X), M, _ptr(W), N, K, _ptr(Y), out, _ptr(workspace), workspace.numel(),
                                  _stream(stream)))
    return Y


def dmr_routed_linear(X: torch.Tensor, mask: torch.Tensor, W: torch.Tensor, q: QuantizedLinear,
                      out: int = OUT_BF16, Y=None, workspace=None, stream=None) -> torch.Tensor:
    """Rows with mask != 0 use the bf16 weights, the others the low-bit weights; Y keeps step order."""
    _dev(X, torch.bfloat16, "X")
    _dev(W, torch.bfloat16, "W")
    _dev(mask, torch.uint8, "mask")
    M, K = X.shape
    if mask.numel() != M or W.shape != (q.N, K) or q.K != K:
        raise DmrError(1, "shape mismatch")
    Y = _out_tensor(M, q.N, out, X.device, Y)
    if workspace is None:
        workspace = new_workspace(OP_ROUTED, M, q.N, K, q.fmt, X.device)
    _check(lib().dmr_routed_linear(_ptr(X), M, _ptr(mask), _ptr(W), _ptr(q.qweight), _ptr(q.scales), _ptr(q.zeros),
                                   q.N, K, q.fmt, _ptr(Y), out, _ptr(workspace), workspace.numel(), _stream(stream)))
    return Y


def dmr_route_partition(mask: torch.Tensor, stream=None):
    """-> (idx_high int32 [M], idx_low int32 [M], counts int32 [2] = {n_high, n_low}), all on the device."""
    _dev(mask, torch.uint8, "mask")
    M = mask.numel()
    ih = torch.empty(max(M, 1), dtype=torch.int32, device=mask.device)
    il = torch.empty(max(M, 1), dtype=torch.int32, device=mask.device)
    counts = torch.empty(2, dtype=torch.int32, device=mask.device)
    _check(lib().dmr_route_partition(_ptr(mask), M, _ptr(ih), _ptr(il), _ptr(counts), _stream(stream)))
    return ih, il, counts


def dmr_lowbit_linear_host(X_host: torch.Tensor, q: QuantizedLinear, Y_host: torch.Tensor, out: int = OUT_BF16,
                           staging=None, workspace=None, stream=None):
    """Host-buffer variant: X_host / Y_host are (pinned) CPU tensors; copies run on `stream`."""
    if X_host.is_cuda or Y_host.is_cuda:
        raise DmrError(1, "X_host and Y_host must be CPU tensors")
    M, K = X_host.shape
    L = lib()
    dev = q.qweight.device
    if staging is None:
        staging = torch.empty(L.dmr_host_staging_bytes(M, q.N, K, out), dtype=torch.uint8, device=dev)
    if workspace is None:
        workspace = new_workspace(OP_LOWBIT, M, q.N, K, q.fmt, dev)
    _check(L.dmr_lowbit_linear_host(_ptr(X_host), M, _ptr(q.qweight), _ptr(q.scales), _ptr(q.zeros), q.N, K, q.fmt,
                                    _ptr(Y_host), out, _ptr(staging), staging.numel(), _ptr(workspace),
                                    workspace.numel(), _stream(stream)))
    return Y_host


def dmr_stepwise_kl(logits_high: torch.Tensor, logits_low: torch.Tensor, step_offsets: torch.Tensor, stream=None):
    """Step-wise KL divergence of two [T, V] logit tensors (bf16 or fp32, same dtype).

    `step_offsets` is an int32 device tensor [S + 1]. Returns (kl_step [S], kl_token [T]), fp32.
    """
    if logits_high.dtype not in (torch.bfloat16, torch.float32) or logits_low.dtype != logits_high.dtype:
        raise DmrError(1, "logits must both be bf16 or both be fp32")
    a = _dev(logits_high, logits_high.dtype, "logits_high")
    b = _dev(logits_low, logits_high.dtype, "logits_low")
    if a.dim() != 2 or a.shape != b.shape:
        raise DmrError(1, "logits must be [T, V] tensors of the same shape")
    off = _dev(step_offsets, torch.int32, "step_offsets")
    T, V = a.shape
    S = off.numel() - 1
    kl_token = torch.empty((T,), dtype=torch.float32, device=a.device)
    kl_step = torch.empty((max(S, 0),), dtype=torch.float32, device=a.device)
    dtype = OUT_F32 if a.dtype == torch.float32 else OUT_BF16
    _check(lib().dmr_stepwise_kl(_ptr(a), _ptr(b), dtype, T, V, _ptr(off), S, _ptr(kl_token), _ptr(kl_step), _stream(stream)))
    return kl_step, kl_token


def dmr_lowbit_linear_noalloc(X: torch.Tensor, q: QuantizedLinear, Y: torch.Tensor, out: int = OUT_BF16, stream=None):
    """dmr_lowbit_linear for M <= 16 without a workspace: the library's own fixed scratch is used, so
    the call itself allocates nothing. The caller passes the output tensor Y ([M][N], bf16 or fp32)."""
    _dev(X, torch.bfloat16, "X")
    _dev(Y, torch.float32 if out == OUT_F32 else torch.bfloat16, "Y")
    M, K = X.shape
    if K != q.K or tuple(Y.shape) != (M, q.N):
        raise DmrError(1, "shape mismatch")
    _check(lib().dmr_lowbit_linear_noalloc(_ptr(X), M, _ptr(q.qweight), _ptr(q.scales), _ptr(q.zeros), q.N, K, q.fmt,
                                           _ptr(Y), out, _stream(stream)))
    return Y


def dmr_router_calibrate(cal_scores: torch.Tensor, rho: float, stream=None) -> torch.Tensor:
    """tau(rho) = Quantile(cal_scores, 1 - rho) on the device. Returns a float64 device tensor [3]; element 0 is tau."""
    _dev(cal_scores, torch.float32, "cal_scores")
    tau = torch.zeros(3, dtype=torch.float64, device=cal_scores.device)
    _check(lib().dmr_router_calibrate(_ptr(cal_scores), cal_scores.numel(), float(rho), _ptr(tau), _stream(stream)))
    return tau


def dmr_router_mask(scores: torch.Tensor, tau: torch.Tensor, stream=None) -> torch.Tensor:
    """mask[m] = 1 where scores[m] >= tau[0] (the step needs the high-precision weights), uint8 on the device."""
    _dev(scores, torch.float32, "scores")
    _dev(tau, torch.float64, "tau")
    mask = torch.empty(scores.numel(), dtype=torch.uint8, device=scores.device)
    _check(lib().dmr_router_mask(_ptr(scores), scores.numel(), _ptr(tau), _ptr(mask), _stream(stream)))
    return mask


def pack_router_params(params: dict, cfg: RouterCfg, device="cuda") -> torch.Tensor:
    """Lays a dict of router parameters (numpy / torch arrays, shapes as in include/dmr.h) out as the one fp32 device
    buffer dmr_router_forward reads: pos; per layer wqkv, bqkv, wo, bo, ln1_g, ln1_b, w1, b1, w2, b2, ln2_g, ln2_b; wc, bc."""
    n = lib().dmr_router_param_floats(cfg)
    if n == 0:
        raise DmrError(1, "invalid router configuration")
    parts = [params["pos"]]
    for lay in params["layers"]:
        parts += [lay[k] for k in ("wqkv", "bqkv", "wo", "bo", "ln1_g", "ln1_b", "w1", "b1", "w2", "b2", "ln2_g", "ln2_b")]
    parts += [params["wc"], params["bc"]]
    flat = torch.cat([torch.as_tensor(a, dtype=torch.float32).reshape(-1) for a in parts])
    if flat.numel() != n or len(params["layers"]) != cfg.layers:
        raise DmrError(1, "router parameters do not match the configuration")
    return flat.to(device)


def dmr_router_forward(params: torch.Tensor, cfg: RouterCfg, Z: torch.Tensor, lengths: torch.Tensor, score_class: int = 0,
                       workspace=None, stream=None):
    """Router forward on the device: Z [B][L][d] fp32, lengths [B] int32 -> (probs [B][classes], scores [B] =
    probs[:, score_class]), both fp32 on the device."""
    _dev(params, torch.float32, "params")
    _dev(Z, torch.float32, "Z")
    _dev(lengths, torch.int32, "lengths")
    B, L, d = Z.shape
    if d != cfg.d or lengths.numel() != B:
        raise DmrError(1, "shape mismatch")
    probs = torch.empty((B, cfg.classes), dtype=torch.float32, device=Z.device)
    scores = torch.empty(B, dtype=torch.float32, device=Z.device)
    if B == 0:
        return probs, scores
    need = lib().dmr_router_workspace_bytes(cfg, B, L)
    if need == 0:
        raise DmrError(1, "invalid router configuration or sizes")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=Z.device)
    _check(lib().dmr_router_forward(_ptr(params), cfg, _ptr(Z), _ptr(lengths), B, L, _ptr(probs), _ptr(scores), int(score_class),
                                    _ptr(workspace), workspace.numel(), _stream(stream)))
    return probs, scores
