"""Conversions between the numpy bit-pattern world of the oracle and torch CUDA tensors."""
import numpy as np
import torch


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def bf16_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bf16_tensor_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()


def qweight_np(q) -> np.ndarray:
    return q.qweight.cpu().numpy().view(np.uint32)


def scales_np(q) -> np.ndarray:
    return bf16_to_bits(q.scales)


def zeros_np(q) -> np.ndarray:
    return q.zeros.cpu().numpy()


def rel_err(Y: np.ndarray, ref: np.ndarray) -> float:
    """max|Y - ref| / max|ref|: the acceptance metric for linear outputs."""
    return float(np.abs(Y - ref).max() / np.abs(ref).max())
