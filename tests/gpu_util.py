"""Helpers for the GPU parity tests: numpy bit patterns <-> torch device tensors."""
import numpy as np
import torch


def dev_bits(a: np.ndarray) -> torch.Tensor:
    """uint16 bit patterns -> int16 CUDA tensor holding the same bits."""
    a = np.ascontiguousarray(a, np.uint16)
    return torch.from_numpy(a.view(np.int16)).cuda()


def dev_i32(a) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, np.int32)).cuda()


def rel_err(y_gpu: np.ndarray, y_ref: np.ndarray) -> float:
    """max_i |y_i - ref_i| / max(|ref_i|, rms(ref)): relative error that does not blow up on
    outputs that happen to be near zero."""
    y_ref = np.asarray(y_ref, np.float64)
    rms = float(np.sqrt(np.mean(y_ref ** 2))) if y_ref.size else 0.0
    den = np.maximum(np.abs(y_ref), max(rms, 1e-30))
    return float(np.max(np.abs(np.asarray(y_gpu, np.float64) - y_ref) / den)) if y_ref.size else 0.0
