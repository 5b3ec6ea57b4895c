"""Helpers shared by the GPU parity tests: numpy inputs -> CUDA tensors and back."""
import numpy as np
import torch


def to_dev_u8(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint8)).cuda()


def to_dev_f16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits, dtype=np.uint16).view(np.float16)).cuda()


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits, dtype=np.uint16).view(np.int16)).cuda().view(torch.bfloat16)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def gemv_error(y: np.ndarray, ref: np.ndarray) -> float:
    """max_i |y_i - ref_i| / max(|ref_i|, 1e-3 * max|ref|): the relative error the tolerance is stated on."""
    ref = np.asarray(ref, dtype=np.float64)
    floor = 1e-3 * np.abs(ref).max()
    return float(np.max(np.abs(np.asarray(y, dtype=np.float64) - ref) / np.maximum(np.abs(ref), floor)))
