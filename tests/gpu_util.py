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


def tensor_core_slack(k_in: int, ref: np.ndarray) -> float:
    """Absolute error the tensor-core accumulation of a K-long product may add on top of the relative tolerance.

    The tensor core adds the 16 products of one MMA step and the running sum with a single truncation, so a sum over
    k_in terms takes k_in / 16 truncations of at most one unit in the last place (2^-23) of the running sum, and the
    running sums of these products stay below a quarter of the largest output.  Measured on the 28672-long rows:
    a fifth of this bound.  Outputs far above the floor of the relative tolerance are not affected by it."""
    return (k_in / 16.0) * 2.0 ** -23 * 0.25 * float(np.abs(ref).max())


def gemm_error(y: np.ndarray, ref: np.ndarray, k_in: int) -> float:
    """gemv_error with the tensor-core accumulation slack taken off the absolute error first."""
    ref = np.asarray(ref, dtype=np.float64)
    floor = 1e-3 * np.abs(ref).max()
    err = np.maximum(np.abs(np.asarray(y, dtype=np.float64) - ref) - tensor_core_slack(k_in, ref), 0.0)
    return float(np.max(err / np.maximum(np.abs(ref), floor)))
