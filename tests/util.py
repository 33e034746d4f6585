"""Helpers shared by the tests: bf16 <-> numpy conversions, nothing of the method."""
import numpy as np
import torch


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 torch tensor -> uint16 bit patterns (numpy, on host)."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16).copy()


def bits_to_f64(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f32_to_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns by torch's round-to-nearest-even."""
    return bits(torch.from_numpy(np.ascontiguousarray(x, np.float32)).to(torch.bfloat16))


def npf(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().numpy()
