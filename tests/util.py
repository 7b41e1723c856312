"""Small helpers shared by the tests (no method arithmetic)."""
import numpy as np
import torch


def bits_of(t: torch.Tensor) -> np.ndarray:
    """BF16 tensor -> uint16 bit patterns (numpy, on the host)."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16).copy()


def bf16_from_bits(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits, np.uint16).view(np.int16).copy()).view(torch.bfloat16)


def f32_of_bits(bits: np.ndarray) -> np.ndarray:
    """uint16 BF16 patterns -> float32 values, by widening the bit pattern (numpy only)."""
    return (np.ascontiguousarray(bits, np.uint16).astype(np.uint32) << 16).view(np.float32)
