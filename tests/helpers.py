"""Shared helpers of the GPU parity tests: host<->device conversion and tolerance rules."""
import numpy as np


def to_dev(bits: np.ndarray):
    """uint16 bf16 bit patterns -> torch.bfloat16 CUDA tensor of the same shape."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def bf16_to_np(t) -> np.ndarray:
    """torch.bfloat16 tensor -> float64 numpy."""
    import torch
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def merged_close(got: np.ndarray, ref: np.ndarray):
    """Merged K/V acceptance: 2e-2 absolute, widened to bf16's rounding step (half an ulp is at
    most |x| * 2^-8) where the value itself is too large for 2e-2 to be representable."""
    tol = np.maximum(2e-2, np.abs(ref) * (2.0 ** -8) * 1.01)
    return np.abs(got - ref) <= tol
