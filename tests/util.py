"""Helpers of the GPU parity tests: tensor conversion and error norms."""
import numpy as np
import torch


def f32(x: float) -> float:
    """The value a float takes when it crosses the C ABI as `float`."""
    return float(np.float32(x))


def np64(t: torch.Tensor) -> np.ndarray:
    """Exact float64 copy of a stored tensor (bf16 and fp32 values are representable)."""
    return t.detach().float().cpu().numpy().astype(np.float64)


def rel_fro(a, b) -> float:
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    nb = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / nb) if nb > 0 else float(np.linalg.norm(a))


def tol_for(dtype) -> float:
    """Relative Frobenius tolerance of dX and dW: 1e-5 for the fp32 path, 2e-2 for bf16 inputs
    with fp32 accumulation (bf16 outputs carry 2^-9 rounding per element, about 2e-3 in norm)."""
    return 1e-5 if dtype == torch.float32 else 2e-2
