"""Shared helpers of the parity tests (harness only: rounding, error metric, marshalling)."""
import math

import numpy as np
import torch

TOL = {"f32": 1e-4, "bf16": 2e-2}   # max relative error allowed against the fp64 oracle


def f64(x: torch.Tensor) -> np.ndarray:
    return x.detach().cpu().to(torch.float64).numpy()


def to_dtype(a: np.ndarray, dtype: torch.dtype) -> torch.Tensor:
    """Round an fp64 array to the run's storage type (round to nearest even)."""
    return torch.from_numpy(np.ascontiguousarray(a)).to(dtype)


def rel_err(a, b) -> float:
    """max_i |a_i - b_i| / max(|b_i|, rms(b)); a = GPU result, b = oracle (fp64).
    The rms floor keeps near-zero elements from dominating a relative error."""
    a = f64(a) if isinstance(a, torch.Tensor) else np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    assert a.shape == b.shape, (a.shape, b.shape)
    if b.size == 0:
        return 0.0
    assert np.all(np.isfinite(a)), "non-finite values in the GPU result"
    rms = math.sqrt(float(np.mean(b * b)))
    den = np.maximum(np.abs(b), max(rms, 1e-30))
    return float(np.max(np.abs(a - b) / den))


def assert_close(a, b, dtype: str, what: str, scale: float = 1.0):
    e = rel_err(a, b)
    assert e <= TOL[dtype] * scale, f"{what}: max relative error {e:.3e} > {TOL[dtype] * scale:.1e}"
    return e
