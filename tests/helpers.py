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


# ---- stratified samples for the full-size parity tests -----------------------------------------
ROW_TILE = 128          # rows of a GEMM output tile (a CTA pair covers two of them)
DW_TILE = (128, 256)    # (channels, inputs) of a weight-gradient output tile, at most


def stratified_tokens(T, rng, n_random=32):
    rows = set()
    for a in range(0, T, ROW_TILE):
        rows.add(a)
        rows.add(min(T, a + ROW_TILE) - 1)
    rows.update(r for r in (127, 128, 255, 256) if r < T)
    rows.update(range(T - T % ROW_TILE, T))                 # the ragged tail, whole
    rows.update(int(r) for r in rng.choice(T, size=min(n_random, T), replace=False))
    return np.array(sorted(rows), dtype=np.int64)


def stratified_entries(t, n_rows, n_cols, rng, n_min=4096, extra_rows=()):
    """(rank, row, col) index arrays over a [t, n_rows, n_cols] weight-shaped tensor with the two extreme corners
    and random entries of every (rank, 128-row block, 256-column block) tile; extra_rows adds whole sampled
    rows' worth of entries around a boundary (the partition edge S)."""
    br, bc = DW_TILE
    tiles = [(m, a, b) for m in range(t) for a in range(0, n_rows, br) for b in range(0, n_cols, bc)]
    per = max(3, -(-n_min // len(tiles)))
    m_, r_, c_ = [], [], []
    for m, a, b in tiles:
        a1, b1 = min(n_rows, a + br), min(n_cols, b + bc)
        rr = [a, a1 - 1] + list(rng.integers(a, a1, per - 2))
        cc = [b, b1 - 1] + list(rng.integers(b, b1, per - 2))
        m_ += [m] * per; r_ += rr; c_ += cc
    for r in extra_rows:
        if 0 <= r < n_rows:
            cols = rng.integers(0, n_cols, 8)
            for m in range(t):
                m_ += [m] * 8; r_ += [r] * 8; c_ += list(cols)
    return np.array(m_, dtype=np.int64), np.array(r_, dtype=np.int64), np.array(c_, dtype=np.int64)
