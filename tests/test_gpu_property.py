"""Property test of the layer against the fp64 oracle over drawn shapes (hypothesis, derandomised: the same
examples on every run): ranks, token counts from one to a few hundred (several row tiles and a ragged tail, and the
few-token path), hidden sizes and shard widths on and off the tensor-core path's alignment, any partition 0 <= S <= h
(on a tile edge, off it, not a multiple of 8), both norms, scaling on and off, bf16 and fp32.  Forward and backward
through the C ABI with canary-padded outputs.  Needs a GPU."""
import math

import numpy as np
import pytest
import torch
from hypothesis import HealthCheck, given, settings
from hypothesis import strategies as st

from paper_2506_19645_b200 import caat, synthetic
from tests import gpu_harness as G
from tests.helpers import TOL, assert_close, f64

pytestmark = pytest.mark.gpu


@st.composite
def layer_case(draw):
    t = draw(st.sampled_from([1, 2, 3, 4, 8]))
    dtype = draw(st.sampled_from(["bf16", "bf16", "f32"]))
    h = 8 * t * draw(st.integers(1, 24 if dtype == "bf16" else 8))          # h % 8 == 0 and t | h
    k_r = draw(st.sampled_from([8, 24, 40, 64, 72, 128, 200]))              # multiples of 8: tensor-core path when S % 8 == 0
    if draw(st.booleans()):
        k_r += draw(st.sampled_from([1, 3, 4]))                             # off the alignment: CUDA-core GEMM
    T = draw(st.one_of(st.integers(1, 8), st.integers(9, 64), st.integers(65, 400)))
    S = draw(st.one_of(st.sampled_from([0, h]), st.integers(0, h), st.integers(0, h // 8).map(lambda q: 8 * q)))
    norm = draw(st.sampled_from([0, 1]))
    alpha = draw(st.sampled_from([None, 1.0]))                              # None: the default sqrt(t)
    seed = draw(st.integers(0, 2 ** 16))
    return t, dtype, h, k_r, T, S, norm, alpha, seed


# rows: the row-kernel family (0 = the library's choice, which is the warp-per-token kernels at these row lengths;
# 2 = the bulk-copy staged kernels and, where the partition falls on a multiple of 8, their lean backward)
@pytest.mark.parametrize("rows", [0, 2])
@settings(max_examples=100, deadline=None, derandomize=True, suppress_health_check=list(HealthCheck))
@given(layer_case())
def test_forward_and_backward_match_the_oracle(rows, case):
    t, dtype, h, k_r, T, S, norm, alpha, seed = case
    ffn = k_r * t                                                            # the MLP-down layer carries the drawn shard width
    ctx = G.make_ctx(t, h, ffn, dtype, S=S, alpha=alpha, norm=norm, direct_rows=rows)
    assert ctx.shared_channels == S and ctx.k_r(caat.CAAT_MLP_DOWN) == k_r
    assert ctx.private_scale == pytest.approx(1.0 if alpha == 1.0 else math.sqrt(t))
    d = synthetic.layer_inputs(t, T, h, k_r, dtype, seed=seed, S=S, backward=True, tied_residual=bool(seed & 1))
    g = torch.Generator().manual_seed(seed + 1)
    td = synthetic.torch_dtype(dtype)
    d["gamma"] = (1 + 0.1 * torch.randn(h, generator=g)).to(td)
    d["beta"] = (0.1 * torch.randn(h, generator=g)).to(td)
    where = f"rows={rows} t={t} {dtype} h={h} K_r={k_r} T={T} S={S} norm={norm} alpha={alpha}"
    gf = G.gpu_forward(ctx, caat.CAAT_MLP_DOWN, d)
    of = G.oracle_forward(ctx, d)
    for k in ("Hn", "X", "rstd"):
        assert_close(gf[k], of[k], dtype, f"{where}: {k}")
    if norm:   # a row's mean can be any small number: its error is judged against the row's spread, 1 / rstd
        scaled = lambda m: np.asarray(f64(m) if isinstance(m, torch.Tensor) else m, dtype=np.float64) * np.asarray(of["rstd"], dtype=np.float64)
        assert np.abs(scaled(gf["mean"]) - scaled(of["mean"])).max() <= TOL[dtype], f"{where}: mean"
    Hn, rstd, mean = G.saved_from_oracle(ctx, of)
    with_dHn = bool(seed & 2)
    gb = G.gpu_backward(ctx, caat.CAAT_MLP_DOWN, d, Hn, rstd, mean, with_dHn=with_dHn)
    ob = G.oracle_backward(ctx, d, Hn, rstd, mean, with_dHn=with_dHn)
    for k in ("dR", "dgamma") + (("dbeta",) if norm else ()):
        assert_close(gb[k], ob[k], dtype, f"{where}: {k}")
    # dY and dW contract the gradient AS STORED (rounded to the storage type, unit roundoff u) with Y or W.  With a
    # handful of tokens or channels an entry is a sum of few terms that may cancel, and the error metric's rms floor is
    # then no measure of it; what the arithmetic guarantees is the forward error bound of a dot product with one rounded
    # operand, |error| <= 2u * sum |g| |operand| per entry (2u: the shared slab is rounded once more after the rank
    # sum).  An entry passes on either criterion; a dropped term or a wrong index breaks both.
    u = 2.0 ** -9 if dtype == "bf16" else 2.0 ** -24
    a_ = 1.0 if alpha == 1.0 else math.sqrt(t)
    g = np.asarray(ob["dR"], dtype=np.float64)                                # [t, T, h], the oracle's unrounded gradient
    G_ = np.concatenate([np.broadcast_to(np.abs(g[:, :, :S]).sum(0), (t, T, S)), a_ * np.abs(g[:, :, S:])], axis=2)
    bound = {"dY": np.einsum("mil,mlk->mik", G_, np.abs(f64(d["W"]))), "dW": np.einsum("mil,mik->mlk", G_, np.abs(f64(d["Y"])))}
    for k in ("dY", "dW"):
        a, b = f64(gb[k]), np.asarray(ob[k], dtype=np.float64)
        rms = math.sqrt(float(np.mean(b * b))) if b.size else 0.0
        ok = (np.abs(a - b) <= TOL[dtype] * np.maximum(np.abs(b), max(rms, 1e-30))) | (np.abs(a - b) <= 2 * u * bound[k] + 1e-6 * rms)
        assert np.all(np.isfinite(a)) and bool(ok.all()), f"{where}: {k}: {int((~ok).sum())} entries outside both criteria"
