"""Numerics of the backward rank sum (Section 4: the sum is accumulated in fp32).

The library's switch CAAT_OPT_BACKWARD_REDUCE selects how the shared channels' gradients of the
ranks are combined: 0 fp32 sum of the terms as computed (default), 1 terms rounded to bf16 first
(a 16-bit payload) and summed in fp32, 2 rounded terms and a bf16 running sum.  Each mode is checked
against the oracle's model of the same scheme, and the three are compared with the exact sum as the
number of ranks grows.  Run with -s to see the table.  Needs a GPU."""
import numpy as np
import pytest
import torch

from paper_2506_19645_b200 import caat, synthetic
from tests import gpu_harness as G
from tests.helpers import assert_close, f64

pytestmark = pytest.mark.gpu


def _case(t, T=256, h=512, seed=0):
    S = h // 2
    ctx_shapes = (t, h, 4 * h)
    d = synthetic.layer_inputs(t, T, h, h // t, dtype="bf16", seed=seed, S=S, backward=True)
    return ctx_shapes, S, d


@pytest.mark.parametrize("mode", [1, 2])
@pytest.mark.parametrize("t", [2, 8])
def test_reduce_modes_match_their_model(mode, t):
    (t_, h, ffn), S, d = _case(t, seed=t)
    ctx = G.make_ctx(t_, h, ffn, "bf16", S=S, bwd_reduce=mode)
    fo = G.oracle_forward(ctx, d)
    Hn, rstd, mean = G.saved_from_oracle(ctx, fo)
    gb = G.gpu_backward(ctx, caat.CAAT_ATTN_OUT, d, Hn, rstd, mean)
    ob = G.oracle_backward(ctx, d, Hn, rstd, mean)
    for k in ("dY", "dW", "dR", "dgamma"):
        assert_close(gb[k], ob[k], "bf16", k)


def test_fp32_accumulation_beats_16_bit_sums_and_the_gap_grows_with_ranks():
    rows = []
    for t in (2, 4, 8, 16, 32):
        (t_, h, ffn), S, d = _case(t, seed=100 + t)
        # the exact gradient: the oracle, no rounding model
        ctx0 = G.make_ctx(t_, h, ffn, "bf16", S=S)
        fo = G.oracle_forward(ctx0, d)
        Hn, rstd, mean = G.saved_from_oracle(ctx0, fo)
        exact = G.oracle_backward(ctx0, d, Hn, rstd, mean)["dZt"][0, :, :S]     # the shared channels' sum
        scale = np.sqrt(np.mean(exact ** 2))
        errs = []
        for mode in (0, 1, 2):
            ctx = G.make_ctx(t_, h, ffn, "bf16", S=S, bwd_reduce=mode, force_simt=True)
            # dW of the shared rows is linear in the shared sum; recover the sum itself from dY instead:
            # with W = identity on the shared block the data gradient's first S columns ARE the sum
            dd = dict(d)
            W = torch.zeros_like(d["W"])
            k = W.shape[2]
            for m in range(t_):
                W[m, m * k:(m + 1) * k, :] = torch.eye(k, dtype=W.dtype)       # rank m exposes channels [m k, (m+1) k)
            dd["W"] = W
            gb = G.gpu_backward(ctx, caat.CAAT_ATTN_OUT, dd, Hn, rstd, mean)
            got = np.concatenate([f64(gb["dY"][m]) for m in range(t_)], axis=1)[:, :S]   # [T, S]: stored bf16
            errs.append(float(np.sqrt(np.mean((got - exact) ** 2)) / scale))
        rows.append((t, *errs))
    print("\n  t   fp32 sum   bf16 terms, fp32 sum   bf16 terms, bf16 sum   (rms error of the shared gradient / its rms;"
          " every result is stored in bf16, which alone costs about 1.7e-3)")
    for t, e0, e1, e2 in rows:
        print(f"{t:3d}   {e0:.3e}      {e1:.3e}               {e2:.3e}")
    for t, e0, e1, e2 in rows:
        assert e0 <= e1 * 1.05 and e1 <= e2 * 1.05
    # the 16-bit running sum degrades with the number of ranks; fp32 accumulation does not
    assert rows[-1][3] > 2.0 * rows[0][3]
    assert rows[-1][1] < 1.5 * rows[0][1]
    assert rows[-1][3] > 3.0 * rows[-1][1]
