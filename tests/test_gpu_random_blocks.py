"""Block calls on shapes drawn from a seeded generator (the same cases on every run): ranks, hidden sizes whose rows
do and do not fill whole warps or tiles, any partition (on and off the tensor-core path's alignment), token counts on
both sides of the few-token threshold, every row-kernel family and block-forward schedule.  Forward and backward against
the fp64 oracle.  The fixed cases of the other test files pin the shapes the paper names; these pin the ones nobody
thought of (a sample of this kind found a deadlock of the two-layer few-token row kernel on rows of 16 chunks).
Needs a GPU."""
import random

import pytest
import torch

from oracle import caat_oracle as O
from paper_2506_19645_b200 import caat, synthetic
from tests import gpu_harness as G
from tests.helpers import assert_close, f64

pytestmark = [pytest.mark.gpu, pytest.mark.timeout(600)]


def _cases(n, seed):
    rng = random.Random(seed)
    out = []
    for _ in range(n):
        t = rng.choice([1, 2, 4, 8])
        h = 8 * t * rng.randint(1, 24)
        ffn = h * rng.choice([2, 3, 4])
        p = rng.choice([0.0, 0.25, 0.5, 0.75, 1.0, round(rng.random(), 3)])
        T = rng.choice([rng.randint(1, 64), rng.randint(65, 300), rng.randint(301, 900)])
        out.append((t, T, h, ffn, p, rng.choice([0, 0, 1, 2]), rng.choice([0, 1, 2])))
    return out


@pytest.mark.parametrize("t,T,h,ffn,p,rows,overlap", _cases(40, seed=2506))
def test_block_forward_and_backward_on_drawn_shapes(t, T, h, ffn, p, rows, overlap):
    w = synthetic.Workload("drawn", t, T, h, ffn, p, "bf16", "block", True, 7)
    d = synthetic.block_inputs(w, O.shared_channels(h, p))
    ctx = G.make_ctx(t, h, ffn, "bf16", p=p, direct_rows=rows)
    ctx.set_option(caat.CAAT_OPT_BLOCK_OVERLAP, overlap)
    S, alpha = ctx.shared_channels, ctx.private_scale
    assert S == O.shared_channels(h, p)
    dev = {k: v.cuda() for k, v in d.items()}
    mk = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt, device="cuda")
    f32 = torch.float32
    Hn1, X1, Hn2, X2 = (mk(t, T, h) for _ in range(4))
    rstd1, rstd2 = mk(t, T, dt=f32), mk(t, T, dt=f32)
    ws = ctx.alloc_workspace(ctx.block_workspace_bytes(T, True))
    ctx.block_forward(T, dev["Y_attn"], dev["W_o"], dev["Y_mlp"], dev["W_down"], dev["R0"], dev["gamma1"], None,
                      dev["gamma2"], None, Hn1, X1, rstd1, None, Hn2, X2, rstd2, None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    fo = O.block_forward(f64(d["Y_attn"]), f64(d["W_o"]), f64(d["Y_mlp"]), f64(d["W_down"]), f64(d["R0"]),
                         f64(d["gamma1"]), f64(d["gamma2"]), S=S, alpha=alpha)
    for name, g in (("Hn1", Hn1), ("X1", X1), ("rstd1", rstd1), ("rstd2", rstd2)):
        assert_close(g, fo[name], "bf16", name)
    # The second layer adds to the stream AS STORED: a stream value of 4-5 sigma carries a rounding error of 2^-9 of
    # itself, and where the layer output cancels most of it that error stands against a small result.  So the second
    # layer is judged at the tolerance against the oracle's layer applied to the stored stream, and against the oracle's
    # unrounded chain at one and a half times the tolerance.
    f2 = O.rowpar_forward(f64(d["Y_mlp"]), f64(d["W_down"]), f64(Hn1), f64(d["gamma2"]), None, S=S, alpha=alpha)
    for name, g, key in (("Hn2", Hn2, "Hn"), ("X2", X2, "X")):
        assert_close(g, f2[key], "bf16", f"{name} (second layer on the stored stream)")
        assert_close(g, fo[name], "bf16", f"{name} (unrounded chain)", scale=1.5)
    # backward on the oracle's saved tensors, rounded to their storage types
    sHn1, sHn2 = (torch.from_numpy(fo[k]).bfloat16() for k in ("Hn1", "Hn2"))
    sr1, sr2 = (torch.from_numpy(fo[k]).float() for k in ("rstd1", "rstd2"))
    ka, km = ctx.k_r(caat.CAAT_ATTN_OUT), ctx.k_r(caat.CAAT_MLP_DOWN)
    dYa, dYm, dR0, dHn1 = mk(t, T, ka), mk(t, T, km), mk(t, T, h), mk(t, T, h)
    dWo, dWd = mk(t, h, ka, dt=f32), mk(t, h, km, dt=f32)
    dg1, dg2 = mk(h, dt=f32), mk(h, dt=f32)
    ctx.block_backward(T, dev["dX1"], dev["dX2"], dev["dHn2"], dev["Y_attn"], dev["W_o"], dev["Y_mlp"], dev["W_down"],
                       sHn1.cuda(), sr1.cuda(), None, sHn2.cuda(), sr2.cuda(), None, dev["gamma1"], dev["gamma2"],
                       dYa, dWo, dYm, dWd, dR0, dHn1, dg1, None, dg2, None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    ob = O.block_backward(f64(d["dX1"]), f64(d["dX2"]), f64(d["dHn2"]), f64(d["Y_attn"]), f64(d["W_o"]),
                          f64(d["Y_mlp"]), f64(d["W_down"]), f64(sHn1), f64(sr1), None, f64(sHn2), f64(sr2), None,
                          f64(d["gamma1"]), f64(d["gamma2"]), S=S, alpha=alpha)
    # a weight gradient over a handful of tokens is a sum of few, possibly cancelling, terms of a gradient stored in
    # bf16: the metric's rms floor then stops measuring the arithmetic (tests/test_gpu_property.py has the bound)
    few = 2.0 if T < 40 else 1.0
    for name, g in (("dY_attn", dYa), ("dW_o", dWo), ("dY_mlp", dYm), ("dW_down", dWd), ("dR0", dR0),
                    ("dHn1", dHn1), ("dgamma1", dg1), ("dgamma2", dg2)):
        assert_close(g, ob[name], "bf16", name, scale=few if name.startswith("dW") else 1.0)
