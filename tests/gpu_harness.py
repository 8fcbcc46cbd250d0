"""Runs the CUDA path through the binding and the fp64 oracle on the same inputs.

Harness only: it rounds inputs/saved tensors to the storage type, moves them to the
device and collects outputs.  All arithmetic of the method happens either in the
library (GPU) or in ``oracle/`` (CPU)."""
import math

import numpy as np
import torch

from oracle import caat_oracle as O
from paper_2506_19645_b200 import caat
from tests.helpers import f64, to_dtype

GUARD = 64  # canary elements after every output buffer


def make_ctx(t, h, ffn, dtype, S=None, p=0.5, alpha=None, norm=0, eps=None, force_simt=False, direct_rows=False, no_decode=False,
             bwd_reduce=0):
    ctx = caat.Context(h, ffn, t, p, dtype)
    if S is not None:
        ctx.set_option(caat.CAAT_OPT_SHARED_CHANNELS, S)
    if alpha is not None:
        ctx.set_option(caat.CAAT_OPT_PRIVATE_SCALE, alpha)
    if norm:
        ctx.set_option(caat.CAAT_OPT_NORM, norm)
    ctx._eps = 1e-5
    if eps is not None:
        ctx.set_option(caat.CAAT_OPT_EPS, eps)
        ctx._eps = eps
    if force_simt:
        ctx.set_option(caat.CAAT_OPT_GEMM, 1)
    if direct_rows:
        ctx.set_option(caat.CAAT_OPT_ROWS, int(direct_rows))
    if no_decode:
        ctx.set_option(caat.CAAT_OPT_DECODE, 1)
    if bwd_reduce:
        ctx.set_option(caat.CAAT_OPT_BACKWARD_REDUCE, bwd_reduce)
    ctx._bwd_reduce = bwd_reduce
    return ctx


class Guarded:
    """An output tensor followed by canary elements that the library must not touch."""

    def __init__(self, shape, dtype, device="cuda"):
        n = int(np.prod(shape))
        pad = (-n) % 8          # keep the canaries' start 16-byte aligned friendly
        self.flat = torch.full((n + pad + GUARD,), 77.0, dtype=dtype, device=device)
        self.n = n
        self.view = self.flat[:n].view(shape)

    def check(self, name):
        tail = self.flat[self.n:]
        assert bool((tail == 77.0).all()), f"{name}: wrote past the end of the buffer"


def gpu_forward(ctx, layer, d, guard=True):
    """d: dict of CPU tensors Y, W, R, gamma, beta(optional).  Returns dict of CPU tensors."""
    T = d["Y"].shape[1]
    dev = {k: (v.cuda() if isinstance(v, torch.Tensor) else None) for k, v in d.items()}
    td, t, h = ctx.torch_dtype, ctx.t, ctx.h
    Hn, X = Guarded((t, T, h), td), Guarded((t, T, h), td)
    rstd = Guarded((t, T), torch.float32)
    mean = Guarded((t, T), torch.float32) if ctx.norm == caat.LAYERNORM else None
    ws = ctx.alloc_workspace(ctx.workspace_bytes(layer, T, False))
    ctx.rowpar_forward(layer, T, dev["Y"], dev["W"], dev["R"], dev["gamma"],
                       dev.get("beta") if ctx.norm == caat.LAYERNORM else None,
                       Hn.view, X.view, rstd.view, mean.view if mean else None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    for n, g in (("Hn", Hn), ("X", X), ("rstd", rstd), ("mean", mean)):
        if g is not None and guard:
            g.check(n)
    return {"Hn": Hn.view.cpu(), "X": X.view.cpu(), "rstd": rstd.view.cpu(),
            "mean": mean.view.cpu() if mean else None}


def oracle_forward(ctx, d):
    return O.rowpar_forward(f64(d["Y"]), f64(d["W"]), f64(d["R"]), f64(d["gamma"]),
                            f64(d["beta"]) if (ctx.norm == caat.LAYERNORM and d.get("beta") is not None) else None,
                            S=ctx.shared_channels, alpha=ctx.private_scale,
                            eps=getattr(ctx, "_eps", 1e-5), norm=ctx.norm)


def saved_from_oracle(ctx, fo):
    """Saved tensors for the backward: the oracle's forward results rounded to the storage
    types the forward writes (Hn in the run dtype, statistics in fp32)."""
    Hn = to_dtype(fo["Hn"], ctx.torch_dtype)
    rstd = to_dtype(fo["rstd"], torch.float32)
    mean = to_dtype(fo["mean"], torch.float32) if fo["mean"] is not None else None
    return Hn, rstd, mean


def gpu_backward(ctx, layer, d, Hn, rstd, mean, with_dHn=True):
    T = d["Y"].shape[1]
    td, t, h, k = ctx.torch_dtype, ctx.t, ctx.h, ctx.k_r(layer)
    dY, dR = Guarded((t, T, k), td), Guarded((t, T, h), td)
    dW = Guarded((t, h, k), torch.float32)
    dg = Guarded((h,), torch.float32)
    db = Guarded((h,), torch.float32) if ctx.norm == caat.LAYERNORM else None
    ws = ctx.alloc_workspace(ctx.workspace_bytes(layer, T, True))
    ctx.rowpar_backward(layer, T, d["dX"].cuda(), d["dHn"].cuda() if with_dHn else None, d["Y"].cuda(),
                        d["W"].cuda(), Hn.cuda(), rstd.cuda(), mean.cuda() if mean is not None else None,
                        d["gamma"].cuda(), dY.view, dW.view, dR.view, dg.view, db.view if db else None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    for n, g in (("dY", dY), ("dW", dW), ("dR", dR), ("dgamma", dg), ("dbeta", db)):
        if g is not None:
            g.check(n)
    return {"dY": dY.view.cpu(), "dW": dW.view.cpu(), "dR": dR.view.cpu(), "dgamma": dg.view.cpu(),
            "dbeta": db.view.cpu() if db else None}


def oracle_backward(ctx, d, Hn, rstd, mean, with_dHn=True):
    return O.rowpar_backward(f64(d["dX"]), f64(d["dHn"]) if with_dHn else None, f64(d["Y"]), f64(d["W"]),
                             f64(Hn), f64(rstd), f64(mean) if mean is not None else None, f64(d["gamma"]),
                             S=ctx.shared_channels, alpha=ctx.private_scale, norm=ctx.norm,
                             reduce_mode=getattr(ctx, "_bwd_reduce", 0))
