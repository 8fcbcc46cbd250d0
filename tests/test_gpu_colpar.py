"""Parity of the column-parallel half (pre = X A^T per rank, plain / SiLU / SwiGLU) and of the whole
CAAT MLP (column-parallel half, then the row-parallel layer with partial channel-reduce) with the fp64
oracle, through the C ABI.  Needs a GPU."""
import numpy as np
import pytest
import torch

from oracle import caat_oracle as O
from paper_2506_19645_b200 import caat, synthetic
from tests import gpu_harness as G
from tests.helpers import assert_close, f64, to_dtype

pytestmark = pytest.mark.gpu

ACTS = {"none": (caat.CAAT_ACT_NONE, O.ACT_NONE), "silu": (caat.CAAT_ACT_SILU, O.ACT_SILU),
        "swiglu": (caat.CAAT_ACT_SWIGLU, O.ACT_SWIGLU)}


def _inputs(t, T, h, n_out, dtype, seed, act):
    td = synthetic.torch_dtype(dtype)
    g = torch.Generator().manual_seed(seed)
    wy = n_out // 2 if act == "swiglu" else n_out
    return {"X": torch.randn((t, T, h), generator=g).to(td),
            "A": (torch.randn((t, n_out, h), generator=g) * (1.0 / np.sqrt(h))).to(td),
            "dY": torch.randn((t, T, wy), generator=g).to(td)}


def _colpar_gpu(ctx, act, n_out, d, pre_saved=None):
    t, h, td = ctx.t, ctx.h, ctx.torch_dtype
    T = d["X"].shape[1]
    wy = d["dY"].shape[2]
    cact = ACTS[act][0]
    pre, Y = G.Guarded((t, T, n_out), td), (G.Guarded((t, T, wy), td) if act != "none" else None)
    ctx.colpar_forward(cact, n_out, T, d["X"].cuda(), d["A"].cuda(), pre.view, Y.view if Y else None)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    pre.check("pre")
    if Y:
        Y.check("Y")
    fwd = {"pre": pre.view.cpu(), "Y": (Y.view if Y else pre.view).cpu()}
    dX, dA = G.Guarded((t, T, h), td), G.Guarded((t, n_out, h), torch.float32)
    ws = ctx.alloc_workspace(ctx.colpar_workspace_bytes(cact, n_out, T))
    ctx.colpar_backward(cact, n_out, T, d["dY"].cuda(), d["X"].cuda(), d["A"].cuda(),
                        (pre_saved if pre_saved is not None else fwd["pre"]).cuda(), dX.view, dA.view, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    dX.check("dX"); dA.check("dA")
    return fwd, {"dX": dX.view.cpu(), "dA": dA.view.cpu()}


@pytest.mark.parametrize("act", ["none", "silu", "swiglu"])
@pytest.mark.parametrize("t,T,h,n_out,dtype,simt", [
    (4, 300, 768, 1536, "bf16", False),     # 130M MLP: gate|up of ffn/t = 768
    (8, 257, 2048, 1408, "bf16", False),    # 1.1B MLP: 2 x 704
    (8, 130, 4096, 1536, "bf16", False),    # 7B QKV width 3 h / t
    (2, 70, 256, 1024, "f32", False),       # fp32 runs on the CUDA-core GEMM
    (3, 45, 264, 176, "bf16", True),        # forced CUDA-core GEMM in bf16
    (8, 5000, 1024, 512, "bf16", False),    # many tokens, persistent CTAs walk many tiles
])
def test_colpar_forward_backward(act, t, T, h, n_out, dtype, simt):
    ctx = G.make_ctx(t, h, 4 * h, dtype, force_simt=simt)
    d = _inputs(t, T, h, n_out, dtype, seed=T + n_out, act=act)
    of = O.colpar_forward(f64(d["X"]), f64(d["A"]), ACTS[act][1])
    pre_saved = to_dtype(of["pre"], ctx.torch_dtype)          # the backward runs on the oracle's saved pre, rounded
    ob = O.colpar_backward(f64(d["dY"]), f64(d["X"]), f64(d["A"]), f64(pre_saved), ACTS[act][1])
    gf, gb = _colpar_gpu(ctx, act, n_out, d, pre_saved)
    assert_close(gf["pre"], of["pre"], dtype, "pre")
    assert_close(gf["Y"], of["Y"], dtype, "Y")
    assert_close(gb["dX"], ob["dX"], dtype, "dX")
    assert_close(gb["dA"], ob["dA"], dtype, "dA")


def test_colpar_rejects_bad_widths():
    ctx = G.make_ctx(2, 256, 1024, "bf16")
    d = _inputs(2, 16, 256, 24, "bf16", 1, "swiglu")      # 24 is not a multiple of 16
    with pytest.raises(caat.CaatError) as e:
        _colpar_gpu(ctx, "swiglu", 24, d)
    assert e.value.status == caat.CAAT_EUNSUPPORTED


def test_whole_mlp_with_partial_channel_reduce():
    # X -> [gate | up] -> SwiGLU -> row-parallel down projection with reduce, scaling, residual, norm (Eq. A3),
    # and the gradient of all of it; the two library calls are chained exactly as a network would chain them
    t, T, h, ffn, S = 4, 300, 768, 3072, 384
    F = ffn // t
    ctx = G.make_ctx(t, h, ffn, "bf16", S=S)
    alpha = ctx.private_scale
    g = torch.Generator().manual_seed(77)
    bf = torch.bfloat16
    d = {"X": torch.randn((t, T, h), generator=g).to(bf), "A": (torch.randn((t, 2 * F, h), generator=g) / np.sqrt(h)).to(bf),
         "B": (torch.randn((t, h, F), generator=g) * 0.02).to(bf), "R": torch.randn((t, T, h), generator=g).to(bf),
         "gamma": (1 + 0.1 * torch.randn(h, generator=g)).to(bf),
         "dXout": torch.randn((t, T, h), generator=g).to(bf), "dHn": torch.randn((t, T, h), generator=g).to(bf)}
    synthetic.tie_shared_channels(d["R"], S)
    of = O.mlp_forward(f64(d["X"]), f64(d["A"]), f64(d["B"]), f64(d["R"]), f64(d["gamma"]), S=S, alpha=alpha)
    c = {k: v.cuda() for k, v in d.items()}
    mk = lambda *s, dt=bf: torch.empty(*s, dtype=dt, device="cuda")
    pre, Y, Hn, Xo, rstd = mk(t, T, 2 * F), mk(t, T, F), mk(t, T, h), mk(t, T, h), mk(t, T, dt=torch.float32)
    ws = ctx.alloc_workspace(max(ctx.workspace_bytes(caat.CAAT_MLP_DOWN, T, True),
                                 ctx.colpar_workspace_bytes(caat.CAAT_ACT_SWIGLU, 2 * F, T)))
    ctx.colpar_forward(caat.CAAT_ACT_SWIGLU, 2 * F, T, c["X"], c["A"], pre, Y)
    ctx.rowpar_forward(caat.CAAT_MLP_DOWN, T, Y, c["B"], c["R"], c["gamma"], None, Hn, Xo, rstd, None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    for k, v in (("pre", pre), ("Y", Y), ("Hn", Hn), ("X", Xo), ("rstd", rstd)):
        assert_close(v.cpu(), of[k], "bf16", k)
    # backward on the oracle's saved tensors (rounded to their storage types)
    sv = {k: to_dtype(of[k], bf) for k in ("pre", "Y", "Hn")}
    sv["rstd"] = to_dtype(of["rstd"], torch.float32)
    ob = O.mlp_backward(f64(d["dXout"]), f64(d["dHn"]), f64(d["X"]), f64(d["A"]), f64(d["B"]), f64(sv["pre"]), f64(sv["Y"]),
                        f64(sv["Hn"]), f64(sv["rstd"]), None, f64(d["gamma"]), S=S, alpha=alpha)
    dY, dB, dR, dg = mk(t, T, F), mk(t, h, F, dt=torch.float32), mk(t, T, h), mk(h, dt=torch.float32)
    dX, dA = mk(t, T, h), mk(t, 2 * F, h, dt=torch.float32)
    ctx.rowpar_backward(caat.CAAT_MLP_DOWN, T, c["dXout"], c["dHn"], sv["Y"].cuda(), c["B"], sv["Hn"].cuda(),
                        sv["rstd"].cuda(), None, c["gamma"], dY, dB, dR, dg, None, ws)
    ctx.colpar_backward(caat.CAAT_ACT_SWIGLU, 2 * F, T, dY, c["X"], c["A"], sv["pre"].cuda(), dX, dA, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    # dX and dA see the library's own dY (rounded to bf16), the oracle its exact one: one storage rounding apart
    for k, v in (("dX", dX), ("dA", dA), ("dB", dB), ("dR", dR), ("dgamma", dg)):
        assert_close(v.cpu(), ob[k], "bf16", k)
