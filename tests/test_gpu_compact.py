"""Parity of the compact-residual-layout entry points (shared part of the stream stored once)
with the fp64 oracle's compact functions, through the C ABI.  Needs a GPU."""
import numpy as np
import pytest
import torch

from oracle import caat_oracle as O
from paper_2506_19645_b200 import caat, synthetic
from tests import gpu_harness as G
from tests.helpers import assert_close, f64, to_dtype

pytestmark = pytest.mark.gpu


def _split(x, S):
    """[t, T, h] -> shared part of rank 0 [T, S] and private parts [t, T, h - S] (views made contiguous)."""
    return x[0, :, :S].contiguous(), x[:, :, S:].contiguous()


def _case(t, T, h, k, dtype, S, seed, norm):
    d = synthetic.layer_inputs(t, T, h, k, dtype=dtype, seed=seed, S=S, backward=True)
    g = torch.Generator().manual_seed(seed + 100)
    td = d["Y"].dtype
    d["gamma"] = (1 + 0.1 * torch.randn(h, generator=g)).to(td)
    d["beta"] = (0.1 * torch.randn(h, generator=g)).to(td) if norm == 1 else None
    d["Rs"], d["Rp"] = _split(d["R"], S)
    d["dHns"], d["dHnp"] = _split(d["dHn"], S)
    return d


def _oracle_fwd(ctx, d):
    return O.rowpar_forward_compact(f64(d["Y"]), f64(d["W"]), f64(d["Rs"]), f64(d["Rp"]), f64(d["gamma"]),
                                    f64(d["beta"]) if d["beta"] is not None else None, S=ctx.shared_channels,
                                    alpha=ctx.private_scale, eps=1e-5, norm=ctx.norm)


def _gpu_fwd(ctx, layer, d):
    t, h, S, td = ctx.t, ctx.h, ctx.shared_channels, ctx.torch_dtype
    T = d["Y"].shape[1]
    Hns, Hnp, X = G.Guarded((T, S), td), G.Guarded((t, T, h - S), td), G.Guarded((t, T, h), td)
    rstd = G.Guarded((t, T), torch.float32)
    mean = G.Guarded((t, T), torch.float32) if ctx.norm == 1 else None
    ws = ctx.alloc_workspace(ctx.workspace_bytes(layer, T, False))
    ctx.rowpar_forward_compact(layer, T, d["Y"].cuda(), d["W"].cuda(), d["Rs"].cuda(), d["Rp"].cuda(), d["gamma"].cuda(),
                               d["beta"].cuda() if d["beta"] is not None else None, Hns.view, Hnp.view, X.view,
                               rstd.view, mean.view if mean else None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    for n, g in (("Hns", Hns), ("Hnp", Hnp), ("X", X), ("rstd", rstd), ("mean", mean)):
        if g is not None:
            g.check(n)
    return {"Hns": Hns.view.cpu(), "Hnp": Hnp.view.cpu(), "X": X.view.cpu(), "rstd": rstd.view.cpu(),
            "mean": mean.view.cpu() if mean else None}


def _check(ctx, layer, d, dtype, with_dh=True):
    t, h, S, td = ctx.t, ctx.h, ctx.shared_channels, ctx.torch_dtype
    T, k = d["Y"].shape[1], ctx.k_r(layer)
    fo = _oracle_fwd(ctx, d)
    go = _gpu_fwd(ctx, layer, d)
    for key in ("Hns", "Hnp", "X", "rstd") + (("mean",) if ctx.norm == 1 else ()):
        if fo[key].size:
            assert_close(go[key], fo[key], dtype, key)
    # backward on the oracle's saved tensors, rounded to their storage types
    Hns, Hnp = to_dtype(fo["Hns"], td), to_dtype(fo["Hnp"], td)
    rstd = to_dtype(fo["rstd"], torch.float32)
    mean = to_dtype(fo["mean"], torch.float32) if fo["mean"] is not None else None
    ob = O.rowpar_backward_compact(f64(d["dX"]), f64(d["dHns"]) if with_dh else None, f64(d["dHnp"]) if with_dh else None,
                                   f64(d["Y"]), f64(d["W"]), f64(Hns), f64(Hnp), f64(rstd),
                                   f64(mean) if mean is not None else None, f64(d["gamma"]), S=S,
                                   alpha=ctx.private_scale, norm=ctx.norm)
    out = {"dY": G.Guarded((t, T, k), td), "dW": G.Guarded((t, h, k), torch.float32), "dRs": G.Guarded((T, S), td),
           "dRp": G.Guarded((t, T, h - S), td), "dgamma": G.Guarded((h,), torch.float32),
           "dbeta": G.Guarded((h,), torch.float32) if ctx.norm == 1 else None}
    ws = ctx.alloc_workspace(ctx.workspace_bytes(layer, T, True))
    ctx.rowpar_backward_compact(layer, T, d["dX"].cuda(), d["dHns"].cuda() if with_dh else None,
                                d["dHnp"].cuda() if with_dh else None, d["Y"].cuda(), d["W"].cuda(), Hns.cuda(), Hnp.cuda(),
                                rstd.cuda(), mean.cuda() if mean is not None else None, d["gamma"].cuda(),
                                out["dY"].view, out["dW"].view, out["dRs"].view, out["dRp"].view, out["dgamma"].view,
                                out["dbeta"].view if out["dbeta"] else None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    for key, g in out.items():
        if g is None:
            continue
        g.check(key)
        if ob[key].size:
            assert_close(g.view.cpu(), ob[key], dtype, key)


@pytest.mark.parametrize("direct_rows", [0, 1, 2])
@pytest.mark.parametrize("t,T,h,ffn,layer,S,norm,dtype", [
    (4, 301, 768, 3072, caat.CAAT_ATTN_OUT, 384, 0, "bf16"),     # 130M shapes: warp-per-token rows
    (4, 2003, 768, 3072, caat.CAAT_MLP_DOWN, 192, 1, "bf16"),    # LayerNorm, persistent CTAs walk many groups
    (8, 200, 2048, 5632, caat.CAAT_ATTN_OUT, 1536, 0, "bf16"),   # 1.1B shapes, p = 0.75: staged rows
    (8, 77, 4096, 11008, caat.CAAT_ATTN_OUT, 2048, 0, "bf16"),   # 7B shapes
    (3, 45, 9216, 9216, caat.CAAT_ATTN_OUT, 4608, 1, "bf16"),    # four chunks per thread
    (2, 131, 256, 1024, caat.CAAT_MLP_DOWN, 104, 1, "f32"),      # fp32, S a multiple of 8 only
    (2, 64, 256, 1024, caat.CAAT_MLP_DOWN, 0, 0, "bf16"),        # p = 0: no shared part
    (2, 64, 256, 1024, caat.CAAT_MLP_DOWN, 256, 0, "bf16"),      # p = 1: no private part
    (16, 70, 512, 2048, caat.CAAT_ATTN_OUT, 256, 0, "bf16"),     # t = 16
    (8, 1, 1024, 4096, caat.CAAT_ATTN_OUT, 512, 0, "bf16"),      # a single token
])
def test_compact_forward_backward(direct_rows, t, T, h, ffn, layer, S, norm, dtype):
    ctx = G.make_ctx(t, h, ffn, dtype, S=S, norm=norm, direct_rows=direct_rows)
    d = _case(t, T, h, ctx.k_r(layer), dtype, S, seed=T, norm=norm)
    _check(ctx, layer, d, dtype)


def test_compact_no_stream_gradient_and_alpha_one():
    ctx = G.make_ctx(4, 768, 3072, "bf16", S=384, alpha=1.0)
    d = _case(4, 96, 768, 768, "bf16", 384, seed=9, norm=0)
    _check(ctx, caat.CAAT_MLP_DOWN, d, "bf16", with_dh=False)


@pytest.mark.parametrize("S", [0, 8, 256, 504, 512])
def test_compact_partition_bit_exact_integer_inputs(S):
    # small integers: every product, rank sum and residual add is exact, so both parts of the new
    # stream must equal the oracle's bit for bit wherever the boundary lies
    t, T, h, K_r = 4, 70, 512, 16
    R = synthetic.small_integers((t, T, h), -8, 8, seed=S + 2)
    d = {"Y": synthetic.small_integers((t, T, K_r), -2, 2, seed=S), "W": synthetic.small_integers((t, h, K_r), -1, 1, seed=S + 1),
         "gamma": torch.ones(h).bfloat16(), "beta": None}
    d["Rs"], d["Rp"] = _split(R, S)
    for alpha in (1.0, 2.0):
        ctx = G.make_ctx(t, h, t * K_r, "bf16", S=S, alpha=alpha)
        go, fo = _gpu_fwd(ctx, caat.CAAT_MLP_DOWN, d), _oracle_fwd(ctx, d)
        assert np.array_equal(f64(go["Hns"]), fo["Hns"]) and np.array_equal(f64(go["Hnp"]), fo["Hnp"])


def test_compact_rejects_unaligned_partition():
    ctx = G.make_ctx(2, 256, 1024, "bf16", S=100)
    d = _case(2, 16, 256, 512, "bf16", 100, seed=1, norm=0)
    with pytest.raises(caat.CaatError) as e:
        _gpu_fwd(ctx, caat.CAAT_MLP_DOWN, d)
    assert e.value.status == caat.CAAT_EUNSUPPORTED


def test_compact_block_matches_oracle():
    t, T, h, ffn, S = 4, 300, 768, 3072, 384
    w = synthetic.Workload("compact_block_case", t, T, h, ffn, 0.5, "bf16", "block", True, 31)
    d = synthetic.block_inputs(w, S)
    ctx = G.make_ctx(t, h, ffn, "bf16", S=S)
    td, f32, alpha = torch.bfloat16, torch.float32, ctx.private_scale
    R0s, R0p = _split(d["R0"], S)
    dHn2s, dHn2p = _split(d["dHn2"], S)
    fo = O.block_forward_compact(f64(d["Y_attn"]), f64(d["W_o"]), f64(d["Y_mlp"]), f64(d["W_down"]), f64(R0s), f64(R0p),
                                 f64(d["gamma1"]), f64(d["gamma2"]), S=S, alpha=alpha)
    mk = lambda *s, dt=td: torch.empty(*s, dtype=dt, device="cuda")
    out = {"Hn1s": mk(T, S), "Hn1p": mk(t, T, h - S), "X1": mk(t, T, h), "rstd1": mk(t, T, dt=f32),
           "Hn2s": mk(T, S), "Hn2p": mk(t, T, h - S), "X2": mk(t, T, h), "rstd2": mk(t, T, dt=f32)}
    ws = ctx.alloc_workspace(ctx.block_workspace_bytes(T, True))
    c = {k: v.cuda() for k, v in d.items()}
    ctx.block_forward_compact(T, c["Y_attn"], c["W_o"], c["Y_mlp"], c["W_down"], R0s.cuda(), R0p.cuda(), c["gamma1"], None,
                              c["gamma2"], None, out["Hn1s"], out["Hn1p"], out["X1"], out["rstd1"], None, out["Hn2s"],
                              out["Hn2p"], out["X2"], out["rstd2"], None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    for k in out:
        assert_close(out[k].cpu(), fo[k], "bf16", k)
    sv = {k: to_dtype(fo[k], td) for k in ("Hn1s", "Hn1p", "Hn2s", "Hn2p")}
    sv.update({k: to_dtype(fo[k], f32) for k in ("rstd1", "rstd2")})
    ob = O.block_backward_compact(f64(d["dX1"]), f64(d["dX2"]), f64(dHn2s), f64(dHn2p), f64(d["Y_attn"]), f64(d["W_o"]),
                                  f64(d["Y_mlp"]), f64(d["W_down"]), f64(sv["Hn1s"]), f64(sv["Hn1p"]), f64(sv["rstd1"]), None,
                                  f64(sv["Hn2s"]), f64(sv["Hn2p"]), f64(sv["rstd2"]), None, f64(d["gamma1"]), f64(d["gamma2"]),
                                  S=S, alpha=alpha)
    ka, km = h // t, ffn // t
    bo = {"dY_attn": mk(t, T, ka), "dW_o": mk(t, h, ka, dt=f32), "dY_mlp": mk(t, T, km), "dW_down": mk(t, h, km, dt=f32),
          "dR0s": mk(T, S), "dR0p": mk(t, T, h - S), "dHn1s": mk(T, S), "dHn1p": mk(t, T, h - S),
          "dgamma1": mk(h, dt=f32), "dgamma2": mk(h, dt=f32)}
    ctx.block_backward_compact(T, c["dX1"], c["dX2"], dHn2s.cuda(), dHn2p.cuda(), c["Y_attn"], c["W_o"], c["Y_mlp"],
                               c["W_down"], sv["Hn1s"].cuda(), sv["Hn1p"].cuda(), sv["rstd1"].cuda(), None,
                               sv["Hn2s"].cuda(), sv["Hn2p"].cuda(), sv["rstd2"].cuda(), None, c["gamma1"], c["gamma2"],
                               bo["dY_attn"], bo["dW_o"], bo["dY_mlp"], bo["dW_down"], bo["dR0s"], bo["dR0p"],
                               bo["dHn1s"], bo["dHn1p"], bo["dgamma1"], None, bo["dgamma2"], None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    # the layer-1 backward consumes the GPU's own dHn1 (rounded to bf16), the oracle its exact one:
    # the difference is one storage rounding, inside the tolerance
    for k in bo:
        assert_close(bo[k].cpu(), ob[k], "bf16", k)


@pytest.mark.parametrize("no_decode", [False, True])
@pytest.mark.parametrize("T,t,h,ffn,S", [(1, 8, 4096, 11008, 2048), (8, 8, 4096, 11008, 4096), (64, 8, 4096, 11008, 2048),
                                         (33, 4, 768, 3072, 384), (64, 2, 256, 1024, 0)])
def test_compact_block_few_tokens(no_decode, T, t, h, ffn, S):
    # few tokens: both layers' weights stream through one swapped-operand GEMM and one row kernel walks both layers of
    # a row, here on the compact stream; the large-batch path (no_decode) must give the same block
    w = synthetic.Workload("compact_decode_case", t, T, h, ffn, S / h, "bf16", "block", False, 7 + T)
    d = synthetic.block_inputs(w, S)
    ctx = G.make_ctx(t, h, ffn, "bf16", S=S, no_decode=no_decode)
    td, f32, alpha = torch.bfloat16, torch.float32, ctx.private_scale
    R0s, R0p = _split(d["R0"], S)
    fo = O.block_forward_compact(f64(d["Y_attn"]), f64(d["W_o"]), f64(d["Y_mlp"]), f64(d["W_down"]), f64(R0s), f64(R0p),
                                 f64(d["gamma1"]), f64(d["gamma2"]), S=S, alpha=alpha)
    out = {"Hn1s": G.Guarded((T, S), td), "Hn1p": G.Guarded((t, T, h - S), td), "X1": G.Guarded((t, T, h), td),
           "rstd1": G.Guarded((t, T), f32), "Hn2s": G.Guarded((T, S), td), "Hn2p": G.Guarded((t, T, h - S), td),
           "X2": G.Guarded((t, T, h), td), "rstd2": G.Guarded((t, T), f32)}
    ws = ctx.alloc_workspace(ctx.block_workspace_bytes(T, False))
    c = {k: v.cuda() for k, v in d.items()}
    ctx.block_forward_compact(T, c["Y_attn"], c["W_o"], c["Y_mlp"], c["W_down"], R0s.cuda(), R0p.cuda(), c["gamma1"], None,
                              c["gamma2"], None, out["Hn1s"].view, out["Hn1p"].view, out["X1"].view, out["rstd1"].view, None,
                              out["Hn2s"].view, out["Hn2p"].view, out["X2"].view, out["rstd2"].view, None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    for k, g in out.items():
        g.check(k)
        if fo[k].size:
            assert_close(g.view.cpu(), fo[k], "bf16", k)
