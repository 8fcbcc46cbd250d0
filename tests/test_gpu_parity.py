"""Parity of the CUDA path (through the C ABI) with the fp64 oracle, element by element,
on seeded synthetic inputs.  Needs a GPU."""
import math

import numpy as np
import pytest
import torch

from oracle import caat_oracle as O
from paper_2506_19645_b200 import caat, synthetic
from tests import gpu_harness as G
from tests.helpers import TOL, assert_close, f64

pytestmark = pytest.mark.gpu


def _layer_case(t, T, h, K_r, dtype, S, seed=0, backward=False, tied=True):
    return synthetic.layer_inputs(t, T, h, K_r, dtype=dtype, seed=seed, S=S, backward=backward, tied_residual=tied)


def _check_forward(ctx, layer, d, dtype):
    go = G.gpu_forward(ctx, layer, d)
    fo = G.oracle_forward(ctx, d)
    errs = {k: assert_close(go[k], fo[k], dtype, k) for k in ("Hn", "X", "rstd")}
    if ctx.norm == caat.LAYERNORM:
        errs["mean"] = assert_close(go["mean"], fo["mean"], dtype, "mean")
    return go, fo, errs


def _check_backward(ctx, layer, d, dtype, with_dHn=True):
    fo = G.oracle_forward(ctx, d)
    Hn, rstd, mean = G.saved_from_oracle(ctx, fo)
    gb = G.gpu_backward(ctx, layer, d, Hn, rstd, mean, with_dHn)
    ob = G.oracle_backward(ctx, d, Hn, rstd, mean, with_dHn)
    for k in ("dY", "dW", "dR", "dgamma"):
        assert_close(gb[k], ob[k], dtype, k)
    if ctx.norm == caat.LAYERNORM:
        assert_close(gb["dbeta"], ob["dbeta"], dtype, "dbeta")
    return gb, ob


# ------------------------------------------------------------------ the small fp32 configuration
def test_config1_fp32_forward():
    w = synthetic.WORKLOADS["layer_fp32_small"]
    d = _layer_case(w.t, w.tokens, w.h, w.kr_mlp, "f32", O.shared_channels(w.h, w.p), seed=w.seed)
    ctx = G.make_ctx(w.t, w.h, w.ffn, "f32", p=w.p)
    assert ctx.shared_channels == 128
    _check_forward(ctx, caat.CAAT_MLP_DOWN, d, "f32")


def test_config1_fp32_backward_and_layernorm():
    w = synthetic.WORKLOADS["layer_fp32_small"]
    d = _layer_case(w.t, w.tokens, w.h, w.kr_mlp, "f32", O.shared_channels(w.h, w.p), seed=1, backward=True)
    for norm in (0, 1):
        ctx = G.make_ctx(w.t, w.h, w.ffn, "f32", p=w.p, norm=norm)
        d["gamma"] = (1 + 0.1 * torch.randn(w.h, generator=torch.Generator().manual_seed(3))).float()
        d["beta"] = (0.1 * torch.randn(w.h, generator=torch.Generator().manual_seed(4))).float()
        _check_forward(ctx, caat.CAAT_MLP_DOWN, d, "f32")
        _check_backward(ctx, caat.CAAT_MLP_DOWN, d, "f32")


# ------------------------------------------------------------------ bf16, several tiles and ragged tails
CASES = [
    # t, T,   h,    ffn,  layer,            S,    alpha, norm
    (4, 300, 768, 3072, caat.CAAT_ATTN_OUT, 384, None, 0),     # 130M shapes, ragged token count
    (4, 257, 768, 3072, caat.CAAT_MLP_DOWN, 384, 1.0, 0),
    (8, 200, 2048, 5632, caat.CAAT_ATTN_OUT, 1536, None, 0),   # 1.1B shapes, p = 0.75
    (8, 129, 2048, 5632, caat.CAAT_MLP_DOWN, 512, None, 1),    # K_r = 704, LayerNorm
    (8, 130, 4096, 11008, caat.CAAT_ATTN_OUT, 2048, None, 0),  # 7B shapes
    (8, 70, 4096, 11008, caat.CAAT_MLP_DOWN, 2048, None, 0),   # K_r = 1376 (not a multiple of 64)
    (2, 64, 256, 1024, caat.CAAT_MLP_DOWN, 0, None, 0),        # p = 0: no shared channels
    (2, 64, 256, 1024, caat.CAAT_MLP_DOWN, 256, None, 0),      # p = 1: full all-reduce
    (3, 50, 264, 792, caat.CAAT_ATTN_OUT, 100, None, 0),       # S not a multiple of 8, K_r = 88
    (1, 33, 128, 512, caat.CAAT_MLP_DOWN, 64, None, 1),        # a single rank
    (16, 40, 512, 2048, caat.CAAT_ATTN_OUT, 256, None, 0),     # t = 16, K_r = 32
]


@pytest.mark.parametrize("t,T,h,ffn,layer,S,alpha,norm", CASES)
def test_bf16_forward_backward(t, T, h, ffn, layer, S, alpha, norm):
    ctx = G.make_ctx(t, h, ffn, "bf16", S=S, alpha=alpha, norm=norm)
    k = ctx.k_r(layer)
    d = _layer_case(t, T, h, k, "bf16", S, seed=T, backward=True)
    g = torch.Generator().manual_seed(5)
    d["gamma"] = (1 + 0.1 * torch.randn(h, generator=g)).bfloat16()
    d["beta"] = (0.1 * torch.randn(h, generator=g)).bfloat16()
    _check_forward(ctx, layer, d, "bf16")
    _check_backward(ctx, layer, d, "bf16")


def test_bf16_untied_residual_and_no_stream_gradient():
    ctx = G.make_ctx(4, 768, 3072, "bf16", S=384)
    d = _layer_case(4, 96, 768, 768, "bf16", 384, seed=9, backward=True, tied=False)
    _check_forward(ctx, caat.CAAT_MLP_DOWN, d, "bf16")
    _check_backward(ctx, caat.CAAT_MLP_DOWN, d, "bf16", with_dHn=False)


@pytest.mark.parametrize("force_simt", [False, True])
def test_both_gemm_paths_agree_with_oracle(force_simt):
    ctx = G.make_ctx(4, 512, 2048, "bf16", S=256, force_simt=force_simt)
    d = _layer_case(4, 384, 512, 512, "bf16", 256, seed=2, backward=True)
    _check_forward(ctx, caat.CAAT_MLP_DOWN, d, "bf16")
    _check_backward(ctx, caat.CAAT_MLP_DOWN, d, "bf16")


@pytest.mark.parametrize("direct_rows", [0, 1, 2])
@pytest.mark.parametrize("t,T,h,ffn,S,norm,dtype", [
    (8, 77, 4096, 11008, 2048, 0, "bf16"), (4, 301, 768, 3072, 380, 1, "bf16"), (2, 131, 256, 1024, 100, 1, "f32"),
    (8, 1500, 2048, 5632, 2048, 0, "bf16"), (3, 45, 9216, 9216, 4608, 0, "bf16"),
    (4, 2003, 768, 3072, 384, 0, "bf16"), (8, 1, 1024, 4096, 100, 1, "bf16"), (16, 70, 512, 2048, 512, 0, "f32")])
def test_both_row_kernel_variants(direct_rows, t, T, h, ffn, S, norm, dtype):
    # the three row-kernel families compute the same thing: automatic choice (warp-per-token for
    # short rows, bulk-copy staged otherwise), plain loads (1), staged always (2);
    # T = 1500 makes persistent CTAs walk several token groups, h = 9216 takes four chunks per thread
    ctx = G.make_ctx(t, h, ffn, dtype, S=S, norm=norm, direct_rows=direct_rows)
    d = _layer_case(t, T, h, ctx.k_r(caat.CAAT_ATTN_OUT), dtype, S, seed=T, backward=True)
    _check_forward(ctx, caat.CAAT_ATTN_OUT, d, dtype)
    _check_backward(ctx, caat.CAAT_ATTN_OUT, d, dtype)


@pytest.mark.parametrize("with_dHn", [True, False])
@pytest.mark.parametrize("t,T,h,S,norm,dtype", [
    (4, 333, 4096, 2056, 0, "bf16"),   # two chunks per thread, the partition inside a warp: lanes of both classes
    (4, 100, 4096, 1024, 1, "bf16"),   # LayerNorm; warps with one shared + one private chunk and with two private ones
    (2, 50, 8192, 6144, 0, "bf16"),    # rows of 512 threads; warps with two shared chunks and with one of each
    (4, 75, 2304, 1152, 1, "bf16"),    # 288 chunks on 2 x 160 threads: chunks past the row end
    (4, 131, 1024, 512, 0, "f32"),     # fp32, two token rows per CTA, odd token count
    (8, 131, 512, 256, 1, "f32"),      # fp32, one chunk per thread, LayerNorm
    (4, 257, 2048, 0, 0, "bf16"),      # no shared channels
    (4, 257, 2048, 2048, 1, "bf16")])  # no private channels
def test_row_kernels_with_the_partition_on_a_chunk_boundary(t, T, h, S, norm, dtype, with_dHn):
    # S a multiple of 8 and the per-rank layout: the backward runs the staged family's lean kernel, whose loop body is
    # compiled once per warp-uniform pattern of shared / private chunks plus a general one (the forward runs the
    # staged kernel on the same shapes)
    ctx = G.make_ctx(t, h, h, dtype, S=S, norm=norm, direct_rows=2)
    d = _layer_case(t, T, h, ctx.k_r(caat.CAAT_ATTN_OUT), dtype, S, seed=T + S, backward=True, tied=with_dHn)
    _check_forward(ctx, caat.CAAT_ATTN_OUT, d, dtype)
    _check_backward(ctx, caat.CAAT_ATTN_OUT, d, dtype, with_dHn=with_dHn)


# ------------------------------------------------------------------ partition: bit-exact
@pytest.mark.parametrize("S", [0, 1, 7, 8, 9, 127, 128, 129, 255, 256, 257, 504, 511, 512])
def test_partition_bit_exact_integer_inputs(S):
    # Small integers: every product, rank sum and residual add is exact in bf16/fp32, so the
    # GPU's Hn must equal the oracle's bit for bit wherever the shared/private boundary lies.
    t, T, h, K_r = 4, 70, 512, 16
    Y = synthetic.small_integers((t, T, K_r), -2, 2, seed=S)
    W = synthetic.small_integers((t, h, K_r), -1, 1, seed=S + 1)
    R = synthetic.small_integers((t, T, h), -8, 8, seed=S + 2)
    d = {"Y": Y, "W": W, "R": R, "gamma": torch.ones(h).bfloat16(), "beta": None}
    ctx = G.make_ctx(t, h, t * K_r, "bf16", S=S, alpha=1.0)
    go = G.gpu_forward(ctx, caat.CAAT_MLP_DOWN, d)
    fo = G.oracle_forward(ctx, d)
    assert np.array_equal(f64(go["Hn"]), fo["Hn"])
    # alpha = 2 (exact): private channels carry the factor, shared ones do not
    ctx2 = G.make_ctx(t, h, t * K_r, "bf16", S=S, alpha=2.0)
    go2 = G.gpu_forward(ctx2, caat.CAAT_MLP_DOWN, d)
    fo2 = G.oracle_forward(ctx2, d)
    assert np.array_equal(f64(go2["Hn"]), fo2["Hn"])


def test_fingerprint_channels():
    # Y_m = (m+1), W_m picks input 0: shared channels = t(t+1)/2, private = alpha (m+1), exactly.
    t, T, h, K_r, S = 4, 40, 256, 64, 96
    Y = torch.stack([torch.full((T, K_r), float(m + 1)) for m in range(t)]).bfloat16()
    W = torch.zeros(t, h, K_r); W[:, :, 0] = 1.0
    d = {"Y": Y, "W": W.bfloat16(), "R": torch.zeros(t, T, h).bfloat16(), "gamma": torch.ones(h).bfloat16()}
    ctx = G.make_ctx(t, h, t * K_r, "bf16", S=S, alpha=2.0)
    Hn = f64(G.gpu_forward(ctx, caat.CAAT_MLP_DOWN, d)["Hn"])
    assert np.all(Hn[:, :, :S] == t * (t + 1) / 2)
    for m in range(t):
        assert np.all(Hn[m, :, S:] == 2.0 * (m + 1))


def test_p0_no_cross_rank_mixing_bitwise():
    t, T, h, K_r = 4, 64, 256, 64
    d = _layer_case(t, T, h, K_r, "bf16", 0, seed=11, tied=False)
    ctx = G.make_ctx(t, h, t * K_r, "bf16", S=0)
    a = G.gpu_forward(ctx, caat.CAAT_MLP_DOWN, d)
    d2 = {k: (v.clone() if isinstance(v, torch.Tensor) else v) for k, v in d.items()}
    d2["Y"][1] += 1; d2["W"][1] *= -2; d2["R"][1] += 3
    b = G.gpu_forward(ctx, caat.CAAT_MLP_DOWN, d2)
    for m in (0, 2, 3):
        assert torch.equal(a["X"][m], b["X"][m]) and torch.equal(a["Hn"][m], b["Hn"][m])
    assert not torch.equal(a["X"][1], b["X"][1])


def test_backward_reduce_accumulates_in_fp32():
    # One rank contributes 256 and seven contribute 1 on a shared channel of the residual-stream
    # gradient (dX = 0, so g = dHn).  Summed in fp32 the result is 263; a bf16 running sum would
    # stay at 256 (ulp 2).  dY = dZt W with W an identity picker exposes the sum: 263 rounds to
    # 264 in bf16.
    t, T, h, K_r, S = 8, 16, 64, 8, 64
    d = {"Y": torch.zeros(t, T, K_r).bfloat16(), "gamma": torch.ones(h).bfloat16(),
         "dX": torch.zeros(t, T, h).bfloat16()}
    W = torch.zeros(t, h, K_r); W[:, 0, 0] = 1.0
    d["W"] = W.bfloat16()
    dHn = torch.zeros(t, T, h); dHn[:, :, 0] = 1.0; dHn[0, :, 0] = 256.0
    d["dHn"] = dHn.bfloat16()
    ctx = G.make_ctx(t, h, t * K_r, "bf16", S=S, alpha=1.0)
    Hn = torch.ones(t, T, h).bfloat16(); rstd = torch.ones(t, T)
    gb = G.gpu_backward(ctx, caat.CAAT_MLP_DOWN, d, Hn, rstd, None)
    assert torch.all(gb["dY"][:, :, 0].float() == 264.0)
    ob = G.oracle_backward(ctx, d, Hn, rstd, None)
    assert np.all(ob["dY"][:, :, 0] == 263.0)


def test_run_to_run_bit_reproducible():
    ctx = G.make_ctx(8, 2048, 5632, "bf16", S=1024)
    d = _layer_case(8, 192, 2048, 704, "bf16", 1024, seed=21, backward=True)
    fo = G.oracle_forward(ctx, d)
    Hn, rstd, mean = G.saved_from_oracle(ctx, fo)
    a = G.gpu_backward(ctx, caat.CAAT_MLP_DOWN, d, Hn, rstd, mean)
    b = G.gpu_backward(ctx, caat.CAAT_MLP_DOWN, d, Hn, rstd, mean)
    for k in ("dY", "dW", "dR", "dgamma"):
        assert torch.equal(a[k], b[k]), k
    fa = G.gpu_forward(ctx, caat.CAAT_MLP_DOWN, d)
    fb = G.gpu_forward(ctx, caat.CAAT_MLP_DOWN, d)
    assert torch.equal(fa["X"], fb["X"]) and torch.equal(fa["Hn"], fb["Hn"])


def test_in_place_residual_update():
    ctx = G.make_ctx(4, 768, 3072, "bf16", S=384)
    T = 100
    d = _layer_case(4, T, 768, 192, "bf16", 384, seed=4)
    ref = G.gpu_forward(ctx, caat.CAAT_ATTN_OUT, d)
    R = d["R"].cuda()
    X = torch.empty_like(R); rstd = torch.empty(4, T, device="cuda")
    ws = ctx.alloc_workspace(ctx.workspace_bytes(caat.CAAT_ATTN_OUT, T, False))
    ctx.rowpar_forward(caat.CAAT_ATTN_OUT, T, d["Y"].cuda(), d["W"].cuda(), R, d["gamma"].cuda(), None, R, X, rstd,
                       None, ws)
    torch.cuda.synchronize()
    assert torch.equal(R.cpu(), ref["Hn"]) and torch.equal(X.cpu(), ref["X"])


# ------------------------------------------------------------------ block
def test_block_forward_backward_small():
    w = synthetic.Workload("blk", 4, 150, 768, 3072, 0.5, "bf16", "block", True, 7)
    d = synthetic.block_inputs(w, O.shared_channels(w.h, w.p))
    ctx = G.make_ctx(w.t, w.h, w.ffn, "bf16", p=w.p)
    t, T, h = w.t, w.tokens, w.h
    dev = {k: v.cuda() for k, v in d.items()}
    mk = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt, device="cuda")
    Hn1, X1, Hn2, X2 = (mk(t, T, h) for _ in range(4))
    rstd1, rstd2 = mk(t, T, dt=torch.float32), mk(t, T, dt=torch.float32)
    ws = ctx.alloc_workspace(ctx.block_workspace_bytes(T, True))
    ctx.block_forward(T, dev["Y_attn"], dev["W_o"], dev["Y_mlp"], dev["W_down"], dev["R0"], dev["gamma1"], None,
                      dev["gamma2"], None, Hn1, X1, rstd1, None, Hn2, X2, rstd2, None, ws)
    fo = O.block_forward(f64(d["Y_attn"]), f64(d["W_o"]), f64(d["Y_mlp"]), f64(d["W_down"]), f64(d["R0"]),
                         f64(d["gamma1"]), f64(d["gamma2"]), S=ctx.shared_channels, alpha=ctx.private_scale)
    for name, g in (("Hn1", Hn1), ("X1", X1), ("Hn2", Hn2), ("X2", X2), ("rstd1", rstd1), ("rstd2", rstd2)):
        assert_close(g, fo[name], "bf16", name)
    # backward on saved tensors taken from the oracle's forward (rounded to storage types)
    sHn1, sHn2 = (torch.from_numpy(fo[k]).bfloat16() for k in ("Hn1", "Hn2"))
    sr1, sr2 = (torch.from_numpy(fo[k]).float() for k in ("rstd1", "rstd2"))
    ka, km = ctx.k_r(caat.CAAT_ATTN_OUT), ctx.k_r(caat.CAAT_MLP_DOWN)
    dYa, dYm, dR0, dHn1 = mk(t, T, ka), mk(t, T, km), mk(t, T, h), mk(t, T, h)
    dWo, dWd = mk(t, h, ka, dt=torch.float32), mk(t, h, km, dt=torch.float32)
    dg1, dg2 = mk(h, dt=torch.float32), mk(h, dt=torch.float32)
    ctx.block_backward(T, dev["dX1"], dev["dX2"], dev["dHn2"], dev["Y_attn"], dev["W_o"], dev["Y_mlp"], dev["W_down"],
                       sHn1.cuda(), sr1.cuda(), None, sHn2.cuda(), sr2.cuda(), None, dev["gamma1"], dev["gamma2"],
                       dYa, dWo, dYm, dWd, dR0, dHn1, dg1, None, dg2, None, ws)
    ob = O.block_backward(f64(d["dX1"]), f64(d["dX2"]), f64(d["dHn2"]), f64(d["Y_attn"]), f64(d["W_o"]),
                          f64(d["Y_mlp"]), f64(d["W_down"]), f64(sHn1), f64(sr1), None, f64(sHn2), f64(sr2), None,
                          f64(d["gamma1"]), f64(d["gamma2"]), S=ctx.shared_channels, alpha=ctx.private_scale)
    for name, g in (("dY_attn", dYa), ("dW_o", dWo), ("dY_mlp", dYm), ("dW_down", dWd), ("dR0", dR0),
                    ("dHn1", dHn1), ("dgamma1", dg1), ("dgamma2", dg2)):
        assert_close(g, ob[name], "bf16", name)


@pytest.mark.parametrize("no_decode", [False, True])
@pytest.mark.parametrize("t,T,h,ffn,S,norm", [(8, 64, 4096, 11008, 2048, 0), (4, 37, 768, 3072, 384, 1),
                                             (8, 1, 2048, 5632, 2048, 0), (2, 5, 256, 1024, 0, 0),
                                             # a handful of tokens: the cluster row kernel (LayerNorm; a shared
                                             # slice that does not divide evenly among the ranks; three ranks)
                                             (4, 3, 768, 3072, 384, 1), (8, 2, 4096, 11008, 1000, 0),
                                             (3, 4, 768, 3072, 256, 0),
                                             # shared part smaller than the cluster: most CTAs own no slice
                                             (8, 2, 4096, 11008, 8, 0), (8, 3, 4096, 11008, 4088, 1)])
def test_few_token_forward_both_paths(no_decode, t, T, h, ffn, S, norm):
    # forward calls with at most 64 tokens take the weight-streaming path (swapped GEMM operands,
    # rank sum in the row kernel); CAAT_OPT_DECODE = 1 sends them down the large-batch path
    ctx = G.make_ctx(t, h, ffn, "bf16", S=S, norm=norm, no_decode=no_decode)
    for layer in (caat.CAAT_ATTN_OUT, caat.CAAT_MLP_DOWN):
        d = _layer_case(t, T, h, ctx.k_r(layer), "bf16", S, seed=T + layer)
        g = torch.Generator().manual_seed(6)
        d["gamma"] = (1 + 0.1 * torch.randn(h, generator=g)).bfloat16()
        d["beta"] = (0.1 * torch.randn(h, generator=g)).bfloat16()
        _check_forward(ctx, layer, d, "bf16")


@pytest.mark.parametrize("T,p,no_decode", [(1, 1.0, False), (8, 0.5, False), (64, 0.5, False), (64, 0.5, True), (33, 0.25, False)])
def test_block_forward_few_tokens(T, p, no_decode):
    # block forward at decode sizes: one GEMM launch for both layers + one row kernel for both
    w = synthetic.Workload("blk_dec", 8, T, 4096, 11008, p, "bf16", "block", False, 3)
    d = synthetic.block_inputs(w, O.shared_channels(w.h, w.p))
    ctx = G.make_ctx(w.t, w.h, w.ffn, "bf16", p=w.p, no_decode=no_decode)
    t, h = w.t, w.h
    dev = {k: v.cuda() for k, v in d.items()}
    mk = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt, device="cuda")
    Hn1, X1, Hn2, X2 = (mk(t, T, h) for _ in range(4))
    rstd1, rstd2 = mk(t, T, dt=torch.float32), mk(t, T, dt=torch.float32)
    ws = ctx.alloc_workspace(ctx.block_workspace_bytes(T, False))
    ctx.block_forward(T, dev["Y_attn"], dev["W_o"], dev["Y_mlp"], dev["W_down"], dev["R0"], dev["gamma1"], None,
                      dev["gamma2"], None, Hn1, X1, rstd1, None, Hn2, X2, rstd2, None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    fo = O.block_forward(f64(d["Y_attn"]), f64(d["W_o"]), f64(d["Y_mlp"]), f64(d["W_down"]), f64(d["R0"]),
                         f64(d["gamma1"]), f64(d["gamma2"]), S=ctx.shared_channels, alpha=ctx.private_scale)
    for name, g in (("Hn1", Hn1), ("X1", X1), ("Hn2", Hn2), ("X2", X2), ("rstd1", rstd1), ("rstd2", rstd2)):
        assert_close(g, fo[name], "bf16", name)


@pytest.mark.timeout(180)
@pytest.mark.parametrize("t,T,h,ffn,p,norm", [
    (1, 28, 128, 256, 1.0, 0),      # a single rank (no cluster of ranks): 16 chunks per row, half a warp
    (16, 20, 896, 1792, 0.5, 1),    # more ranks than a cluster holds; 112 chunks per row: 3 1/2 warps
    (4, 23, 160, 320, 0.95, 0),     # the cluster kernel on a row of 20 chunks, slices of 5, 5, 5, 4 chunks
    (2, 64, 96, 192, 0.5, 1)])      # 12 chunks per row
def test_block_forward_few_tokens_with_rows_that_do_not_fill_their_warps(t, T, h, ffn, p, norm):
    # two layers in one row-kernel launch, rows whose 16-byte chunks are no multiple of 32: lanes without a chunk skip
    # the chunk loop, so nothing inside it may synchronise the warp (a sync there deadlocked the second layer)
    w = synthetic.Workload("blk_dec_small", t, T, h, ffn, p, "bf16", "block", False, 5)
    S = O.shared_channels(h, p) // 8 * 8
    d = synthetic.block_inputs(w, S)
    g = torch.Generator().manual_seed(8)
    b1 = (0.1 * torch.randn(h, generator=g)).to(torch.bfloat16).cuda() if norm else None
    b2 = (0.1 * torch.randn(h, generator=g)).to(torch.bfloat16).cuda() if norm else None
    ctx = G.make_ctx(t, h, ffn, "bf16", S=S, norm=norm)
    dev = {k: v.cuda() for k, v in d.items()}
    mk = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt, device="cuda")
    o = {"Hn1": mk(t, T, h), "X1": mk(t, T, h), "rstd1": mk(t, T, dt=torch.float32), "Hn2": mk(t, T, h), "X2": mk(t, T, h),
         "rstd2": mk(t, T, dt=torch.float32)}
    m1 = mk(t, T, dt=torch.float32) if norm else None
    m2 = mk(t, T, dt=torch.float32) if norm else None
    ws = ctx.alloc_workspace(ctx.block_workspace_bytes(T, False))
    launches = caat.kernel_launches()
    ctx.block_forward(T, dev["Y_attn"], dev["W_o"], dev["Y_mlp"], dev["W_down"], dev["R0"], dev["gamma1"], b1,
                      dev["gamma2"], b2, o["Hn1"], o["X1"], o["rstd1"], m1, o["Hn2"], o["X2"], o["rstd2"], m2, ws)
    torch.cuda.synchronize()
    assert caat.kernel_launches() - launches == 2          # the weight-streaming GEMM and one row kernel for both layers
    assert ctx.last_device_status() == caat.CAAT_OK
    fo = O.block_forward(f64(d["Y_attn"]), f64(d["W_o"]), f64(d["Y_mlp"]), f64(d["W_down"]), f64(d["R0"]), f64(d["gamma1"]),
                         f64(d["gamma2"]), f64(b1.cpu()) if norm else None, f64(b2.cpu()) if norm else None, S=S,
                         alpha=math.sqrt(t), norm=norm)
    for k in o:
        assert_close(o[k], fo[k], "bf16", k)


# ------------------------------------------------------------------ decode shapes (forward only)
@pytest.mark.parametrize("T", [1, 8, 64])
@pytest.mark.parametrize("p", [1.0, 0.5])
def test_decode_7b_forward(T, p):
    w = synthetic.WORKLOADS[f"decode_7b_T{T}_p{int(p * 100):03d}"]
    ctx = G.make_ctx(w.t, w.h, w.ffn, "bf16", p=w.p)
    for layer, k in ((caat.CAAT_ATTN_OUT, w.kr_attn), (caat.CAAT_MLP_DOWN, w.kr_mlp)):
        d = _layer_case(w.t, T, w.h, k, "bf16", O.shared_channels(w.h, w.p), seed=T)
        _check_forward(ctx, layer, d, "bf16")


@pytest.mark.parametrize("t,T,h,ffn,p,norm", [(4, 1500, 768, 3072, 0.5, 0), (8, 700, 2048, 5632, 0.25, 1), (8, 300, 4096, 11008, 1.0, 0)])
def test_block_forward_side_by_side_schedule_equals_the_serial_one(t, T, h, ffn, p, norm):
    # the block forward that runs the first layer's row kernel beside the second layer's GEMM (second stream,
    # plain-load row kernel, a GEMM with one pipeline stage less) against the same call with the overlap switched
    # off, and against a workspace too small for two scratch regions (which must fall back to the serial schedule)
    w = synthetic.Workload("blk_ovl", t, T, h, ffn, p, "bf16", "block", False, 11)
    S = O.shared_channels(h, p)
    d = synthetic.block_inputs(w, S)
    g = torch.Generator().manual_seed(5)
    for k in ("gamma1", "gamma2"):
        d[k] = (1 + 0.1 * torch.randn(h, generator=g)).to(torch.bfloat16)
    b1 = (0.1 * torch.randn(h, generator=g)).to(torch.bfloat16).cuda() if norm else None
    b2 = (0.1 * torch.randn(h, generator=g)).to(torch.bfloat16).cuda() if norm else None
    dev = {k: v.cuda() for k, v in d.items()}
    mk = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt, device="cuda")
    outs = []
    for overlap, small_ws in ((1, False), (0, False), (1, True)):
        ctx = G.make_ctx(t, h, ffn, "bf16", p=p, norm=norm)
        assert ctx.set_option(caat.CAAT_OPT_BLOCK_OVERLAP, overlap) is ctx
        nbytes = ctx.block_workspace_bytes(T, False)
        one = max(ctx.workspace_bytes(caat.CAAT_ATTN_OUT, T, False), ctx.workspace_bytes(caat.CAAT_MLP_DOWN, T, False))
        assert nbytes > one
        ws = ctx.alloc_workspace(one if small_ws else nbytes)
        o = {"Hn1": mk(t, T, h), "X1": mk(t, T, h), "rstd1": mk(t, T, dt=torch.float32), "Hn2": mk(t, T, h), "X2": mk(t, T, h),
             "rstd2": mk(t, T, dt=torch.float32)}
        m1 = mk(t, T, dt=torch.float32) if norm else None
        m2 = mk(t, T, dt=torch.float32) if norm else None
        launches = caat.kernel_launches()
        ctx.block_forward(T, dev["Y_attn"], dev["W_o"], dev["Y_mlp"], dev["W_down"], dev["R0"], dev["gamma1"], b1,
                          dev["gamma2"], b2, o["Hn1"], o["X1"], o["rstd1"], m1, o["Hn2"], o["X2"], o["rstd2"], m2, ws)
        torch.cuda.synchronize()
        assert caat.kernel_launches() - launches == 4
        assert ctx.last_device_status() == caat.CAAT_OK
        outs.append(o)
    fo = O.block_forward(f64(d["Y_attn"]), f64(d["W_o"]), f64(d["Y_mlp"]), f64(d["W_down"]), f64(d["R0"]), f64(d["gamma1"]),
                         f64(d["gamma2"]), f64(b1.cpu()) if norm else None, f64(b2.cpu()) if norm else None, S=S,
                         alpha=math.sqrt(t), norm=norm)
    for k in outs[0]:
        assert_close(outs[0][k], fo[k], "bf16", f"side by side: {k}")
        assert torch.equal(outs[1][k], outs[2][k]), f"serial schedule, two workspace sizes: {k}"
        if k.startswith("Hn"):        # sums and one rounding per element: the same on every row-kernel variant
            assert torch.equal(outs[0][k], outs[1][k]), f"side by side against serial: {k}"
        else:                         # the row statistics are reduced in another order by the plain-load kernel
            assert_close(outs[0][k], f64(outs[1][k]), "bf16", f"side by side against serial: {k}", scale=0.5)


def test_side_by_side_block_forward_inside_a_stream_capture():
    # the fork onto the library's own stream and the join back are events recorded and waited on inside the call,
    # which a stream capture turns into graph edges: the captured call replays to the same results as the eager one
    t, T, h, ffn, p = 4, 1500, 768, 3072, 0.5
    w = synthetic.Workload("blk_graph", t, T, h, ffn, p, "bf16", "block", False, 13)
    dev = {k: v.cuda() for k, v in synthetic.block_inputs(w, O.shared_channels(h, p)).items()}
    ctx = G.make_ctx(t, h, ffn, "bf16", p=p)
    ctx.set_option(caat.CAAT_OPT_BLOCK_OVERLAP, 1)
    ws = ctx.alloc_workspace(ctx.block_workspace_bytes(T, False))
    mk = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt, device="cuda")
    outs = [{"Hn1": mk(t, T, h), "X1": mk(t, T, h), "rstd1": mk(t, T, dt=torch.float32), "Hn2": mk(t, T, h), "X2": mk(t, T, h),
             "rstd2": mk(t, T, dt=torch.float32)} for _ in range(2)]

    def call(o):
        ctx.block_forward(T, dev["Y_attn"], dev["W_o"], dev["Y_mlp"], dev["W_down"], dev["R0"], dev["gamma1"], None,
                          dev["gamma2"], None, o["Hn1"], o["X1"], o["rstd1"], None, o["Hn2"], o["X2"], o["rstd2"], None, ws)

    call(outs[0])                                   # eager; also creates the library's stream before any capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        call(outs[1])
    for v in outs[1].values():
        v.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    for k in outs[0]:
        assert torch.equal(outs[0][k], outs[1][k]), k
