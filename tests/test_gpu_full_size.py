"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (block
forward + backward through the C ABI on the full token count).

The fp64 oracle cannot hold a full-size problem at once, so it walks the tokens in chunks
(tokens are independent rows in everything except dW and dgamma, which are sums over tokens
and are accumulated across chunks).  Compared:

* every forward/backward activation output on a STRATIFIED sample of tokens (whole rows, all
  ranks): the first and the last row of every 128-row tile of the token axis (that also
  covers both sides of every 256-row pair-tile edge), the ragged tail after the last full
  tile, and a few seeded random rows - at least 256 rows in all, so every row tile of every
  GEMM and every token group of the row kernels is touched; the 130M block compares the
  forward outputs on ALL tokens;
* dgamma in full;
* dW on a stratified sample of (rank, channel, input) entries, each a full sum over all
  tokens (hence over every split-K slice): at least one entry - the two extreme corners
  plus random ones - in every (rank, 128-channel block, 256-input block) output tile, at
  least 4096 entries in all.

Saved tensors handed to the GPU backward are the oracle's forward results rounded to their
storage types, never GPU outputs - except in the chained case, where the GPU backward runs
on the GPU forward's own saved tensors while the oracle keeps to its own chain."""
import math

import numpy as np
import pytest
import torch

from oracle import caat_oracle as O
from paper_2506_19645_b200 import caat, synthetic
from tests.helpers import assert_close, f64, stratified_entries, stratified_tokens

pytestmark = pytest.mark.gpu

CHUNK = 1024


def _chunks(T):
    for a in range(0, T, CHUNK):
        yield a, min(T, a + CHUNK)


def _check_block_full(name, seed=123, all_forward_rows=False, chained=False):
    w = synthetic.WORKLOADS[name]
    t, T, h = w.t, w.tokens, w.h
    S = O.shared_channels(h, w.p)
    alpha = math.sqrt(t)
    ka, km = w.kr_attn, w.kr_mlp
    dev = synthetic.block_inputs(w, S, device="cuda")
    host = {k: v.cpu() for k, v in dev.items()}
    rng = np.random.default_rng(seed)
    tok = stratified_tokens(T, rng)
    assert len(tok) >= 256 or len(tok) == T
    edge = (S - 1, S)
    dws = {"attn": stratified_entries(t, h, ka, rng, extra_rows=edge), "mlp": stratified_entries(t, h, km, rng, extra_rows=edge)}
    assert all(len(v[0]) >= 4096 for v in dws.values())
    Wd = {"attn": f64(host["W_o"]), "mlp": f64(host["W_down"])}
    g1, g2 = f64(host["gamma1"]), f64(host["gamma2"])

    # ---------------- GPU: the bench's launch configuration (block forward, then block backward)
    ctx = caat.Context(w.h, w.ffn, t, w.p, "bf16")
    assert ctx.shared_channels == S
    mk = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt, device="cuda")
    f32 = torch.float32
    out = {"Hn1": mk(t, T, h), "X1": mk(t, T, h), "rstd1": mk(t, T, dt=f32), "Hn2": mk(t, T, h), "X2": mk(t, T, h),
           "rstd2": mk(t, T, dt=f32)}
    ws = ctx.alloc_workspace(ctx.block_workspace_bytes(T, True))
    ctx.block_forward(T, dev["Y_attn"], dev["W_o"], dev["Y_mlp"], dev["W_down"], dev["R0"], dev["gamma1"], None,
                      dev["gamma2"], None, out["Hn1"], out["X1"], out["rstd1"], None, out["Hn2"], out["X2"],
                      out["rstd2"], None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK

    # ---------------- oracle forward, chunked; keep saved tensors (rounded) and sampled rows
    sHn1 = torch.empty((t, T, h), dtype=torch.bfloat16); sHn2 = torch.empty_like(sHn1)
    sr1 = torch.empty((t, T), dtype=torch.float32); sr2 = torch.empty_like(sr1)
    fkeys = ("Hn1", "X1", "rstd1", "Hn2", "X2", "rstd2")
    fwd_s = {k: [] for k in fkeys}
    for a, b in _chunks(T):
        sl = slice(a, b)
        o = O.block_forward(f64(host["Y_attn"][:, sl]), Wd["attn"], f64(host["Y_mlp"][:, sl]), Wd["mlp"],
                            f64(host["R0"][:, sl]), g1, g2, S=S, alpha=alpha)
        sHn1[:, sl] = torch.from_numpy(o["Hn1"]).to(torch.bfloat16); sHn2[:, sl] = torch.from_numpy(o["Hn2"]).to(torch.bfloat16)
        sr1[:, sl] = torch.from_numpy(o["rstd1"]).float(); sr2[:, sl] = torch.from_numpy(o["rstd2"]).float()
        if all_forward_rows:
            for k in fkeys:
                assert_close(out[k][:, sl], o[k], "bf16", f"{name}:{k}[{a}:{b}]")
        loc = tok[(tok >= a) & (tok < b)] - a
        for k in fkeys:
            fwd_s[k].append(o[k][:, loc])
    fwd_s = {k: np.concatenate(v, axis=1) for k, v in fwd_s.items()}
    tk = torch.from_numpy(tok).cuda()
    for k in fkeys:
        assert_close(out[k].index_select(1, tk), fwd_s[k], "bf16", f"{name}:{k}")
    if not w.backward:
        return
    bo = {"dY_attn": mk(t, T, ka), "dW_o": mk(t, h, ka, dt=f32), "dY_mlp": mk(t, T, km), "dW_down": mk(t, h, km, dt=f32),
          "dR0": mk(t, T, h), "dHn1": mk(t, T, h), "dgamma1": mk(h, dt=f32), "dgamma2": mk(h, dt=f32)}
    if chained:       # the GPU's own saved tensors; the oracle below keeps its own
        sv = (out["Hn1"], out["rstd1"], out["Hn2"], out["rstd2"])
    else:
        del out
        sv = (sHn1.cuda(), sr1.cuda(), sHn2.cuda(), sr2.cuda())
    ctx.block_backward(T, dev["dX1"], dev["dX2"], dev["dHn2"], dev["Y_attn"], dev["W_o"], dev["Y_mlp"], dev["W_down"],
                       sv[0], sv[1], None, sv[2], sv[3], None, dev["gamma1"], dev["gamma2"],
                       bo["dY_attn"], bo["dW_o"], bo["dY_mlp"], bo["dW_down"], bo["dR0"], bo["dHn1"], bo["dgamma1"], None,
                       bo["dgamma2"], None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK

    # ---------------- oracle backward, chunked (MLP-down first, then attention-out on its dR)
    acc = {"dgamma1": np.zeros(h), "dgamma2": np.zeros(h), "dW_attn": np.zeros(len(dws["attn"][0])),
           "dW_mlp": np.zeros(len(dws["mlp"][0]))}
    bwd_s = {k: [] for k in ("dY_attn", "dY_mlp", "dR0", "dHn1")}
    for a, b in _chunks(T):
        sl = slice(a, b)
        loc = tok[(tok >= a) & (tok < b)] - a
        Hn2, r2 = f64(sHn2[:, sl]), f64(sr2[:, sl])
        gm = O.residual_stream_gradient(f64(host["dX2"][:, sl]), f64(host["dHn2"][:, sl]), Hn2, r2, None, g2, O.RMSNORM)
        acc["dgamma2"] += O.norm_param_gradients(f64(host["dX2"][:, sl]), Hn2, r2, None, O.RMSNORM)[0]
        dZ2 = O.backward_partial_channel_reduce(gm, S, alpha)
        Hn1, r1 = f64(sHn1[:, sl]), f64(sr1[:, sl])
        ga = O.residual_stream_gradient(f64(host["dX1"][:, sl]), gm, Hn1, r1, None, g1, O.RMSNORM)
        acc["dgamma1"] += O.norm_param_gradients(f64(host["dX1"][:, sl]), Hn1, r1, None, O.RMSNORM)[0]
        dZ1 = O.backward_partial_channel_reduce(ga, S, alpha)
        bwd_s["dY_mlp"].append(O.data_gradient(dZ2[:, loc], Wd["mlp"]))
        bwd_s["dY_attn"].append(O.data_gradient(dZ1[:, loc], Wd["attn"]))
        bwd_s["dHn1"].append(gm[:, loc]); bwd_s["dR0"].append(ga[:, loc])
        for key, dZ, Yk in (("attn", dZ1, "Y_attn"), ("mlp", dZ2, "Y_mlp")):
            m_, l_, k_ = dws[key]
            Y = f64(host[Yk][:, sl])
            acc["dW_" + key] += np.einsum("ni,ni->n", dZ[m_, :, l_], Y[m_, :, k_])   # dW[m,l,k] = sum_i dZt[m,i,l] Y[m,i,k]
    bwd_s = {k: np.concatenate(v, axis=1) for k, v in bwd_s.items()}

    for k in bwd_s:
        assert_close(bo[k].index_select(1, tk), bwd_s[k], "bf16", f"{name}:{k}")
    assert_close(bo["dgamma1"], acc["dgamma1"], "bf16", f"{name}:dgamma1")
    assert_close(bo["dgamma2"], acc["dgamma2"], "bf16", f"{name}:dgamma2")
    for key, gk in (("attn", "dW_o"), ("mlp", "dW_down")):
        m_, l_, k_ = (torch.from_numpy(x).cuda() for x in dws[key])
        assert_close(bo[gk][m_, l_, k_], acc["dW_" + key], "bf16", f"{name}:{gk}")


def test_full_size_block_130m():
    _check_block_full("block_130m", all_forward_rows=True)


def test_full_size_block_130m_chained():
    # forward -> backward on the library's own saved tensors (Hn, rstd as the GPU wrote them)
    _check_block_full("block_130m", seed=77, chained=True)


@pytest.mark.parametrize("name", ["block_1p1b_p100", "block_1p1b_p075", "block_1p1b_p050", "block_1p1b_p025"])
def test_full_size_block_1p1b(name):
    _check_block_full(name)


def test_full_size_block_7b():
    _check_block_full("block_7b")


def _check_mlp_full(name, seed=321):
    """Whole MLP (column-parallel gate|up + SwiGLU, then MLP-down with partial channel-reduce) at the bench's
    size and launch sequence; the oracle walks the tokens in chunks and accumulates the token sums."""
    w = synthetic.WORKLOADS[name]
    t, T, h, F = w.t, w.tokens, w.h, w.kr_mlp
    S = O.shared_channels(h, w.p)
    alpha = math.sqrt(t)
    dev = synthetic.mlp_inputs(w, S, device="cuda")
    host = {k: v.cpu() for k, v in dev.items()}
    rng = np.random.default_rng(seed)
    tok = stratified_tokens(T, rng)
    iA = stratified_entries(t, 2 * F, h, rng, extra_rows=(F - 1, F))          # dA [t, 2F, h]; F = the gate | up edge
    iB = stratified_entries(t, h, F, rng, extra_rows=(S - 1, S))              # dB [t, h, F]
    assert len(iA[0]) >= 4096 and len(iB[0]) >= 4096
    A, B, g = f64(host["A"]), f64(host["B"]), f64(host["gamma"])
    bf, f32 = torch.bfloat16, torch.float32

    spre = torch.empty((t, T, 2 * F), dtype=bf); sY = torch.empty((t, T, F), dtype=bf)
    sHn = torch.empty((t, T, h), dtype=bf); sr = torch.empty((t, T), dtype=f32)
    fwd_s = {k: [] for k in ("pre", "Y", "Hn", "X", "rstd")}
    for a, b in _chunks(T):
        sl = slice(a, b)
        o = O.mlp_forward(f64(host["X"][:, sl]), A, B, f64(host["R"][:, sl]), g, S=S, alpha=alpha)
        spre[:, sl] = torch.from_numpy(o["pre"]).to(bf); sY[:, sl] = torch.from_numpy(o["Y"]).to(bf)
        sHn[:, sl] = torch.from_numpy(o["Hn"]).to(bf); sr[:, sl] = torch.from_numpy(o["rstd"]).float()
        loc = tok[(tok >= a) & (tok < b)] - a
        for k in fwd_s:
            fwd_s[k].append(o[k][:, loc])
    fwd_s = {k: np.concatenate(v, axis=1) for k, v in fwd_s.items()}

    ctx = caat.Context(w.h, w.ffn, t, w.p, "bf16")
    assert ctx.shared_channels == S
    mk = lambda *s, dt=bf: torch.empty(*s, dtype=dt, device="cuda")
    out = {"pre": mk(t, T, 2 * F), "Y": mk(t, T, F), "Hn": mk(t, T, h), "X": mk(t, T, h), "rstd": mk(t, T, dt=f32)}
    ws = ctx.alloc_workspace(max(ctx.workspace_bytes(caat.CAAT_MLP_DOWN, T, True),
                                 ctx.colpar_workspace_bytes(caat.CAAT_ACT_SWIGLU, 2 * F, T)))
    ctx.colpar_forward(caat.CAAT_ACT_SWIGLU, 2 * F, T, dev["X"], dev["A"], out["pre"], out["Y"])
    ctx.rowpar_forward(caat.CAAT_MLP_DOWN, T, out["Y"], dev["B"], dev["R"], dev["gamma"], None, out["Hn"], out["X"],
                       out["rstd"], None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    tk = torch.from_numpy(tok).cuda()
    for k in fwd_s:
        assert_close(out[k].index_select(1, tk), fwd_s[k], "bf16", f"{name}:{k}")
    del out

    bo = {"dY": mk(t, T, F), "dB": mk(t, h, F, dt=f32), "dR": mk(t, T, h), "dgamma": mk(h, dt=f32), "dX": mk(t, T, h),
          "dA": mk(t, 2 * F, h, dt=f32)}
    dY_saved = torch.empty((t, T, F), dtype=bf)
    acc = {"dgamma": np.zeros(h), "dA": np.zeros(len(iA[0])), "dB": np.zeros(len(iB[0]))}
    bwd_s = {k: [] for k in ("dX", "dR", "dY")}
    for a, b in _chunks(T):
        sl = slice(a, b)
        loc = tok[(tok >= a) & (tok < b)] - a
        Hn, r = f64(sHn[:, sl]), f64(sr[:, sl])
        gm = O.residual_stream_gradient(f64(host["dXout"][:, sl]), f64(host["dHn"][:, sl]), Hn, r, None, g, O.RMSNORM)
        acc["dgamma"] += O.norm_param_gradients(f64(host["dXout"][:, sl]), Hn, r, None, O.RMSNORM)[0]
        dZ = O.backward_partial_channel_reduce(gm, S, alpha)
        Y = f64(sY[:, sl])
        dY = O.data_gradient(dZ, B)
        dY_saved[:, sl] = torch.from_numpy(dY).to(bf)
        m_, l_, k_ = iB
        acc["dB"] += np.einsum("ni,ni->n", dZ[m_, :, l_], Y[m_, :, k_])
        cb = O.colpar_backward(f64(dY_saved[:, sl]), f64(host["X"][:, sl]), A, f64(spre[:, sl]), O.ACT_SWIGLU)
        m_, n_, j_ = iA
        acc["dA"] += np.einsum("ni,ni->n", cb["dpre"][m_, :, n_], f64(host["X"][:, sl])[m_, :, j_])
        bwd_s["dX"].append(cb["dX"][:, loc]); bwd_s["dR"].append(gm[:, loc]); bwd_s["dY"].append(dY[:, loc])
    bwd_s = {k: np.concatenate(v, axis=1) for k, v in bwd_s.items()}
    ctx.rowpar_backward(caat.CAAT_MLP_DOWN, T, dev["dXout"], dev["dHn"], sY.cuda(), dev["B"], sHn.cuda(), sr.cuda(), None,
                        dev["gamma"], bo["dY"], bo["dB"], bo["dR"], bo["dgamma"], None, ws)
    # the column-parallel backward runs on the oracle's dY (rounded), so the two halves are checked independently
    ctx.colpar_backward(caat.CAAT_ACT_SWIGLU, 2 * F, T, dY_saved.cuda(), dev["X"], dev["A"], spre.cuda(), bo["dX"], bo["dA"], ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    for k in bwd_s:
        assert_close(bo[k].index_select(1, tk), bwd_s[k], "bf16", f"{name}:{k}")
    assert_close(bo["dgamma"], acc["dgamma"], "bf16", f"{name}:dgamma")
    m_, l_, k_ = (torch.from_numpy(x).cuda() for x in iB)
    assert_close(bo["dB"][m_, l_, k_], acc["dB"], "bf16", f"{name}:dB")
    m_, n_, j_ = (torch.from_numpy(x).cuda() for x in iA)
    assert_close(bo["dA"][m_, n_, j_], acc["dA"], "bf16", f"{name}:dA")


@pytest.mark.parametrize("name", ["mlp_130m", "mlp_7b"])
def test_full_size_mlp(name):
    _check_mlp_full(name)


def _check_block_full_compact(name, seed=456):
    """The block on the compact residual stream (shared channels stored once) at the bench's size and launch
    sequence: chunked oracle, stratified tokens for per-token outputs, token sums accumulated over chunks."""
    w = synthetic.WORKLOADS[name]
    t, T, h = w.t, w.tokens, w.h
    S = O.shared_channels(h, w.p)
    alpha = math.sqrt(t)
    ka, km = w.kr_attn, w.kr_mlp
    dev = synthetic.block_inputs(w, S, device="cuda")
    host = {k: v.cpu() for k, v in dev.items()}
    split = lambda x: (x[0, :, :S].contiguous(), x[:, :, S:].contiguous())
    R0s, R0p = split(host["R0"]); dH2s, dH2p = split(host["dHn2"])
    rng = np.random.default_rng(seed)
    tok = stratified_tokens(T, rng)
    edge = (S - 1, S)
    dws = {"attn": stratified_entries(t, h, ka, rng, extra_rows=edge), "mlp": stratified_entries(t, h, km, rng, extra_rows=edge)}
    Wd = {"attn": f64(host["W_o"]), "mlp": f64(host["W_down"])}
    g1, g2 = f64(host["gamma1"]), f64(host["gamma2"])
    bf, f32 = torch.bfloat16, torch.float32

    sv = {"Hn1s": torch.empty((T, S), dtype=bf), "Hn1p": torch.empty((t, T, h - S), dtype=bf), "rstd1": torch.empty((t, T), dtype=f32),
          "Hn2s": torch.empty((T, S), dtype=bf), "Hn2p": torch.empty((t, T, h - S), dtype=bf), "rstd2": torch.empty((t, T), dtype=f32)}
    keys = ("Hn1s", "Hn1p", "X1", "rstd1", "Hn2s", "Hn2p", "X2", "rstd2")
    fwd_s = {k: [] for k in keys}
    tdim = lambda k: 0 if k.endswith("s") else 1           # token axis of a tensor: shared parts are [T, S]
    for a, b in _chunks(T):
        sl = slice(a, b)
        o = O.block_forward_compact(f64(host["Y_attn"][:, sl]), Wd["attn"], f64(host["Y_mlp"][:, sl]), Wd["mlp"],
                                    f64(R0s[sl]), f64(R0p[:, sl]), g1, g2, S=S, alpha=alpha)
        for k in sv:
            if tdim(k) == 0:
                sv[k][sl] = torch.from_numpy(o[k]).to(sv[k].dtype)
            else:
                sv[k][:, sl] = torch.from_numpy(o[k]).to(sv[k].dtype)
        loc = tok[(tok >= a) & (tok < b)] - a
        for k in keys:
            fwd_s[k].append(np.take(o[k], loc, axis=tdim(k)))
    fwd_s = {k: np.concatenate(v, axis=tdim(k)) for k, v in fwd_s.items()}

    ctx = caat.Context(w.h, w.ffn, t, w.p, "bf16")
    assert ctx.shared_channels == S
    mk = lambda *s, dt=bf: torch.empty(*s, dtype=dt, device="cuda")
    out = {"Hn1s": mk(T, S), "Hn1p": mk(t, T, h - S), "X1": mk(t, T, h), "rstd1": mk(t, T, dt=f32),
           "Hn2s": mk(T, S), "Hn2p": mk(t, T, h - S), "X2": mk(t, T, h), "rstd2": mk(t, T, dt=f32)}
    ws = ctx.alloc_workspace(ctx.block_workspace_bytes(T, True))
    ctx.block_forward_compact(T, dev["Y_attn"], dev["W_o"], dev["Y_mlp"], dev["W_down"], R0s.cuda(), R0p.cuda(), dev["gamma1"],
                              None, dev["gamma2"], None, out["Hn1s"], out["Hn1p"], out["X1"], out["rstd1"], None,
                              out["Hn2s"], out["Hn2p"], out["X2"], out["rstd2"], None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    tk = torch.from_numpy(tok).cuda()
    for k in keys:
        assert_close(out[k].index_select(tdim(k), tk), fwd_s[k], "bf16", f"{name}:{k}")
    del out

    bo = {"dY_attn": mk(t, T, ka), "dW_o": mk(t, h, ka, dt=f32), "dY_mlp": mk(t, T, km), "dW_down": mk(t, h, km, dt=f32),
          "dR0s": mk(T, S), "dR0p": mk(t, T, h - S), "dHn1s": mk(T, S), "dHn1p": mk(t, T, h - S),
          "dgamma1": mk(h, dt=f32), "dgamma2": mk(h, dt=f32)}
    ctx.block_backward_compact(T, dev["dX1"], dev["dX2"], dH2s.cuda(), dH2p.cuda(), dev["Y_attn"], dev["W_o"], dev["Y_mlp"],
                               dev["W_down"], sv["Hn1s"].cuda(), sv["Hn1p"].cuda(), sv["rstd1"].cuda(), None,
                               sv["Hn2s"].cuda(), sv["Hn2p"].cuda(), sv["rstd2"].cuda(), None, dev["gamma1"], dev["gamma2"],
                               bo["dY_attn"], bo["dW_o"], bo["dY_mlp"], bo["dW_down"], bo["dR0s"], bo["dR0p"], bo["dHn1s"],
                               bo["dHn1p"], bo["dgamma1"], None, bo["dgamma2"], None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK

    acc = {"dgamma1": np.zeros(h), "dgamma2": np.zeros(h), "dW_attn": np.zeros(len(dws["attn"][0])),
           "dW_mlp": np.zeros(len(dws["mlp"][0]))}
    bkeys = ("dY_attn", "dY_mlp", "dR0s", "dR0p", "dHn1s", "dHn1p")
    bwd_s = {k: [] for k in bkeys}
    for a, b in _chunks(T):
        sl = slice(a, b)
        loc = tok[(tok >= a) & (tok < b)] - a
        b2 = O.rowpar_backward_compact(f64(host["dX2"][:, sl]), f64(dH2s[sl]), f64(dH2p[:, sl]), f64(host["Y_mlp"][:, sl]),
                                       Wd["mlp"], f64(sv["Hn2s"][sl]), f64(sv["Hn2p"][:, sl]), f64(sv["rstd2"][:, sl]), None, g2,
                                       S=S, alpha=alpha)
        b1 = O.rowpar_backward_compact(f64(host["dX1"][:, sl]), b2["dRs"], b2["dRp"], f64(host["Y_attn"][:, sl]), Wd["attn"],
                                       f64(sv["Hn1s"][sl]), f64(sv["Hn1p"][:, sl]), f64(sv["rstd1"][:, sl]), None, g1,
                                       S=S, alpha=alpha)
        acc["dgamma2"] += b2["dgamma"]; acc["dgamma1"] += b1["dgamma"]
        for key, bb in (("attn", b1), ("mlp", b2)):
            m_, l_, k_ = dws[key]
            acc["dW_" + key] += bb["dW"][m_, l_, k_]
        for k, v in (("dY_attn", b1["dY"]), ("dY_mlp", b2["dY"]), ("dR0s", b1["dRs"]), ("dR0p", b1["dRp"]),
                     ("dHn1s", b2["dRs"]), ("dHn1p", b2["dRp"])):
            bwd_s[k].append(np.take(v, loc, axis=tdim(k) if k.startswith("dR") or k.startswith("dHn") else 1))
    for k in bkeys:
        ax = tdim(k) if k.startswith("dR") or k.startswith("dHn") else 1
        assert_close(bo[k].index_select(ax, tk), np.concatenate(bwd_s[k], axis=ax), "bf16", f"{name}:{k}")
    assert_close(bo["dgamma1"], acc["dgamma1"], "bf16", f"{name}:dgamma1")
    assert_close(bo["dgamma2"], acc["dgamma2"], "bf16", f"{name}:dgamma2")
    for key, gk in (("attn", "dW_o"), ("mlp", "dW_down")):
        m_, l_, k_ = (torch.from_numpy(x).cuda() for x in dws[key])
        assert_close(bo[gk][m_, l_, k_], acc["dW_" + key], "bf16", f"{name}:{gk}")


@pytest.mark.parametrize("name", ["block_130m", "block_7b"])
def test_full_size_block_compact(name):
    _check_block_full_compact(name)
