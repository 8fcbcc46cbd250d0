"""Real tensor parallelism, checked on one GPU: the t ranks are split into G groups (one per GPU in a real run),
every group runs the first half of the layer call, the all-reduce of the shared-channel slab is stood in for by
summing the groups' slabs the way tp.py's collective does (carried in fp32, rounded once; a second test measures
what a 16-bit payload with 16-bit partial sums costs), every group runs the second half, and the concatenated results
must match the fp64 oracle with all t ranks — forward and backward.  Needs a GPU."""
import numpy as np
import pytest
import torch

from oracle import caat_oracle as O
from paper_2506_19645_b200 import caat, synthetic
from tests.helpers import assert_close, f64, to_dtype

pytestmark = pytest.mark.gpu
BF = torch.bfloat16


def _sum_slabs(slabs, accumulate):
    """Stands in for the all-reduce that tp.py issues between the halves.  A collective accumulates in its payload
    type: tp.py carries the slab in fp32 by default (forward and backward), so the sum is rounded once at the end;
    `accumulate = bf16` models the slab sent as it is, where every partial sum is rounded to bf16 (here in rank
    order, as a ring that starts at rank 0 would)."""
    total = slabs[0].to(accumulate)
    for s in slabs[1:]:
        total = (total.float() + s.float()).to(accumulate)
    for s in slabs:
        s.copy_(total)


@pytest.mark.parametrize("t,G,T,h,ffn,S,layer,norm", [
    (8, 4, 300, 1024, 4096, 512, caat.CAAT_ATTN_OUT, 0),
    (8, 8, 130, 1024, 4096, 256, caat.CAAT_MLP_DOWN, 0),      # one rank per GPU
    (4, 2, 257, 768, 3072, 768, caat.CAAT_MLP_DOWN, 1),       # p = 1 (a full all-reduce), LayerNorm
    (4, 2, 200, 768, 3072, 0, caat.CAAT_ATTN_OUT, 0),         # p = 0: nothing to exchange
])
def test_groups_with_slab_sum_match_oracle(t, G, T, h, ffn, S, layer, norm):
    tl = t // G
    K = (h if layer == caat.CAAT_ATTN_OUT else ffn) // t
    ctxs = []
    for _ in range(G):
        c = caat.Context(h, ffn, tl, 0.5, "bf16")
        c.set_option(caat.CAAT_OPT_SHARED_CHANNELS, S).set_option(caat.CAAT_OPT_NORM, norm)
        c.set_option(caat.CAAT_OPT_TP_GROUPS, G)
        assert c.k_r(layer) == K and abs(c.private_scale - np.sqrt(t)) < 1e-12
        ctxs.append(c)
    alpha = ctxs[0].private_scale
    d = synthetic.layer_inputs(t, T, h, K, "bf16", seed=3 + T, S=S, backward=True)
    g = torch.Generator().manual_seed(9)
    d["gamma"] = (1 + 0.1 * torch.randn(h, generator=g)).to(BF)
    d["beta"] = (0.1 * torch.randn(h, generator=g)).to(BF) if norm else None
    dev = {k: (v.cuda() if v is not None else None) for k, v in d.items()}
    sl = lambda x, q: x[q * tl:(q + 1) * tl]
    mk = lambda *s, dt=BF: torch.empty(*s, dtype=dt, device="cuda")
    f32 = torch.float32

    # ---- forward
    ws = [c.alloc_workspace(c.workspace_bytes(layer, T, True)) for c in ctxs]
    Hn, X = mk(t, T, h), mk(t, T, h)
    rstds = [mk(tl, T, dt=f32) for _ in range(G)]          # each GPU's own statistics (own allocations: alignment)
    means = [mk(tl, T, dt=f32) if norm else None for _ in range(G)]
    for q, c in enumerate(ctxs):
        c.tp_forward_local(layer, T, sl(dev["Y"], q), sl(dev["W"], q), ws[q])
    if S > 0:
        _sum_slabs([c.tp_slab(layer, T, False, ws[q]) for q, c in enumerate(ctxs)], torch.float32)
    for q, c in enumerate(ctxs):
        c.tp_forward_finish(layer, T, sl(dev["R"], q), dev["gamma"], dev["beta"], sl(Hn, q), sl(X, q), rstds[q],
                            means[q], ws[q])
    torch.cuda.synchronize()
    assert all(c.last_device_status() == caat.CAAT_OK for c in ctxs)
    fo = O.rowpar_forward(f64(d["Y"]), f64(d["W"]), f64(d["R"]), f64(d["gamma"]), f64(d["beta"]) if norm else None,
                          S=S, alpha=alpha, norm=norm)
    for k, v in (("Hn", Hn), ("X", X), ("rstd", torch.cat(rstds))):
        assert_close(v.cpu(), fo[k], "bf16", k)

    # ---- backward on the oracle's saved tensors (rounded to their storage types)
    sHn, srs = to_dtype(fo["Hn"], BF).cuda(), to_dtype(fo["rstd"], f32).cuda()
    smu = to_dtype(fo["mean"], f32).cuda() if norm else None
    dY, dW, dR = mk(t, T, K), mk(t, h, K, dt=f32), mk(t, T, h)
    dgs = [mk(h, dt=f32) for _ in range(G)]
    dbs = [mk(h, dt=f32) if norm else None for _ in range(G)]
    for q, c in enumerate(ctxs):
        c.tp_backward_local(layer, T, sl(dev["dX"], q), sl(dev["dHn"], q), sl(dev["W"], q), sl(sHn, q),
                            sl(srs, q).clone(), sl(smu, q).clone() if norm else None, dev["gamma"], sl(dR, q), dgs[q],
                            dbs[q], ws[q])
    if S > 0:
        _sum_slabs([c.tp_slab(layer, T, True, ws[q]) for q, c in enumerate(ctxs)], torch.float32)
    dgamma = torch.stack(dgs).sum(0)                   # the fp32 all-reduce of the norm-parameter gradients
    for q, c in enumerate(ctxs):
        c.tp_backward_finish(layer, T, sl(dev["Y"], q), sl(dev["W"], q), sl(dR, q), sl(dY, q), sl(dW, q), ws[q])
    torch.cuda.synchronize()
    assert all(c.last_device_status() == caat.CAAT_OK for c in ctxs)
    ob = O.rowpar_backward(f64(d["dX"]), f64(d["dHn"]), f64(d["Y"]), f64(d["W"]), f64(sHn.cpu()), f64(srs.cpu()),
                           f64(smu.cpu()) if norm else None, f64(d["gamma"]), S=S, alpha=alpha, norm=norm)
    for k, v in (("dY", dY), ("dW", dW), ("dR", dR), ("dgamma", dgamma)):
        assert_close(v.cpu(), ob[k], "bf16", k)
    if norm:
        assert_close(torch.stack(dbs).sum(0).cpu(), ob["dbeta"], "bf16", "dbeta")


def test_sixteen_bit_collective_is_less_accurate_than_the_fp32_carry():
    # The forward slab sent through a collective in its own 16-bit type: every partial sum is rounded.  With 8 ranks
    # that is visibly worse than carrying fp32 (the library's default in tp.py) - the reason for that default.
    t, G, T, h, ffn, S, layer = 8, 8, 130, 1024, 4096, 256, caat.CAAT_MLP_DOWN
    K = ffn // t
    d = synthetic.layer_inputs(t, T, h, K, "bf16", seed=3 + T, S=S)
    exact = O.partial_channel_reduce(O.rank_partials(f64(d["Y"]), f64(d["W"])), S, 1.0)[0, :, :S]
    errs = {}
    for acc in (torch.float32, BF):
        ctxs, ws = [], []
        for q in range(G):
            c = caat.Context(h, ffn, 1, 0.5, "bf16")
            c.set_option(caat.CAAT_OPT_SHARED_CHANNELS, S).set_option(caat.CAAT_OPT_TP_GROUPS, G)
            w = c.alloc_workspace(c.workspace_bytes(layer, T, False))
            c.tp_forward_local(layer, T, d["Y"][q:q + 1].cuda(), d["W"][q:q + 1].cuda(), w)
            ctxs.append(c); ws.append(w)
        slabs = [c.tp_slab(layer, T, False, ws[q]) for q, c in enumerate(ctxs)]
        _sum_slabs(slabs, acc)
        torch.cuda.synchronize()
        got = f64(slabs[0])
        errs[acc] = float(np.sqrt(np.mean((got - exact) ** 2)) / np.sqrt(np.mean(exact ** 2)))
    assert errs[torch.float32] < 4e-3                   # bf16 partials of each group + one final rounding
    assert errs[BF] > 1.5 * errs[torch.float32]


def test_one_group_halves_equal_the_single_call():
    # G = 1: the two halves with nothing in between are the single call, bit for bit
    t, T, h, ffn, S, layer = 4, 300, 768, 3072, 384, caat.CAAT_MLP_DOWN
    ctx = caat.Context(h, ffn, t, 0.5, "bf16")
    K = ctx.k_r(layer)
    d = {k: v.cuda() for k, v in synthetic.layer_inputs(t, T, h, K, "bf16", seed=5, S=S, backward=True).items()}
    mk = lambda *s, dt=BF: torch.empty(*s, dtype=dt, device="cuda")
    f32 = torch.float32
    ws = ctx.alloc_workspace(ctx.workspace_bytes(layer, T, True))
    a = {"Hn": mk(t, T, h), "X": mk(t, T, h), "rstd": mk(t, T, dt=f32)}
    b = {"Hn": mk(t, T, h), "X": mk(t, T, h), "rstd": mk(t, T, dt=f32)}
    ctx.rowpar_forward(layer, T, d["Y"], d["W"], d["R"], d["gamma"], None, a["Hn"], a["X"], a["rstd"], None, ws)
    ctx.tp_forward_local(layer, T, d["Y"], d["W"], ws)
    ctx.tp_forward_finish(layer, T, d["R"], d["gamma"], None, b["Hn"], b["X"], b["rstd"], None, ws)
    for k in a:
        assert torch.equal(a[k], b[k]), k
    ga = {"dY": mk(t, T, K), "dW": mk(t, h, K, dt=f32), "dR": mk(t, T, h), "dg": mk(h, dt=f32)}
    gb = {"dY": mk(t, T, K), "dW": mk(t, h, K, dt=f32), "dR": mk(t, T, h), "dg": mk(h, dt=f32)}
    ctx.rowpar_backward(layer, T, d["dX"], d["dHn"], d["Y"], d["W"], a["Hn"], a["rstd"], None, d["gamma"], ga["dY"],
                        ga["dW"], ga["dR"], ga["dg"], None, ws)
    ctx.tp_backward_local(layer, T, d["dX"], d["dHn"], d["W"], a["Hn"], a["rstd"], None, d["gamma"], gb["dR"], gb["dg"],
                          None, ws)
    ctx.tp_backward_finish(layer, T, d["Y"], d["W"], gb["dR"], gb["dY"], gb["dW"], ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    for k in ga:
        assert torch.equal(ga[k], gb[k]), k


def test_tp_wrapper_with_a_group_of_one():
    from paper_2506_19645_b200 import tp
    t, T, h, ffn, layer = 2, 140, 512, 2048, caat.CAAT_ATTN_OUT
    lay = tp.TensorParallelRowLinear(h, ffn, t, 0.5)
    K = lay.ctx.k_r(layer)
    d = {k: v.cuda() for k, v in synthetic.layer_inputs(t, T, h, K, "bf16", seed=2, S=h // 2, backward=True).items()}
    mk = lambda *s, dt=BF: torch.empty(*s, dtype=dt, device="cuda")
    f32 = torch.float32
    ws = lay.workspace(layer, T)
    Hn, X, rstd = mk(t, T, h), mk(t, T, h), mk(t, T, dt=f32)
    lay.forward(layer, T, d["Y"], d["W"], d["R"], d["gamma"], None, Hn, X, rstd, None, ws)
    dY, dW, dR, dg = mk(t, T, K), mk(t, h, K, dt=f32), mk(t, T, h), mk(h, dt=f32)
    lay.backward(layer, T, d["dX"], d["dHn"], d["Y"], d["W"], Hn, rstd, None, d["gamma"], dY, dW, dR, dg, None, ws)
    torch.cuda.synchronize()
    fo = O.rowpar_forward(f64(d["Y"].cpu()), f64(d["W"].cpu()), f64(d["R"].cpu()), f64(d["gamma"].cpu()), None,
                          S=h // 2, alpha=lay.ctx.private_scale)
    assert_close(X.cpu(), fo["X"], "bf16", "X")
    ob = O.rowpar_backward(f64(d["dX"].cpu()), f64(d["dHn"].cpu()), f64(d["Y"].cpu()), f64(d["W"].cpu()), f64(Hn.cpu()),
                           f64(rstd.cpu()), None, f64(d["gamma"].cpu()), S=h // 2, alpha=lay.ctx.private_scale)
    assert_close(dY.cpu(), ob["dY"], "bf16", "dY")
    assert_close(dW.cpu(), ob["dW"], "bf16", "dW")
