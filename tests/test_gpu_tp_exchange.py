"""The slab exchange over peer memory (the library's own reduce-scatter + all-gather kernels), checked on ONE GPU:
the G groups of a tensor-parallel job each get their own workspace, receive buffer and flag words on the same
device and address each other's buffers as "peers"; the phases run group after group (all scatters, then all
reduces, then all waits), so no kernel ever waits for a later launch.  Checked: the reduced slab against the fp32
sum of the groups' slabs in group order rounded once (bit for bit - that is the kernel's definition), the layer's
forward and backward against the fp64 oracle with all ranks, the fused form (forward GEMM storing the shared tiles
straight into the owners' slots) against the unfused one, and a wait that nothing satisfies.  Needs a GPU."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from oracle import caat_oracle as O
from paper_2506_19645_b200 import caat, synthetic
from tests.helpers import assert_close, f64, to_dtype

pytestmark = pytest.mark.gpu
BF, F32 = torch.bfloat16, torch.float32


class Group:
    """One GPU of the job: context for its ranks, workspace, receive buffer, flag words."""

    def __init__(self, t_local, G, h, ffn, S, layer, T, norm=0):
        c = caat.Context(h, ffn, t_local, 0.5, "bf16")
        c.set_option(caat.CAAT_OPT_SHARED_CHANNELS, S).set_option(caat.CAAT_OPT_NORM, norm)
        c.set_option(caat.CAAT_OPT_TP_GROUPS, G)
        self.ctx = c
        self.ws = c.alloc_workspace(c.workspace_bytes(layer, T, True))
        nbytes, self.slice = c.tp_exchange_bytes(layer, T, G)
        self.recv = torch.full((nbytes,), 0x7F, dtype=torch.uint8, device="cuda")      # NaN-ish bf16 pattern: stale data shows
        self.flags = torch.zeros(caat.CAAT_TP_FLAG_BYTES // 4, dtype=torch.int32, device="cuda")


def make_peers(groups, layer, T, backward):
    slabs = [g.ctx.tp_slab(layer, T, backward, g.ws) for g in groups]
    out = []
    for q, g in enumerate(groups):
        out.append(g.ctx.make_peers(q, [x.recv.data_ptr() for x in groups], [s.data_ptr() for s in slabs],
                                    [x.flags.data_ptr() for x in groups]))
    return out, slabs


def exchange(groups, peers, layer, T, backward, epoch, scatter=True):
    if scatter:
        for g, pe in zip(groups, peers):
            g.ctx.tp_exchange_scatter(layer, T, backward, pe, epoch, g.ws)
    for g, pe in zip(groups, peers):
        g.ctx.tp_exchange_reduce(layer, T, pe, epoch)
    for g, pe in zip(groups, peers):
        g.ctx.tp_exchange_wait(pe, epoch)


def fp32_sum_rounded_once(slabs):
    total = slabs[0].float()
    for s in slabs[1:]:
        total = total + s.float()
    return total.to(BF)


@pytest.mark.parametrize("t,G,T,h,ffn,S,layer,norm", [
    (8, 4, 300, 1024, 4096, 512, caat.CAAT_ATTN_OUT, 0),      # ragged slices of 80 tokens (the last owner holds 60)
    (8, 8, 130, 1024, 4096, 256, caat.CAAT_MLP_DOWN, 0),      # one rank per GPU; the last owners hold nothing
    (4, 2, 257, 768, 3072, 768, caat.CAAT_MLP_DOWN, 1),       # p = 1 (a full all-reduce), LayerNorm
    (2, 1, 200, 512, 2048, 256, caat.CAAT_ATTN_OUT, 0),       # a group of one: the exchange is a copy
])
def test_exchange_gives_the_fp32_sum_and_the_layer_matches_the_oracle(t, G, T, h, ffn, S, layer, norm):
    tl = t // G
    K = (h if layer == caat.CAAT_ATTN_OUT else ffn) // t
    groups = [Group(tl, G, h, ffn, S, layer, T, norm) for _ in range(G)]
    alpha = groups[0].ctx.private_scale
    d = synthetic.layer_inputs(t, T, h, K, "bf16", seed=11 + T, S=S, backward=True)
    gen = torch.Generator().manual_seed(9)
    d["gamma"] = (1 + 0.1 * torch.randn(h, generator=gen)).to(BF)
    d["beta"] = (0.1 * torch.randn(h, generator=gen)).to(BF) if norm else None
    dev = {k: (v.cuda() if v is not None else None) for k, v in d.items()}
    sl = lambda x, q: x[q * tl:(q + 1) * tl]
    mk = lambda *s, dt=BF: torch.empty(*s, dtype=dt, device="cuda")

    # ---- forward
    for q, g in enumerate(groups):
        g.ctx.tp_forward_local(layer, T, sl(dev["Y"], q), sl(dev["W"], q), g.ws)
    peers, slabs = make_peers(groups, layer, T, False)
    want = fp32_sum_rounded_once(slabs)
    exchange(groups, peers, layer, T, False, epoch=1)
    torch.cuda.synchronize()
    for q, s in enumerate(slabs):
        assert torch.equal(s, want), f"forward slab of group {q}"
    Hn, X = mk(t, T, h), mk(t, T, h)
    rstds = [mk(tl, T, dt=F32) for _ in range(G)]
    means = [mk(tl, T, dt=F32) if norm else None for _ in range(G)]
    for q, g in enumerate(groups):
        g.ctx.tp_forward_finish(layer, T, sl(dev["R"], q), dev["gamma"], dev["beta"], sl(Hn, q), sl(X, q), rstds[q], means[q], g.ws)
    torch.cuda.synchronize()
    assert all(g.ctx.last_device_status() == caat.CAAT_OK for g in groups)
    fo = O.rowpar_forward(f64(d["Y"]), f64(d["W"]), f64(d["R"]), f64(d["gamma"]), f64(d["beta"]) if norm else None,
                          S=S, alpha=alpha, norm=norm)
    for k, v in (("Hn", Hn), ("X", X), ("rstd", torch.cat(rstds))):
        assert_close(v.cpu(), fo[k], "bf16", k)

    # ---- backward on the oracle's saved tensors, second exchange on the same buffers (epoch 2)
    sHn, srs = to_dtype(fo["Hn"], BF).cuda(), to_dtype(fo["rstd"], F32).cuda()
    smu = to_dtype(fo["mean"], F32).cuda() if norm else None
    dY, dW, dR = mk(t, T, K), mk(t, h, K, dt=F32), mk(t, T, h)
    dgs = [mk(h, dt=F32) for _ in range(G)]
    dbs = [mk(h, dt=F32) if norm else None for _ in range(G)]
    for q, g in enumerate(groups):
        g.ctx.tp_backward_local(layer, T, sl(dev["dX"], q), sl(dev["dHn"], q), sl(dev["W"], q), sl(sHn, q), sl(srs, q).clone(),
                                sl(smu, q).clone() if norm else None, dev["gamma"], sl(dR, q), dgs[q], dbs[q], g.ws)
    peers, slabs = make_peers(groups, layer, T, True)
    want = fp32_sum_rounded_once(slabs)
    exchange(groups, peers, layer, T, True, epoch=2)
    torch.cuda.synchronize()
    for q, s in enumerate(slabs):
        assert torch.equal(s, want), f"backward slab of group {q}"
    for q, g in enumerate(groups):
        g.ctx.tp_backward_finish(layer, T, sl(dev["Y"], q), sl(dev["W"], q), sl(dR, q), sl(dY, q), sl(dW, q), g.ws)
    torch.cuda.synchronize()
    assert all(g.ctx.last_device_status() == caat.CAAT_OK for g in groups)
    ob = O.rowpar_backward(f64(d["dX"]), f64(d["dHn"]), f64(d["Y"]), f64(d["W"]), f64(sHn.cpu()), f64(srs.cpu()),
                           f64(smu.cpu()) if norm else None, f64(d["gamma"]), S=S, alpha=alpha, norm=norm)
    for k, v in (("dY", dY), ("dW", dW), ("dR", dR), ("dgamma", torch.stack(dgs).sum(0))):
        assert_close(v.cpu(), ob[k], "bf16", k)


@pytest.mark.parametrize("t,G,T,h,ffn,S,layer", [
    (8, 4, 1000, 1024, 4096, 512, caat.CAAT_MLP_DOWN),       # slices of 256 tokens, the last owner holds 232
    (8, 8, 4096, 1024, 4096, 256, caat.CAAT_ATTN_OUT),       # one rank per GPU, 512 tokens each: CTA-pair tiles
    (4, 2, 700, 768, 3072, 768, caat.CAAT_MLP_DOWN),         # p = 1: every output tile is pushed
])
def test_forward_gemm_pushing_its_shared_tiles_equals_gemm_plus_scatter(t, G, T, h, ffn, S, layer):
    tl = t // G
    K = (h if layer == caat.CAAT_ATTN_OUT else ffn) // t
    d = {k: v.cuda() for k, v in synthetic.layer_inputs(t, T, h, K, "bf16", seed=5 + T, S=S).items()}
    sl = lambda x, q: x[q * tl:(q + 1) * tl]
    results = []
    for fused in (False, True):
        groups = [Group(tl, G, h, ffn, S, layer, T) for _ in range(G)]
        assert groups[0].slice % 256 == 0
        peers, slabs = make_peers(groups, layer, T, False)
        for q, (g, pe) in enumerate(zip(groups, peers)):
            if fused:
                g.ctx.tp_forward_local_push(layer, T, sl(d["Y"], q), sl(d["W"], q), pe, 7, g.ws)
            else:
                g.ctx.tp_forward_local(layer, T, sl(d["Y"], q), sl(d["W"], q), g.ws)
        exchange(groups, peers, layer, T, False, epoch=7, scatter=not fused)
        Hn, X = torch.empty(t, T, h, dtype=BF, device="cuda"), torch.empty(t, T, h, dtype=BF, device="cuda")
        for q, g in enumerate(groups):
            rstd = torch.empty(tl, T, dtype=F32, device="cuda")
            g.ctx.tp_forward_finish(layer, T, sl(d["R"], q), d["gamma"], None, sl(Hn, q), sl(X, q), rstd, None, g.ws)
        torch.cuda.synchronize()
        assert all(g.ctx.last_device_status() == caat.CAAT_OK for g in groups)
        results.append((slabs[0].clone(), Hn, X))
    for a, b, name in zip(results[0], results[1], ("slab", "Hn", "X")):
        assert torch.equal(a, b), name
    fo = O.rowpar_forward(f64(d["Y"]), f64(d["W"]), f64(d["R"]), f64(d["gamma"]), None, S=S, alpha=float(np.sqrt(t)))
    assert_close(results[1][2].cpu(), fo["X"], "bf16", "X (fused) against the oracle")


def test_push_needs_whole_tiles_per_owner():
    ctx = caat.Context(1024, 4096, 2, 0.5, "bf16")
    ctx.set_option(caat.CAAT_OPT_TP_GROUPS, 4)
    T = 300                                             # slices of 80 tokens: a 128-row tile would span two owners
    g = torch.zeros(64, dtype=torch.int32, device="cuda")
    pe = ctx.make_peers(0, [g.data_ptr()] * 4, [g.data_ptr()] * 4, [g.data_ptr()] * 4)
    ws = ctx.alloc_workspace(ctx.workspace_bytes(caat.CAAT_ATTN_OUT, T, False))
    Y = torch.zeros(2, T, ctx.k_r(caat.CAAT_ATTN_OUT), dtype=BF, device="cuda")
    W = torch.zeros(2, 1024, ctx.k_r(caat.CAAT_ATTN_OUT), dtype=BF, device="cuda")
    with pytest.raises(caat.CaatError) as e:
        ctx.tp_forward_local_push(caat.CAAT_ATTN_OUT, T, Y, W, pe, 1, ws)
    assert e.value.status == caat.CAAT_EUNSUPPORTED


CHILD = r"""
import torch
from paper_2506_19645_b200 import caat
ctx = caat.Context(512, 2048, 1, 0.5, "bf16")
ctx.set_option(caat.CAAT_OPT_TP_GROUPS, 2)
flags = torch.zeros(caat.CAAT_TP_FLAG_BYTES // 4, dtype=torch.int32, device="cuda")     # nothing will ever raise them
pe = ctx.make_peers(0, None, None, [flags.data_ptr()] * 2)
ctx.tp_exchange_wait(pe, 1)
torch.cuda.synchronize()                      # the kernel returned: no hang, no CUDA error
first = ctx.last_device_status()
second = ctx.last_device_status()             # reading the status clears it
x = torch.ones(1024, device="cuda").sum().item()   # the context still works
print("STATUS", first, second, int(x))
"""


def test_a_wait_nothing_satisfies_runs_out_and_reports_timeout():
    # a flag that no one raises (the permitted way to make a wait run out): short poll limit, status word, usable context
    env = dict(os.environ, CAAT_TP_POLLCAP="64")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", CHILD], env=env, cwd=root, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("STATUS")][-1].split()
    assert int(line[1]) == caat.CAAT_ETIMEOUT
    assert int(line[2]) == caat.CAAT_OK
    assert int(line[3]) == 1024


@pytest.mark.parametrize("T", [512, 200])       # whole tiles per owner (the GEMM pushes) / a short slice (GEMM, then scatter)
def test_wrapper_with_its_own_exchange_in_a_group_of_one(T):
    # tp.py's push path end to end - buffer carving, slab offsets of both directions, epochs, the fused and the
    # unfused forward - where the group is this GPU alone (the exchange then is a copy through the slot)
    from paper_2506_19645_b200 import tp
    t, h, ffn, layer = 2, 512, 2048, caat.CAAT_MLP_DOWN
    lay = tp.TensorParallelRowLinear(h, ffn, t, 0.5)
    K, S = lay.ctx.k_r(layer), lay.ctx.shared_channels
    pb = tp.PeerBuffers(lay.ctx, layer, T, addresses=[0], rank=0)
    assert (pb.slice_rows % 256 == 0) == (T == 512)
    d = {k: v.cuda() for k, v in synthetic.layer_inputs(t, T, h, K, "bf16", seed=2, S=S, backward=True).items()}
    mk = lambda *s, dt=BF: torch.empty(*s, dtype=dt, device="cuda")
    ref = {"Hn": mk(t, T, h), "X": mk(t, T, h), "rstd": mk(t, T, dt=F32), "dY": mk(t, T, K), "dW": mk(t, h, K, dt=F32),
           "dR": mk(t, T, h), "dg": mk(h, dt=F32)}
    got = {k: torch.empty_like(v) for k, v in ref.items()}
    ws = lay.workspace(layer, T)
    lay.forward(layer, T, d["Y"], d["W"], d["R"], d["gamma"], None, ref["Hn"], ref["X"], ref["rstd"], None, ws)
    lay.backward(layer, T, d["dX"], d["dHn"], d["Y"], d["W"], ref["Hn"], ref["rstd"], None, d["gamma"], ref["dY"], ref["dW"],
                 ref["dR"], ref["dg"], None, ws)
    for _ in range(2):                               # twice: the second round runs on the epochs and leftovers of the first
        lay.forward_push(layer, T, d["Y"], d["W"], d["R"], d["gamma"], None, got["Hn"], got["X"], got["rstd"], None, pb)
        lay.backward_push(layer, T, d["dX"], d["dHn"], d["Y"], d["W"], got["Hn"], got["rstd"], None, d["gamma"], got["dY"],
                          got["dW"], got["dR"], got["dg"], None, pb)
        torch.cuda.synchronize()
        assert lay.ctx.last_device_status() == caat.CAAT_OK
        for k in ref:
            assert torch.equal(ref[k], got[k]), k
    assert pb.epoch == 4


@pytest.mark.parametrize("t,G,T,h,ffn,S,layer,norm", [
    (8, 4, 300, 1024, 4096, 512, caat.CAAT_ATTN_OUT, 0),      # warp-per-token row kernel, ragged slices of 80 tokens
    (8, 8, 130, 2048, 8192, 1024, caat.CAAT_MLP_DOWN, 1),     # staged row kernel, LayerNorm, owners without tokens
    (4, 2, 700, 768, 3072, 768, caat.CAAT_MLP_DOWN, 0),       # p = 1
])
def test_backward_row_kernel_sending_the_slab_rows_equals_row_kernel_plus_scatter(t, G, T, h, ffn, S, layer, norm):
    tl = t // G
    K = (h if layer == caat.CAAT_ATTN_OUT else ffn) // t
    d = synthetic.layer_inputs(t, T, h, K, "bf16", seed=9 + T, S=S, backward=True)
    fo = O.rowpar_forward(f64(d["Y"]), f64(d["W"]), f64(d["R"]), f64(d["gamma"]), f64(d["beta"]) if norm else None, S=S,
                          alpha=float(np.sqrt(t)), norm=norm)
    sHn, srs = to_dtype(fo["Hn"], BF).cuda(), to_dtype(fo["rstd"], F32).cuda()
    smu = to_dtype(fo["mean"], F32).cuda() if norm else None
    dev = {k: v.cuda() for k, v in d.items()}
    sl = lambda x, q: x[q * tl:(q + 1) * tl]
    mk = lambda *s, dt=BF: torch.empty(*s, dtype=dt, device="cuda")
    results = []
    for fused in (False, True):
        groups = [Group(tl, G, h, ffn, S, layer, T, norm) for _ in range(G)]
        peers, slabs = make_peers(groups, layer, T, True)
        dY, dW, dR = mk(t, T, K), mk(t, h, K, dt=F32), mk(t, T, h)
        dgs = [mk(h, dt=F32) for _ in range(G)]
        dbs = [mk(h, dt=F32) if norm else None for _ in range(G)]
        for q, (g, pe) in enumerate(zip(groups, peers)):
            args = (layer, T, sl(dev["dX"], q), sl(dev["dHn"], q), sl(dev["W"], q), sl(sHn, q), sl(srs, q).clone(),
                    sl(smu, q).clone() if norm else None, dev["gamma"], sl(dR, q), dgs[q], dbs[q])
            if fused:
                g.ctx.tp_backward_local_push(*args, pe, 3, g.ws)
            else:
                g.ctx.tp_backward_local(*args, g.ws)
        exchange(groups, peers, layer, T, True, epoch=3, scatter=not fused)
        for q, g in enumerate(groups):
            g.ctx.tp_backward_finish(layer, T, sl(dev["Y"], q), sl(dev["W"], q), sl(dR, q), sl(dY, q), sl(dW, q), g.ws)
        torch.cuda.synchronize()
        assert all(g.ctx.last_device_status() == caat.CAAT_OK for g in groups)
        results.append((slabs[0].clone(), dY, dW, dR, torch.stack(dgs).sum(0)))
    for a, b, name in zip(results[0], results[1], ("slab", "dY", "dW", "dR", "dgamma")):
        assert torch.equal(a, b), name
    ob = O.rowpar_backward(f64(d["dX"]), f64(d["dHn"]), f64(d["Y"]), f64(d["W"]), f64(sHn.cpu()), f64(srs.cpu()),
                           f64(smu.cpu()) if norm else None, f64(d["gamma"]), S=S, alpha=float(np.sqrt(t)), norm=norm)
    assert_close(results[1][1].cpu(), ob["dY"], "bf16", "dY (fused) against the oracle")
    assert_close(results[1][2].cpu(), ob["dW"], "bf16", "dW (fused) against the oracle")
