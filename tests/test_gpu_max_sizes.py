"""Large-extent case: more than 2^31 elements per activation tensor (t = 8, T = 66000, h = 4096), so every
kernel's index arithmetic has to be 64-bit.  Tokens are independent rows in everything except dW and dgamma,
so the oracle checks sampled tokens (forward outputs, dY, dR) on the subset alone; the token sums (dW, dgamma)
are checked by a property that holds at any size: the sum over all tokens equals the sum of the two halves'
results, each computed by a separate call.  About 45 GB of device memory.  Needs a GPU."""
import numpy as np
import pytest
import torch

from oracle import caat_oracle as O
from paper_2506_19645_b200 import caat
from tests.helpers import assert_close, f64

pytestmark = pytest.mark.gpu


def _randn(shape, gen, std=1.0):
    out = torch.empty(shape, dtype=torch.bfloat16, device="cuda")
    flat = out.view(-1)
    step = 1 << 28
    for a in range(0, flat.numel(), step):       # fp32 draws in slabs, rounded to bf16
        n = min(step, flat.numel() - a)
        flat[a:a + n] = (torch.randn(n, generator=gen, device="cuda") * std).to(torch.bfloat16)
    return out


def test_rowpar_beyond_2_31_elements():
    free, _ = torch.cuda.mem_get_info()
    if free < 60 * 2 ** 30:
        pytest.skip("needs about 45 GB of free device memory")
    t, T, h, ffn, S = 8, 66000, 4096, 11008, 2048
    assert t * T * h > 2 ** 31
    k = h // t
    ctx = caat.Context(h, ffn, t, 0.5, "bf16")
    alpha = ctx.private_scale
    gen = torch.Generator(device="cuda").manual_seed(5)
    Y, W = _randn((t, T, k), gen), _randn((t, h, k), gen, 0.02)
    R = _randn((t, T, h), gen)
    R[1:, :, :S] = R[0:1, :, :S]
    gamma = (1 + 0.1 * torch.randn(h, generator=gen, device="cuda")).to(torch.bfloat16)
    rng = np.random.default_rng(11)
    tok = np.sort(np.concatenate([rng.choice(T, size=20, replace=False), [0, T - 1, 65535, 65536]])).astype(np.int64)
    tk = torch.from_numpy(tok).cuda()
    sub = lambda x: f64(x.index_select(1, tk).cpu())

    # ---- forward: sampled tokens against the oracle on those tokens alone
    Hn, X = torch.empty_like(R), torch.empty_like(R)
    rstd = torch.empty((t, T), dtype=torch.float32, device="cuda")
    ws = ctx.alloc_workspace(ctx.workspace_bytes(caat.CAAT_ATTN_OUT, T, True))
    ctx.rowpar_forward(caat.CAAT_ATTN_OUT, T, Y, W, R, gamma, None, Hn, X, rstd, None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    fo = O.rowpar_forward(sub(Y), f64(W.cpu()), sub(R), f64(gamma.cpu()), None, S=S, alpha=alpha)
    assert_close(Hn.index_select(1, tk).cpu(), fo["Hn"], "bf16", "Hn")
    assert_close(X.index_select(1, tk).cpu(), fo["X"], "bf16", "X")
    assert_close(rstd.index_select(1, tk).cpu(), fo["rstd"], "bf16", "rstd")
    del X

    # ---- backward on synthetic saved tensors (any Hn, any positive rstd define a valid backward problem)
    Hs = R                                      # reuse the residual buffer as the "saved stream"
    rs = (0.5 + torch.rand((t, T), generator=gen, device="cuda")).float()
    dX = _randn((t, T, h), gen)
    dHn = Hn                                    # reuse: its values are just another input here
    dY = torch.empty_like(Y)
    dW = torch.empty((t, h, k), dtype=torch.float32, device="cuda")
    dR = torch.empty((t, T, h), dtype=torch.bfloat16, device="cuda")
    dg = torch.empty(h, dtype=torch.float32, device="cuda")
    ctx.rowpar_backward(caat.CAAT_ATTN_OUT, T, dX, dHn, Y, W, Hs, rs, None, gamma, dY, dW, dR, dg, None, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    bo = O.rowpar_backward(sub(dX), sub(dHn), sub(Y), f64(W.cpu()), sub(Hs), f64(rs.index_select(1, tk).cpu()), None,
                           f64(gamma.cpu()), S=S, alpha=alpha)
    assert_close(dY.index_select(1, tk).cpu(), bo["dY"], "bf16", "dY")
    assert_close(dR.index_select(1, tk).cpu(), bo["dR"], "bf16", "dR")

    # ---- token sums: whole call == sum of two half calls (fp32 outputs; different summation orders only)
    half = T // 2
    parts_W, parts_g = [], []
    for a, b in ((0, half), (half, T)):
        n = b - a
        sl = lambda x: x[:, a:b].contiguous()
        dW2 = torch.empty_like(dW); dg2 = torch.empty_like(dg)
        dY2 = torch.empty((t, n, k), dtype=torch.bfloat16, device="cuda")
        dR2 = torch.empty((t, n, h), dtype=torch.bfloat16, device="cuda")
        ctx.rowpar_backward(caat.CAAT_ATTN_OUT, n, sl(dX), sl(dHn), sl(Y), W, sl(Hs), sl(rs), None, gamma, dY2, dW2, dR2,
                            dg2, None, ws)
        torch.cuda.synchronize()
        assert ctx.last_device_status() == caat.CAAT_OK
        assert torch.equal(dR2, dR[:, a:b])      # per-token outputs do not depend on how tokens are batched
        parts_W.append(dW2); parts_g.append(dg2)
        del dY2, dR2
    assert_close((parts_W[0] + parts_W[1]).cpu(), f64(dW.cpu()), "f32", "dW halves")
    assert_close((parts_g[0] + parts_g[1]).cpu(), f64(dg.cpu()), "f32", "dgamma halves")


@pytest.mark.parametrize("T,norm", [(3, 0), (40, 1)])
def test_longest_rows_with_few_tokens(T, norm):
    # h = 16384, the longest row the library takes (2048 16-byte chunks): the few-token row kernels keep a whole
    # row in shared memory as fp32, 64 KB here - more than a kernel gets without asking for it
    from paper_2506_19645_b200 import synthetic
    t, h, ffn, S = 2, 16384, 16384, 8192
    ctx = caat.Context(h, ffn, t, 0.5, "bf16")
    ctx.set_option(caat.CAAT_OPT_NORM, norm)
    layer, k = caat.CAAT_MLP_DOWN, ffn // t
    d = synthetic.layer_inputs(t, T, h, k, "bf16", seed=T, S=S)
    dev = {n: v.cuda() for n, v in d.items()}
    out = ctx.alloc_forward_outputs(T)
    mean = torch.empty((t, T), dtype=torch.float32, device="cuda") if norm else None
    ws = ctx.alloc_workspace(ctx.workspace_bytes(layer, T, False))
    ctx.rowpar_forward(layer, T, dev["Y"], dev["W"], dev["R"], dev["gamma"], dev["beta"] if norm else None, out["Hn"], out["X"],
                       out["rstd"], mean, ws)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    fo = O.rowpar_forward(f64(d["Y"]), f64(d["W"]), f64(d["R"]), f64(d["gamma"]), f64(d["beta"]) if norm else None, S=S,
                          alpha=ctx.private_scale, norm=norm)
    for name in ("Hn", "X", "rstd"):
        assert_close(out[name].cpu(), fo[name], "bf16", name)
