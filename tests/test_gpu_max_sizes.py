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
