"""caat_rowpar_forward_noalloc: the forward for callers that cannot allocate device memory at call
time (a serving loop with a frozen memory pool, a framework that forbids allocation on its compute
stream, a process whose device memory is managed elsewhere).  It takes no workspace: its scratch
is a fixed array inside the library.  The test calls it through the C ABI twice in a row, with
different inputs and sizes, and checks every output against the regular entry point's.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.  Passes alone in a fresh process and after the other tests."""
import pytest
import torch

from paper_2506_19645_b200 import caat, synthetic
from tests.helpers import TOL, rel_err

pytestmark = pytest.mark.gpu


def _regular(ctx, layer, d, T):
    out = ctx.alloc_forward_outputs(T)
    ws = ctx.alloc_workspace(ctx.workspace_bytes(layer, T, False))
    ctx.rowpar_forward(layer, T, d["Y"], d["W"], d["R"], d["gamma"], None, out["Hn"], out["X"], out["rstd"], None, ws)
    torch.cuda.synchronize()
    return out


def _noalloc(ctx, layer, d, T):
    out = ctx.alloc_forward_outputs(T)      # outputs are still the caller's; only the scratch is built in
    ctx.rowpar_forward_noalloc(layer, T, d["Y"], d["W"], d["R"], d["gamma"], None, out["Hn"], out["X"], out["rstd"], None)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    return out


def test_noalloc_forward_matches_regular_entry_point_twice():
    t, h, ffn, p = 4, 768, 3072, 0.5
    ctx = caat.Context(h, ffn, t, p, "bf16")
    layer = caat.CAAT_MLP_DOWN
    # two calls in a row; the second has other inputs and a smaller, ragged token count, so
    # anything the first call left in the shared scratch would show up as a mismatch
    for T, seed in ((700, 1), (333, 2)):
        d = {k: v.cuda() for k, v in synthetic.layer_inputs(t, T, h, ctx.k_r(layer), "bf16", seed=seed,
                                                            S=ctx.shared_channels).items()}
        ref = _regular(ctx, layer, d, T)
        got = _noalloc(ctx, layer, d, T)
        for name in ("Hn", "X", "rstd"):
            e = rel_err(got[name], ref[name].double().cpu().numpy())
            assert e <= TOL["bf16"], f"{name}: {e:.3e} (T={T})"


def test_noalloc_rejects_sizes_beyond_its_scratch():
    t, h, ffn = 8, 4096, 11008
    ctx = caat.Context(h, ffn, t, 0.5, "bf16")
    T = 4096                                         # scratch need: 4096 * (2048 + 8 * 2048) * 2 bytes = 144 MiB
    assert ctx.workspace_bytes(caat.CAAT_ATTN_OUT, T, False) > caat.CAAT_NOALLOC_SCRATCH_BYTES
    x = torch.zeros(8, device="cuda", dtype=torch.bfloat16)   # never dereferenced: rejected before any launch
    st = caat.lib.caat_rowpar_forward_noalloc(ctx._h, caat.CAAT_ATTN_OUT, T, *([x.data_ptr()] * 9), None)
    assert st == caat.CAAT_ELIMIT
    assert b"scratch" in caat.lib.caat_strerror(st)
