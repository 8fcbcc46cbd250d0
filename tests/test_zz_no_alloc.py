"""caat_rowpar_forward_noalloc: the forward for callers that cannot allocate device memory at call
time (a serving loop with a frozen memory pool, a framework that forbids allocation on its compute
stream, a process whose device memory is managed elsewhere).  It takes no workspace: its scratch
is a fixed array inside the library, shared by every call on the device and never cleared.

The tests call it through the C ABI several times in a row - different shapes, token counts and
kernel paths (large-batch tensor-core path, few-token path with its fp32 partial planes, CUDA-core
path for fp32 and for a partition that is not a multiple of 8), so every call finds the previous
call's leftovers in the scratch - and check that every output is bit-identical to the regular
entry point's (same kernels, deterministic), that it matches the fp64 oracle, and that a call
leaves the device's free memory and the framework's allocation count where they were.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.  Passes alone in a fresh process and after the other tests."""
import gc

import pytest
import torch

from oracle import caat_oracle as O
from paper_2506_19645_b200 import caat, synthetic
from tests.helpers import assert_close, f64

pytestmark = pytest.mark.gpu


def _ctx(t, h, ffn, dtype, S):
    ctx = caat.Context(h, ffn, t, 0.5, dtype)
    ctx.set_option(caat.CAAT_OPT_SHARED_CHANNELS, S)
    return ctx


def _inputs(ctx, layer, T, dtype, seed):
    return {k: v.cuda() for k, v in synthetic.layer_inputs(ctx.t, T, ctx.h, ctx.k_r(layer), dtype, seed=seed,
                                                           S=ctx.shared_channels).items()}


def _regular(ctx, layer, d, T):
    out = ctx.alloc_forward_outputs(T)
    ws = ctx.alloc_workspace(ctx.workspace_bytes(layer, T, False))
    ctx.rowpar_forward(layer, T, d["Y"], d["W"], d["R"], d["gamma"], None, out["Hn"], out["X"], out["rstd"], None, ws)
    torch.cuda.synchronize()
    return out


def _noalloc(ctx, layer, d, T, out=None):
    out = out or ctx.alloc_forward_outputs(T)      # outputs are still the caller's; only the scratch is built in
    ctx.rowpar_forward_noalloc(layer, T, d["Y"], d["W"], d["R"], d["gamma"], None, out["Hn"], out["X"], out["rstd"], None)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == caat.CAAT_OK
    return out


# (t, h, ffn, dtype, S, layer, T): consecutive calls differ in shape and path, so each runs on stale scratch
CALLS = [
    (4, 768, 3072, "bf16", 384, caat.CAAT_MLP_DOWN, 700),     # tensor-core GEMM + warp-per-token rows
    (4, 768, 3072, "bf16", 384, caat.CAAT_MLP_DOWN, 333),     # smaller, ragged token count
    (4, 1024, 4096, "bf16", 512, caat.CAAT_ATTN_OUT, 64),     # few tokens: fp32 partial planes in the scratch
    (4, 1024, 4096, "bf16", 256, caat.CAAT_MLP_DOWN, 8),
    (4, 1024, 4096, "bf16", 1024, caat.CAAT_MLP_DOWN, 1),     # one token, every channel shared
    (2, 256, 1024, "f32", 128, caat.CAAT_MLP_DOWN, 128),      # fp32: CUDA-core GEMM
    (4, 768, 3072, "bf16", 380, caat.CAAT_ATTN_OUT, 200),     # S % 8 != 0: CUDA-core GEMM, padded scratch columns
    (8, 2048, 5632, "bf16", 1024, caat.CAAT_MLP_DOWN, 500),   # long rows: staged row kernel
    (4, 768, 3072, "bf16", 384, caat.CAAT_MLP_DOWN, 700),     # the first call again, after all of the above
]


def test_noalloc_forward_equals_regular_entry_point_on_stale_scratch():
    for n, (t, h, ffn, dtype, S, layer, T) in enumerate(CALLS):
        ctx = _ctx(t, h, ffn, dtype, S)
        assert ctx.workspace_bytes(layer, T, False) <= caat.CAAT_NOALLOC_SCRATCH_BYTES
        d = _inputs(ctx, layer, T, dtype, seed=n + 1)
        ref = _regular(ctx, layer, d, T)
        got = _noalloc(ctx, layer, d, T)
        for name in ("Hn", "X", "rstd"):
            assert torch.equal(got[name], ref[name]), f"call {n} (T={T}, S={S}, {dtype}): {name} differs"
        fo = O.rowpar_forward(f64(d["Y"]), f64(d["W"]), f64(d["R"]), f64(d["gamma"]), None, S=S, alpha=ctx.private_scale)
        for name in ("Hn", "X", "rstd"):
            assert_close(got[name], fo[name], dtype, f"call {n}: {name} against the oracle")


def test_noalloc_call_allocates_nothing():
    t, h, ffn, S, layer = 4, 768, 3072, 384, caat.CAAT_MLP_DOWN
    ctx = _ctx(t, h, ffn, "bf16", S)
    for T in (600, 40):                       # large-batch path and few-token path
        d = _inputs(ctx, layer, T, "bf16", seed=5)
        out = ctx.alloc_forward_outputs(T)
        _noalloc(ctx, layer, d, T, out)       # the first call per device may load the module: not measured
        torch.cuda.synchronize()
        gc.collect()                          # leftovers of earlier tests must not be released in the middle of the check
        gc.disable()
        try:
            free0, _ = torch.cuda.mem_get_info()
            count0 = torch.cuda.memory_stats()["allocation.all.allocated"]
            alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
            _noalloc(ctx, layer, d, T, out)
            free1, _ = torch.cuda.mem_get_info()
            assert free1 == free0, f"T={T}: free device memory moved by {free0 - free1} bytes across the call"
            assert torch.cuda.memory_stats()["allocation.all.allocated"] == count0     # no request to the framework's allocator
            assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
        finally:
            gc.enable()


def test_noalloc_rejects_sizes_beyond_its_scratch():
    t, h, ffn = 8, 4096, 11008
    ctx = caat.Context(h, ffn, t, 0.5, "bf16")
    T = 4096                                         # scratch need: 4096 * (2048 + 8 * 2048) * 2 bytes = 144 MiB
    assert ctx.workspace_bytes(caat.CAAT_ATTN_OUT, T, False) > caat.CAAT_NOALLOC_SCRATCH_BYTES
    x = torch.zeros(8, device="cuda", dtype=torch.bfloat16)   # never dereferenced: rejected before any launch
    st = caat.lib.caat_rowpar_forward_noalloc(ctx._h, caat.CAAT_ATTN_OUT, T, *([x.data_ptr()] * 9), None)
    assert st == caat.CAAT_ELIMIT
    assert b"scratch" in caat.lib.caat_strerror(st)
