"""Calls from several host threads at once: each thread has its own stream, workspace and outputs and shares only
the (read-only) context and inputs; the library's host-side caches and the fork / join of the block forward's second
stream are the shared state under test.  Every thread's results must be bit-identical to the same calls made alone.
Needs a GPU."""
import threading

import pytest
import torch

from oracle import caat_oracle as O
from paper_2506_19645_b200 import caat, synthetic

pytestmark = pytest.mark.gpu


def _run_block(ctx, w, dev, rounds):
    t, T, h = w.t, w.tokens, w.h
    mk = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt, device="cuda")
    f32 = torch.float32
    o = {"Hn1": mk(t, T, h), "X1": mk(t, T, h), "rstd1": mk(t, T, dt=f32), "Hn2": mk(t, T, h), "X2": mk(t, T, h),
         "rstd2": mk(t, T, dt=f32), "dY_attn": mk(t, T, w.kr_attn), "dW_o": mk(t, h, w.kr_attn, dt=f32),
         "dY_mlp": mk(t, T, w.kr_mlp), "dW_down": mk(t, h, w.kr_mlp, dt=f32), "dR0": mk(t, T, h), "dHn1": mk(t, T, h),
         "dgamma1": mk(h, dt=f32), "dgamma2": mk(h, dt=f32)}
    ws = ctx.alloc_workspace(ctx.block_workspace_bytes(T, True))
    for _ in range(rounds):
        ctx.block_forward(T, dev["Y_attn"], dev["W_o"], dev["Y_mlp"], dev["W_down"], dev["R0"], dev["gamma1"], None,
                          dev["gamma2"], None, o["Hn1"], o["X1"], o["rstd1"], None, o["Hn2"], o["X2"], o["rstd2"], None, ws)
        ctx.block_backward(T, dev["dX1"], dev["dX2"], dev["dHn2"], dev["Y_attn"], dev["W_o"], dev["Y_mlp"], dev["W_down"],
                           o["Hn1"], o["rstd1"], None, o["Hn2"], o["rstd2"], None, dev["gamma1"], dev["gamma2"], o["dY_attn"],
                           o["dW_o"], o["dY_mlp"], o["dW_down"], o["dR0"], o["dHn1"], o["dgamma1"], None, o["dgamma2"], None, ws)
    torch.cuda.current_stream().synchronize()
    return o


def test_block_calls_from_four_threads_equal_the_single_threaded_results():
    w = synthetic.Workload("blk_threads", 4, 700, 768, 3072, 0.5, "bf16", "block", True, 21)
    dev = {k: v.cuda() for k, v in synthetic.block_inputs(w, O.shared_channels(w.h, w.p)).items()}
    ctx = caat.Context(w.h, w.ffn, w.t, w.p, "bf16")
    ctx.set_option(caat.CAAT_OPT_BLOCK_OVERLAP, 1)          # the fork / join on the library's own stream, from every thread
    ref = _run_block(ctx, w, dev, 1)
    torch.cuda.synchronize()
    results, errors = [None] * 4, []

    def worker(n):
        try:
            torch.cuda.set_device(0)
            with torch.cuda.stream(torch.cuda.Stream()):
                results[n] = _run_block(ctx, w, dev, 6)
        except Exception as ex:  # noqa: BLE001
            errors.append(repr(ex))

    threads = [threading.Thread(target=worker, args=(n,)) for n in range(4)]
    for th in threads:
        th.start()
    for th in threads:
        th.join(timeout=300)
    torch.cuda.synchronize()
    assert not errors, errors
    assert ctx.last_device_status() == caat.CAAT_OK
    for n, o in enumerate(results):
        assert o is not None, f"thread {n} did not finish"
        for k in ref:
            assert torch.equal(o[k], ref[k]), f"thread {n}: {k}"
