"""Every device-side wait of the tensor-core GEMM and of the bulk-copy row kernels is bounded: when a stage never
fills, the roles give up, raise the status word, let their copies in flight land and leave through the normal exit,
and the host reads CAAT_ETIMEOUT from caat_last_device_status while the CUDA context stays usable.  The case is made
on the host side: a switch of the kernel announces bytes to the stage barrier that never arrive (the GEMM: its A
boxes, not issued; the row kernels: 16 bytes on top of their copies), and a short poll limit keeps the run to
milliseconds.  Runs in child processes because the switches are read from the environment once per process.
Needs a GPU."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

CHILD = r"""
import torch
from paper_2506_19645_b200 import caat, synthetic
t, T, h, ffn = 2, 512, 512, 2048
ctx = caat.Context(h, ffn, t, 0.5, "bf16")
k = ctx.k_r(caat.CAAT_ATTN_OUT)
d = synthetic.layer_inputs(t, T, h, k, "bf16", seed=1, S=ctx.shared_channels, device="cuda")
mk = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt, device="cuda")
Hn, X, rstd = mk(t, T, h), mk(t, T, h), mk(t, T, dt=torch.float32)
ws = ctx.alloc_workspace(ctx.workspace_bytes(caat.CAAT_ATTN_OUT, T, False))
ctx.rowpar_forward(caat.CAAT_ATTN_OUT, T, d["Y"], d["W"], d["R"], d["gamma"], None, Hn, X, rstd, None, ws)
torch.cuda.synchronize()                      # the kernels returned: no hang, no CUDA error
first = ctx.last_device_status()
second = ctx.last_device_status()             # reading the status clears it
x = torch.ones(1024, device="cuda").sum().item()   # the context still works
print("STATUS", first, second, int(x))
"""


def test_gemm_wait_runs_out_and_reports_timeout():
    from paper_2506_19645_b200 import caat
    env = dict(os.environ, CAAT_TC_DEBUG="1024", CAAT_TC_SPINCAP="2048")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", CHILD], env=env, cwd=root, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("STATUS")][-1].split()
    assert int(line[1]) == caat.CAAT_ETIMEOUT
    assert int(line[2]) == caat.CAAT_OK
    assert int(line[3]) == 1024


ROWS_CHILD = r"""
import torch
from paper_2506_19645_b200 import caat, synthetic
mk = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt, device="cuda")
f32 = torch.float32
out = []
# (h, S, rows option): staged forward + lean backward, staged forward + staged backward (partition off a multiple
# of 8), warp-per-token forward + backward
for h, S, rows in ((2048, 1024, 2), (2048, 1020, 2), (512, 256, 0)):
    t, T, ffn = 2, 200, 4 * h
    ctx = caat.Context(h, ffn, t, 0.5, "bf16")
    ctx.set_option(caat.CAAT_OPT_SHARED_CHANNELS, S)
    ctx.set_option(caat.CAAT_OPT_ROWS, rows)
    ctx.set_option(caat.CAAT_OPT_GEMM, 1)          # the CUDA-core GEMM: the stalled waits are the row kernels' own
    layer = caat.CAAT_ATTN_OUT
    k = ctx.k_r(layer)
    d = synthetic.layer_inputs(t, T, h, k, "bf16", seed=1, S=S, backward=True, device="cuda")
    Hn, X, rstd = mk(t, T, h), mk(t, T, h), mk(t, T, dt=f32)
    ws = ctx.alloc_workspace(ctx.workspace_bytes(layer, T, True))
    ctx.rowpar_forward(layer, T, d["Y"], d["W"], d["R"], d["gamma"], None, Hn, X, rstd, None, ws)
    torch.cuda.synchronize()
    out += [ctx.last_device_status(), ctx.last_device_status()]
    Hn.normal_(); rstd.fill_(1.0)
    ctx.rowpar_backward(layer, T, d["dX"], d["dHn"], d["Y"], d["W"], Hn, rstd, None, d["gamma"], mk(t, T, k),
                        mk(t, h, k, dt=f32), mk(t, T, h), mk(h, dt=f32), None, ws)
    torch.cuda.synchronize()
    out += [ctx.last_device_status(), ctx.last_device_status()]
x = torch.ones(1024, device="cuda").sum().item()   # the context still works
print("STATUS", *out, int(x))
"""


def test_row_kernel_waits_run_out_and_report_timeout():
    from paper_2506_19645_b200 import caat
    env = dict(os.environ, CAAT_ROWS_STALL="1", CAAT_ROWS_SPINCAP="64")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", ROWS_CHILD], env=env, cwd=root, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [int(v) for v in [l for l in out.stdout.splitlines() if l.startswith("STATUS")][-1].split()[1:]]
    # every launch of a bulk-copy row kernel (forward, backward; three configurations) timed out and said so once
    assert line[:-1] == [caat.CAAT_ETIMEOUT, caat.CAAT_OK] * 6
    assert line[-1] == 1024
