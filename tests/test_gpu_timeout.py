"""Every device-side wait of the tensor-core GEMM is bounded: when a stage never fills, the roles give up,
raise the status word, let their copies in flight land and leave through the normal exit, and the host reads
CAAT_ETIMEOUT from caat_last_device_status while the CUDA context stays usable.  The case is made on the host
side: a measurement switch of the kernel announces the A boxes to the stage barrier without issuing them, and a
short poll limit keeps the run to milliseconds.  Runs in a child process because both switches are read from the
environment once per process.  Needs a GPU."""
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
