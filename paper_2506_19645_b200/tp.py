"""The row-parallel CAAT layer over several GPUs: one group of ``t`` tensor-parallel ranks per GPU, and between
the two halves of the library's layer call the all-reduce of the shared-channel slab (Section 3; Appendix D:
reduce-scatter + all-gather of tokens * S elements, a fraction p of a full all-reduce).

Argument marshalling and the collective only: every arithmetic step of the layer runs in the library's kernels.
The one exception is off the kernels' path: a library collective accumulates in its payload type, and a chain of
16-bit partial sums over 8 ranks leaves the layer output outside the 2e-2 tolerance against the exact sum (measured:
2.3e-2), so by default the slab is carried through the collective in fp32, forward and backward (Section 4 asks
for fp32 accumulation of the backward reduce; the forward is held to the same), which costs a cast before and
after it and twice the wire bytes.  ``forward_accumulate=None`` / ``backward_accumulate=None`` send the 16-bit
slab as it is.  With a process group of one the collective is skipped and the layer
equals ``rowpar_forward`` / ``rowpar_backward``.

The collective is ``torch.distributed.all_reduce`` (NCCL between GPUs, gloo in CPU tests of this module's own
logic) on the current stream.  Not run on more than one GPU so far: this module is exercised with one GPU per
process only when such a machine is available; its arithmetic is checked on a single GPU by running the groups
one after the other (tests/test_gpu_tp.py) and its collective step with gloo (tests/test_tp_gloo.py)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def group_size(group=None) -> int:
    return dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1


def allreduce_slab(slab: torch.Tensor, group=None, accumulate_dtype=None) -> torch.Tensor:
    """Sums ``slab`` over the ranks of ``group`` in place.  ``accumulate_dtype`` (e.g. ``torch.float32``) carries
    the slab through the collective in that type and rounds once at the end."""
    if group_size(group) == 1:
        return slab
    if accumulate_dtype is None or accumulate_dtype == slab.dtype:
        dist.all_reduce(slab, op=dist.ReduceOp.SUM, group=group)
        return slab
    wide = slab.to(accumulate_dtype)
    dist.all_reduce(wide, op=dist.ReduceOp.SUM, group=group)
    slab.copy_(wide)
    return slab


class TensorParallelRowLinear:
    """``t_local`` ranks of a ``t_local * world`` tensor-parallel group on this GPU.  Tensors are the ones of
    ``Context.rowpar_forward`` / ``rowpar_backward`` restricted to this GPU's ranks (``K_r = K / (t_local * world)``)."""

    def __init__(self, h, ffn, t_local, p, dtype="bf16", group=None, backward_accumulate=torch.float32,
                 forward_accumulate=torch.float32):
        from . import caat
        self.caat = caat
        self.group = group
        self.world = group_size(group)
        self.ctx = caat.Context(h, ffn, t_local, p, dtype)
        self.ctx.set_option(caat.CAAT_OPT_TP_GROUPS, self.world)     # also sets alpha = sqrt(t_local * world)
        self.backward_accumulate = backward_accumulate
        self.forward_accumulate = forward_accumulate

    def workspace(self, layer, tokens, backward=True, device="cuda"):
        return self.ctx.alloc_workspace(self.ctx.workspace_bytes(layer, tokens, backward), device=device)

    def forward(self, layer, tokens, Y, W, R, gamma, beta, Hn, X, rstd, mean, workspace):
        c = self.ctx
        c.tp_forward_local(layer, tokens, Y, W, workspace)
        if c.shared_channels > 0:
            allreduce_slab(c.tp_slab(layer, tokens, False, workspace), self.group, self.forward_accumulate)
        c.tp_forward_finish(layer, tokens, R, gamma, beta, Hn, X, rstd, mean, workspace)

    def backward(self, layer, tokens, dX, dHn, Y, W, Hn, rstd, mean, gamma, dY, dW, dR, dgamma, dbeta, workspace):
        c = self.ctx
        c.tp_backward_local(layer, tokens, dX, dHn, W, Hn, rstd, mean, gamma, dR, dgamma, dbeta, workspace)
        if c.shared_channels > 0:
            allreduce_slab(c.tp_slab(layer, tokens, True, workspace), self.group, self.backward_accumulate)
        allreduce_slab(dgamma, self.group)          # fp32 [h]: the norm parameters are replicated (Eq. 10-11)
        if dbeta is not None:
            allreduce_slab(dbeta, self.group)
        c.tp_backward_finish(layer, tokens, Y, W, dR, dY, dW, workspace)
