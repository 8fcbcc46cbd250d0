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
logic) on the current stream - or, with ``exchange="push"``, the library's own exchange kernels over peer memory
(reduce-scatter by token slice into per-source slots of the owner, fp32 sum in fixed order, all-gather by peer
stores; the forward GEMM stores its shared tiles straight into the owners' slots): 16-bit wire, fp32 accumulation,
no cast and no library collective on the slab.  The peers' addresses come from torch's symmetric memory
(``PeerBuffers``).  Not run on more than one GPU so far: this module is exercised with one GPU per
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


def _align(n: int, a: int = 256) -> int:
    return (n + a - 1) // a * a


class PeerBuffers:
    """This GPU's buffers of the peer-memory exchange for one (layer, tokens) shape - the workspace (it holds the
    slab), the receive slots and the flag words - in ONE symmetric-memory allocation, so that a single rendezvous
    yields every peer's addresses.  `addresses` may be injected (a list of base addresses, one per GPU) where the
    peers are not separate processes (single-GPU tests)."""

    def __init__(self, ctx, layer, tokens, group=None, device="cuda", addresses=None, rank=None):
        from . import caat
        self.ctx, self.layer, self.tokens = ctx, layer, tokens
        world = len(addresses) if addresses is not None else group_size(group)
        self.world = world
        ws_bytes = _align(ctx.workspace_bytes(layer, tokens, True))
        recv_bytes, self.slice_rows = ctx.tp_exchange_bytes(layer, tokens, world)
        self.offsets = (0, ws_bytes, ws_bytes + recv_bytes)
        total = ws_bytes + recv_bytes + caat.CAAT_TP_FLAG_BYTES
        if addresses is None:
            import torch.distributed._symmetric_memory as symm_mem
            self.buf = symm_mem.empty(total, dtype=torch.uint8, device=device)
            self.handle = symm_mem.rendezvous(self.buf, group if group is not None else dist.group.WORLD)
            addresses = [int(self.handle.buffer_ptrs[q]) for q in range(world)]
            rank = dist.get_rank(group)
        else:
            self.buf = torch.empty(total, dtype=torch.uint8, device=device)
            addresses = list(addresses)
            addresses[rank] = self.buf.data_ptr()
        self.rank = rank
        self.workspace = self.buf[:ws_bytes]
        self.buf[self.offsets[2]:].zero_()                       # the flag words start at zero, once
        self.epoch = 0
        self._addresses = addresses
        self._peers = {}
        if dist.is_available() and dist.is_initialized() and world > 1:
            torch.cuda.synchronize()
            dist.barrier(group)                                   # no flag is raised before every GPU has zeroed its own

    def peers(self, backward: bool):
        """caat_peers for the forward or the backward slab (they sit at different workspace offsets)."""
        key = bool(backward)
        if key not in self._peers:
            slab = self.ctx.tp_slab(self.layer, self.tokens, backward, self.workspace)
            slab_off = slab.data_ptr() - self.buf.data_ptr()
            a = self._addresses
            self._peers[key] = self.ctx.make_peers(self.rank, [x + self.offsets[1] for x in a], [x + slab_off for x in a],
                                                   [x + self.offsets[2] for x in a])
        return self._peers[key]

    def next_epoch(self) -> int:
        self.epoch = (self.epoch + 1) & 0xFFFFFFFF
        return self.epoch


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
        self._peer_buffers = {}

    def peer_buffers(self, layer, tokens, device="cuda") -> PeerBuffers:
        """Buffers for exchange="push" (allocated and registered with the peers on first use: a collective call)."""
        key = (layer, tokens)
        if key not in self._peer_buffers:
            if self.world == 1:     # no peers to meet: plain device memory, this GPU's own address
                self._peer_buffers[key] = PeerBuffers(self.ctx, layer, tokens, device=device, addresses=[0], rank=0)
            else:
                self._peer_buffers[key] = PeerBuffers(self.ctx, layer, tokens, self.group, device)
        return self._peer_buffers[key]

    def forward_push(self, layer, tokens, Y, W, R, gamma, beta, Hn, X, rstd, mean, pb: PeerBuffers):
        """The forward with the library's own exchange over peer memory; `pb.workspace` is the layer's workspace."""
        c = self.ctx
        if c.shared_channels == 0:
            c.tp_forward_local(layer, tokens, Y, W, pb.workspace)
        else:
            pe, epoch = pb.peers(False), pb.next_epoch()
            if pb.slice_rows % 256 == 0:          # whole output tiles per owner: the GEMM stores them into the owners' slots
                c.tp_forward_local_push(layer, tokens, Y, W, pe, epoch, pb.workspace)
            else:
                c.tp_forward_local(layer, tokens, Y, W, pb.workspace)
                c.tp_exchange_scatter(layer, tokens, False, pe, epoch, pb.workspace)
            c.tp_exchange_reduce(layer, tokens, pe, epoch)
            c.tp_exchange_wait(pe, epoch)
        c.tp_forward_finish(layer, tokens, R, gamma, beta, Hn, X, rstd, mean, pb.workspace)

    def backward_push(self, layer, tokens, dX, dHn, Y, W, Hn, rstd, mean, gamma, dY, dW, dR, dgamma, dbeta, pb: PeerBuffers):
        c = self.ctx
        if c.shared_channels > 0:     # the row kernel sends each token's reduced gradient row to its owner's slot
            pe, epoch = pb.peers(True), pb.next_epoch()
            c.tp_backward_local_push(layer, tokens, dX, dHn, W, Hn, rstd, mean, gamma, dR, dgamma, dbeta, pe, epoch,
                                     pb.workspace)
            c.tp_exchange_reduce(layer, tokens, pe, epoch)
            c.tp_exchange_wait(pe, epoch)
        else:
            c.tp_backward_local(layer, tokens, dX, dHn, W, Hn, rstd, mean, gamma, dR, dgamma, dbeta, pb.workspace)
        allreduce_slab(dgamma, self.group)          # fp32 [h], a few KB: the library collective
        if dbeta is not None:
            allreduce_slab(dbeta, self.group)
        c.tp_backward_finish(layer, tokens, Y, W, dR, dY, dW, pb.workspace)

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
