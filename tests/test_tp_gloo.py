"""The exchange step of the multi-GPU layer on CPU: two gloo ranks all-reduce a shared-channel slab, in the
slab's own type (the forward) and carried in fp32 (the backward, Section 4), and the fp32 norm-parameter
gradients.  The kernels on either side of the exchange are covered on a GPU (tests/test_gpu_tp.py)."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2506_19645_b200 import tp


def _slab(rank, T=37, S=24):
    g = torch.Generator().manual_seed(100 + rank)
    return torch.randn((T, S), generator=g).to(torch.bfloat16)


def _worker(rank, world, port, out):
    os.environ.update({"MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port), "RANK": str(rank),
                       "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world)})
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert tp.group_size() == world
        ws = torch.zeros(4096, dtype=torch.uint8)                 # a workspace; the slab is a view into it
        slab = ws[256:256 + 37 * 24 * 2].view(torch.bfloat16).view(37, 24)
        slab.copy_(_slab(rank))
        tp.allreduce_slab(slab, None, torch.float32)              # backward: fp32 through the collective
        fwd = _slab(rank).clone()
        tp.allreduce_slab(fwd)                                    # forward: the slab's own type
        dg = torch.full((16,), float(rank + 1))
        tp.allreduce_slab(dg)
        out.put((rank, ws[256:256 + 37 * 24 * 2].clone(), fwd, dg))
    finally:
        dist.destroy_process_group()


def test_slab_allreduce_two_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted((out.get(timeout=120) for _ in procs), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    exact = _slab(0).float() + _slab(1).float()                   # two bf16 values add exactly in fp32
    want = exact.to(torch.bfloat16)
    for rank, raw, fwd, dg in got:
        assert torch.equal(raw.view(torch.bfloat16).view(37, 24), want)     # one rounding, written through the view
        assert torch.equal(fwd, want)                                        # two terms: a 16-bit sum rounds the same
        assert torch.equal(dg, torch.full((16,), 3.0))


def test_group_of_one_is_identity():
    x = _slab(0)
    y = x.clone()
    assert tp.group_size() == 1
    tp.allreduce_slab(y, None, torch.float32)
    assert torch.equal(x, y)
