"""The N > 1 path of the benchmark on CPU: two gloo ranks, independent replicas, time = max over ranks."""
import os

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2506_19645_b200 import replicas


def _worker(rank, world, port, out):
    os.environ.update({"MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port), "RANK": str(rank),
                       "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world)})
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert replicas.rank_env() == (rank, rank, world)
        replicas.barrier()
        ms_local = 10.0 + 3.0 * rank                      # rank 1 is the slow one
        ms = replicas.max_over_ranks(ms_local)
        rate = replicas.whole_job_rate(16384, 5, world, ms)
        out.put((rank, ms, rate))
        replicas.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_time_is_max_over_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, rate in got:
        assert ms == pytest.approx(13.0)                                   # the slowest rank's time, on every rank
        assert rate == pytest.approx(2 * 16384 * 5 / 13.0e-3)              # whole-job tokens/s over both replicas


def test_single_process_is_identity():
    assert replicas.max_over_ranks(7.5) == 7.5
    assert replicas.whole_job_rate(100, 2, 1, 4.0) == pytest.approx(100 * 2 / 4e-3)
    replicas.barrier()
