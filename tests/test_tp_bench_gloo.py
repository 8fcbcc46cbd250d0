"""The `bench.py --mode tp` path on CPU: two gloo ranks walk the p sweep with a stand-in for the GPU layers (the
kernels are covered on a GPU by tests/test_gpu_tp.py), so the plan, the collectives, the timing protocol
(barrier, max over ranks) and the printed line are exercised end to end."""
import io
import json
import os
import types

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import caat_oracle as O
from paper_2506_19645_b200 import tp, tp_bench


class _CpuLayers:
    """Stands in for the library calls of one GPU: only the exchange steps of a block step run (on CPU tensors)."""

    def __init__(self, pl, p, device, group=None):
        self.pl, self.group = pl, group
        self.S = O.shared_channels(pl["h"], p)
        self.payload_elems = pl["tokens"] * self.S
        self.slab = torch.ones((pl["tokens"], self.S), dtype=torch.bfloat16)
        self.payload_keys = ("16bit", "fp32")
        self.calls = 0

    def step(self):
        if self.S > 0:
            for _ in range(2):
                tp.allreduce_slab(self.slab.clone(), self.group)                     # forward, 16-bit
            for _ in range(2):
                tp.allreduce_slab(self.slab.clone(), self.group, torch.float32)     # backward, carried in fp32
        self.calls += 1

    def sync(self):
        pass

    def check(self):
        pass

    def slab_like(self, dtype):
        return torch.zeros((self.pl["tokens"], self.S), dtype=dtype)


def _worker(rank, world, port, out):
    os.environ.update({"MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port), "RANK": str(rank),
                       "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world)})
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        args = types.SimpleNamespace(workload="block_130m", steps=3, warmup=1, tokens=64)
        buf = io.StringIO()
        rows = tp_bench.run(args, make_layers=_CpuLayers, backend="gloo", out=buf)
        out.put((rank, rows, buf.getvalue()))
    finally:
        dist.destroy_process_group()


def test_tp_mode_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 33500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted((out.get(timeout=180) for _ in procs), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, rows0, text0), (_, rows1, text1) = got
    assert text1 == ""                                    # only rank 0 prints
    line = json.loads(text0)
    assert line["mode"] == "tp" and line["n_gpus"] == 2 and line["config"]["tp_ranks"] == 4
    assert line["config"]["ranks_per_gpu"] == 2
    assert [r["p"] for r in line["p_sweep"]] == [1.0, 0.75, 0.5, 0.25, 0.0]
    for r0, r1 in zip(rows0, rows1):
        assert r0["ms_per_step"] == pytest.approx(r1["ms_per_step"])      # the max over ranks, on every rank
        assert r0["S"] == O.shared_channels(768, r0["p"])
        assert r0["payload_bytes_16bit"] == 64 * r0["S"] * 2              # App. D: tokens * S elements per reduce
        if r0["S"] > 0:
            assert r0["allreduce_busbw_gbs_16bit"] > 0 and r0["allreduce_busbw_gbs_fp32"] > 0
        assert "model_ms_per_step" in r0 and r0["model_ms_per_step"] > 0
    assert line["p_sweep"][0]["model_speedup_vs_p1"] == pytest.approx(1.0)


def test_plan_and_bus_bandwidth():
    pl = tp_bench.plan("block_7b", 8)
    assert (pl["t_local"], pl["t_total"], pl["kr_attn"], pl["kr_mlp"]) == (1, 8, 512, 1376)
    pl = tp_bench.plan("block_7b", 2)
    assert (pl["t_local"], pl["t_total"]) == (4, 8)
    with pytest.raises(SystemExit):
        tp_bench.plan("block_130m", 7)                    # 7 ranks do not divide h = 768
    # 1 GB over 8 ranks in 2.414 ms is 725 GB/s of bus bandwidth
    assert tp_bench.bus_bandwidth_gbs(10 ** 9, 8, 2.4138) == pytest.approx(725.0, rel=1e-3)
    assert tp_bench.bus_bandwidth_gbs(10 ** 9, 1, 1.0) == 0.0
