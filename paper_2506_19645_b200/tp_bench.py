"""``bench.py --gpus N --mode tp``: the row-parallel layers of a block under REAL tensor parallelism.

The workload's ``t`` tensor-parallel ranks are split over the ``N`` GPUs of the job (``t / N`` per GPU, at least
one).  Every step runs both row-parallel layers of a block forward and backward through
``tp.TensorParallelRowLinear``: the library's kernels on either side of an all-reduce of the packed
``[T, S]`` shared-channel slab (Section 3; Appendix D).  The synchronisation factor is swept over
``p in {1, 0.75, 0.5, 0.25, 0}`` and for each value the line reports

* the step time (device events, barrier on both sides, max over ranks) and tokens/s,
* the all-reduce of that payload timed alone, as bus bandwidth ``2 (n-1)/n * bytes / time``
  (16-bit forward payload and fp32 backward payload),
* what Appendix C's model predicts for the step from two measured numbers - the step without any exchange
  (``p = 0``) and the exchange time at ``p = 1``:  ``step(p) = step(0) + p * exchange(1)``.

Host-side orchestration only; no arithmetic of the method happens here.  The compute side is injectable
(``make_layers``) so that the plan, the collectives and the reporting can be exercised with gloo ranks on CPU.
"""
from __future__ import annotations

import json
import os
import sys
import time

import torch
import torch.distributed as dist

from . import replicas, synthetic, tp

P_SWEEP = (1.0, 0.75, 0.5, 0.25, 0.0)
ATTN_OUT, MLP_DOWN = 0, 1


def plan(workload: str, world: int, tokens: int = 0, exchange: str = "nccl") -> dict:
    """How the workload's ranks map onto `world` GPUs: ranks per GPU, total ranks, per-rank contraction widths."""
    w = synthetic.WORKLOADS[workload]
    if tokens > 0:
        w = w.with_tokens(tokens)
    t_local = max(1, w.t // world)
    t_total = t_local * world
    if w.h % t_total or w.ffn % t_total:
        raise SystemExit(f"--mode tp: {t_total} tensor-parallel ranks do not divide h={w.h} / ffn={w.ffn}")
    return {"workload": w.name, "tokens": w.tokens, "h": w.h, "ffn": w.ffn, "world": world, "t_local": t_local, "exchange": exchange,
            "t_total": t_total, "kr_attn": w.h // t_total, "kr_mlp": w.ffn // t_total, "backward": bool(w.backward)}


class _GpuLayers:
    """The two row-parallel layers of a block on this GPU's ranks, on synthetic tensors."""

    def __init__(self, pl: dict, p: float, device, group=None):
        from . import caat
        self.pl, self.group = pl, group
        self.exchange = pl.get("exchange", "nccl")
        self.lay = tp.TensorParallelRowLinear(pl["h"], pl["ffn"], pl["t_local"], p, "bf16", group)
        ctx = self.lay.ctx
        self.S = ctx.shared_channels
        t, T, h = pl["t_local"], pl["tokens"], pl["h"]
        rank = dist.get_rank() if dist.is_initialized() else 0
        self.layers = []
        mk = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt, device=device)
        f32 = torch.float32
        for layer in (caat.CAAT_ATTN_OUT, caat.CAAT_MLP_DOWN):
            k = ctx.k_r(layer)
            d = synthetic.layer_inputs(t, T, h, k, "bf16", seed=17 * rank + layer, S=self.S, backward=True, device=device)
            o = {"Hn": mk(t, T, h), "X": mk(t, T, h), "rstd": mk(t, T, dt=f32), "dY": mk(t, T, k),
                 "dW": mk(t, h, k, dt=f32), "dR": mk(t, T, h), "dg": mk(h, dt=f32)}
            self.layers.append((layer, d, o))
        self.payload_elems = T * self.S
        if self.exchange == "push":
            # the library's own exchange over peer memory: 16-bit wire both ways, fp32 accumulation at the owner
            self.pbs = [self.lay.peer_buffers(layer, T, device) for layer, _, _ in self.layers]
            self.ws = self.pbs[0].workspace
            self.payload_keys = ("16bit", "16bit")
        else:
            self.ws = ctx.alloc_workspace(ctx.block_workspace_bytes(T, True), device=device)
            key = lambda acc: "fp32" if acc == torch.float32 else "16bit"
            self.payload_keys = (key(self.lay.forward_accumulate), key(self.lay.backward_accumulate))

    def step(self):
        T, ws = self.pl["tokens"], self.ws
        if self.exchange == "push":
            for (layer, d, o), pb in zip(self.layers, self.pbs):
                self.lay.forward_push(layer, T, d["Y"], d["W"], d["R"], d["gamma"], None, o["Hn"], o["X"], o["rstd"], None, pb)
            if self.pl["backward"]:
                for (layer, d, o), pb in zip(reversed(self.layers), reversed(self.pbs)):
                    self.lay.backward_push(layer, T, d["dX"], d["dHn"], d["Y"], d["W"], o["Hn"], o["rstd"], None, d["gamma"],
                                           o["dY"], o["dW"], o["dR"], o["dg"], None, pb)
            return
        for layer, d, o in self.layers:
            self.lay.forward(layer, T, d["Y"], d["W"], d["R"], d["gamma"], None, o["Hn"], o["X"], o["rstd"], None, ws)
        if self.pl["backward"]:
            for layer, d, o in reversed(self.layers):
                self.lay.backward(layer, T, d["dX"], d["dHn"], d["Y"], d["W"], o["Hn"], o["rstd"], None, d["gamma"],
                                  o["dY"], o["dW"], o["dR"], o["dg"], None, ws)

    def sync(self):
        torch.cuda.synchronize()

    def check(self):
        from . import caat
        assert self.lay.ctx.last_device_status() == caat.CAAT_OK

    def slab_like(self, dtype):
        return torch.zeros((self.pl["tokens"], self.S), dtype=dtype, device=self.ws.device)


def _timed(fn, steps, sync, use_cuda_events):
    """Time of `steps` calls of fn between two barriers; the max over ranks, in ms per call."""
    sync()
    replicas.barrier()
    if use_cuda_events:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        sync()
        ms = e0.elapsed_time(e1)
    else:
        t0 = time.perf_counter()
        for _ in range(steps):
            fn()
        sync()
        ms = (time.perf_counter() - t0) * 1e3
    replicas.barrier()
    dev = "cuda" if use_cuda_events else "cpu"
    return replicas.max_over_ranks(ms, dev) / steps


def bus_bandwidth_gbs(nbytes: int, world: int, ms: float) -> float:
    """NCCL's convention for an all-reduce: 2 (n - 1) / n * bytes / time."""
    if world < 2 or ms <= 0 or nbytes == 0:
        return 0.0
    return 2.0 * (world - 1) / world * nbytes / (ms * 1e-3) / 1e9


def sweep(pl: dict, steps: int, warmup: int, device, make_layers=_GpuLayers, use_cuda_events=True, group=None) -> list:
    world = pl["world"]
    rows = []
    for p in P_SWEEP:
        L = make_layers(pl, p, device, group)
        if L.S % 8:
            continue
        for _ in range(max(warmup, 3)):
            L.step()
        L.sync()
        L.check()
        ms = _timed(L.step, steps, L.sync, use_cuda_events)
        row = {"p": p, "S": L.S, "ms_per_step": ms, "tokens_per_s": pl["tokens"] / (ms * 1e-3),
               "payload_bytes_16bit": L.payload_elems * 2, "payload_bytes_fp32": L.payload_elems * 4,
               "allreduces_per_step": 4 if pl["backward"] else 2,
               "payload_forward": L.payload_keys[0], "payload_backward": L.payload_keys[1]}
        if L.S > 0 and world > 1:
            # the exchange alone, on slab-sized buffers: the forward's 16-bit payload and the backward's fp32 carry
            for key, dt in (("16bit", torch.bfloat16), ("fp32", torch.float32)):
                buf = L.slab_like(dt)
                for _ in range(3):
                    tp.allreduce_slab(buf, group)
                ar = _timed(lambda: tp.allreduce_slab(buf, group), max(5, min(steps, 20)), L.sync, use_cuda_events)
                row[f"allreduce_ms_{key}"] = ar
                row[f"allreduce_busbw_gbs_{key}"] = bus_bandwidth_gbs(buf.numel() * buf.element_size(), world, ar)
        rows.append(row)
        del L
        if use_cuda_events:
            torch.cuda.empty_cache()
    # Appendix C with measured constants: the step without exchange and the exchange at p = 1
    base = next((r for r in rows if r["p"] == 1.0), None)
    none = next((r for r in rows if r["p"] == 0.0), None)
    if base and none:
        exch1 = 2 * base.get("allreduce_ms_" + base["payload_forward"], 0.0)
        if pl["backward"]:
            exch1 += 2 * base.get("allreduce_ms_" + base["payload_backward"], 0.0)
        for r in rows:
            r["speedup_vs_p1"] = base["ms_per_step"] / r["ms_per_step"]
            r["model_ms_per_step"] = none["ms_per_step"] + r["p"] * exch1
            r["model_speedup_vs_p1"] = (none["ms_per_step"] + exch1) / r["model_ms_per_step"]
    return rows


def run(args, make_layers=_GpuLayers, backend="nccl", out=sys.stdout):
    rank, local, world = replicas.rank_env()
    on_gpu = backend == "nccl"
    if on_gpu:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py --mode tp: no CUDA device (there is no CPU path)")
        torch.cuda.set_device(local)
        device = torch.device("cuda", local)
        # keep the communicator's own log lines, so that the number of ranks it was built for can be checked
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    else:
        device = torch.device("cpu")
    created = False
    if world > 1 and not dist.is_initialized():
        dist.init_process_group(backend, **({"device_id": device} if on_gpu else {}))
        created = True
    pl = plan(args.workload, world, getattr(args, "tokens", 0), getattr(args, "tp_exchange", "nccl"))
    rows = sweep(pl, args.steps, args.warmup, device, make_layers, on_gpu)
    if rank == 0:
        head = next((r for r in rows if r["p"] == 0.5), rows[0])
        line = {
            "metric": "CAAT block row-parallel layers tokens/s (real TP over GPUs, sync p)", "mode": "tp",
            "value": head["tokens_per_s"], "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": head["ms_per_step"], "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": pl["workload"], "tokens": pl["tokens"], "h": pl["h"], "ffn": pl["ffn"],
                       "tp_ranks": pl["t_total"], "ranks_per_gpu": pl["t_local"], "p": head["p"],
                       "parallelism": f"tp{pl['t_total']} over {world} GPUs",
                       "exchange": ("the library's exchange kernels over peer memory (reduce-scatter into per-source slots, fp32 "
                                    "sum in fixed order, all-gather by peer stores; forward GEMM pushes its shared tiles)"
                                    if pl["exchange"] == "push" else
                                    "all-reduce of the packed [T, S] slab between the library's two halves of a layer call") +
                                   f" (forward payload {head['payload_forward']}, backward payload {head['payload_backward']})"},
            "p_sweep": rows,
            "model": "Appendix C with measured constants: step(p) = step(p=0) + p * exchange(p=1), exchange = the step's "
                     "all-reduces timed alone",
        }
        out.write(json.dumps(line) + "\n")
        out.flush()
    if created:
        dist.barrier()
        dist.destroy_process_group()
    return rows
