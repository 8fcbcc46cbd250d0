#!/usr/bin/env python
"""Benchmark of the CAAT-Net row-parallel hot path on B200.

A step is one pass of the whole path over one batch of synthetic input: block forward
(attention-out layer, then MLP-down layer: GEMM + partial channel-reduce + residual +
norm) followed, for training workloads, by the block backward.  The t tensor-parallel
ranks are simulated as a batch dimension on one GPU.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  With N > 1 (launched by torch.distributed.run) every GPU
runs an independent replica of the workload (the path has no cross-GPU exchange step):
weak scaling, no data-path collective; time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2506_19645_b200 import replicas, synthetic  # noqa: E402

DEFAULT_WORKLOAD = "block_130m"
METRIC = "CAAT block tokens/s (sim. TP=t, sync p) on 1 B200"


def metric_name(w):
    return METRIC.replace("block", "MLP (column- + row-parallel half)") if w.kind == "mlp" else METRIC
# lightest first: the 7B workloads run into the power cap and leave the GPU's clocks low for what follows
SWEEP = ["mlp_130m", "block_1p1b_p100", "block_1p1b_p075", "block_1p1b_p050", "block_1p1b_p025", "mlp_1p1b_p050",
         "block_7b", "mlp_7b"]


# --------------------------------------------------------------------------- peaks
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured (MEASURED_PEAKS.json; sustained bf16 figure: kernels timed inside a long step)"}
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1400.0, "source": "fallback (earlier measurement on this pool)"}


def recorded_traffic(kernel: str, workload: str):
    """DRAM bytes per launch from a committed ncu capture (profiles/traffic.json), else None."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            return json.load(f).get(workload, {}).get(kernel)
    except Exception:
        return None


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons while the timed region runs (read-only NVML)."""

    def __init__(self, index: int, period_s: float = 0.005):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                 "hw_power_brake_slowdown": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self) -> dict:
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------- algorithmic work
def layer_work(w, k_r, backward, compact=False):
    """Algorithmic flops and bytes of ONE layer per kernel kind (inputs read once, outputs
    written once, given the kernel's interface; e = 2 bytes).  compact: the residual stream and
    its gradient are stored shared-once + private-per-rank, like the scratch."""
    t, T, h, S, e = w.t, w.tokens, w.h, w.S, 2
    K = k_r * t
    zsz = (T * S + t * T * (h - S)) * e            # split scratch: shared once, private per rank
    full = t * T * h * e
    stream = zsz if compact else full              # one tensor of the residual stream
    out = {
        "tc_gemm_forward": {"flops": 2.0 * T * K * h, "bytes": (T * K + K * h) * e + zsz},
        "rows_forward": {"flops": 0.0, "bytes": zsz + 2 * stream + full + t * T * 4},
    }
    if backward:
        # reads dX, Hn, dHn; writes dR and the reduced shared gradient gs [T, S] (compact: gs is dRs, part of dR).
        # The GEMMs read the private gradient from dR itself: no scaled copy is written.
        bwd_out = stream if compact else stream + T * S * e
        out["rows_backward"] = {"flops": 0.0, "bytes": full + 2 * stream + bwd_out + t * T * 4}
        out["tc_gemm_dgrad"] = {"flops": 2.0 * T * K * h, "bytes": zsz + K * h * e + T * K * e}
        out["tc_gemm_wgrad"] = {"flops": 2.0 * T * K * h, "bytes": zsz + T * K * e + K * h * 4}
    return out


def colpar_work(w):
    """Algorithmic work of the column-parallel MLP half (gate|up GEMM per rank + SwiGLU), e = 2 bytes."""
    t, T, h, F, e = w.t, w.tokens, w.h, w.kr_mlp, 2
    fl = 2.0 * t * T * h * 2 * F
    out = {"tc_gemm_forward": {"flops": fl, "bytes": (t * T * h + t * 2 * F * h + t * T * 2 * F) * e},
           "activation": {"flops": 0.0, "bytes": t * T * 3 * F * e}}
    if w.backward:
        out["activation"]["bytes"] += t * T * 5 * F * e
        out["tc_gemm_dgrad"] = {"flops": fl, "bytes": (t * T * 2 * F + t * 2 * F * h + t * T * h) * e}
        out["tc_gemm_wgrad"] = {"flops": fl, "bytes": (t * T * 2 * F + t * T * h) * e + t * 2 * F * h * 4}
    return out


def step_work(w, compact=False):
    tot = {}
    parts = [layer_work(w, k_r, w.backward, compact) for k_r in ((w.kr_mlp,) if w.kind == "mlp" else (w.kr_attn, w.kr_mlp))]
    if w.kind == "mlp":
        parts.append(colpar_work(w))
    for part in parts:
        for kind, v in part.items():
            a = tot.setdefault(kind, {"flops": 0.0, "bytes": 0.0})
            a["flops"] += v["flops"]
            a["bytes"] += v["bytes"]
    return tot


def paper_level_work(w, compact=False):
    """Whole-path algorithmic work per step (no scratch traffic): the roofline of the path."""
    t, T, h, e = w.t, w.tokens, w.h, 2
    full = t * T * h
    stream = T * w.S + t * T * (h - w.S) if compact else full
    fl = by = 0.0
    if w.kind == "mlp":   # column-parallel half: X, A in; pre kept for the backward; dX, dA out
        F = w.kr_mlp
        fl += 2.0 * t * T * h * 2 * F * (3 if w.backward else 1)
        by += e * (full + t * 2 * F * h + t * T * 2 * F) + (e * (t * T * 2 * F + full) + 4 * t * 2 * F * h if w.backward else 0)
    for k_r in ((w.kr_mlp,) if w.kind == "mlp" else (w.kr_attn, w.kr_mlp)):
        K = k_r * t
        fl += 2.0 * T * K * h
        by += e * (T * K + K * h + 2 * stream + full)
        if w.backward:
            fl += 4.0 * T * K * h
            by += e * (full + 3 * stream + 2 * T * K + K * h) + 4 * K * h
    return fl, by


def r_w_compact_ok(w):
    """The compact-layout entry points need a partition on a 16-byte boundary."""
    return w.S % 8 == 0


# --------------------------------------------------------------------------- the CUDA arm
class BlockRunner:
    def __init__(self, w, device, compact=False):
        from paper_2506_19645_b200 import caat
        self.caat, self.w, self.dev, self.compact = caat, w, device, compact
        self.ctx = caat.Context(w.h, w.ffn, w.t, w.p, w.dtype)
        self.inp = synthetic.block_inputs(w, device=device)
        t, T, h = w.t, w.tokens, w.h
        td = self.ctx.torch_dtype
        mk = lambda *s, dt=td: torch.empty(*s, dtype=dt, device=device)
        f32 = torch.float32
        if compact:
            # same synthetic block, with the (tied) shared channels of the stream kept once
            S, i = w.S, self.inp
            for name in ("R0", "dHn2"):
                if name in i:
                    x = i.pop(name)
                    i[name + "s"], i[name + "p"] = x[0, :, :S].contiguous(), x[:, :, S:].contiguous()
            sh, pr = (T, S), (t, T, h - S)
            self.out = {"Hn1s": mk(*sh), "Hn1p": mk(*pr), "X1": mk(t, T, h), "rstd1": mk(t, T, dt=f32),
                        "Hn2s": mk(*sh), "Hn2p": mk(*pr), "X2": mk(t, T, h), "rstd2": mk(t, T, dt=f32)}
            if w.backward:
                self.out.update({"dY_attn": mk(t, T, w.kr_attn), "dW_o": mk(t, h, w.kr_attn, dt=f32),
                                 "dY_mlp": mk(t, T, w.kr_mlp), "dW_down": mk(t, h, w.kr_mlp, dt=f32),
                                 "dR0s": mk(*sh), "dR0p": mk(*pr), "dHn1s": mk(*sh), "dHn1p": mk(*pr),
                                 "dgamma1": mk(h, dt=f32), "dgamma2": mk(h, dt=f32)})
            self.ws = self.ctx.alloc_workspace(self.ctx.block_workspace_bytes(T, w.backward), device=device)
            return
        self.out = {"Hn1": mk(t, T, h), "X1": mk(t, T, h), "rstd1": mk(t, T, dt=f32),
                    "Hn2": mk(t, T, h), "X2": mk(t, T, h), "rstd2": mk(t, T, dt=f32)}
        if w.backward:
            self.out.update({"dY_attn": mk(t, T, w.kr_attn), "dW_o": mk(t, h, w.kr_attn, dt=f32),
                             "dY_mlp": mk(t, T, w.kr_mlp), "dW_down": mk(t, h, w.kr_mlp, dt=f32),
                             "dR0": mk(t, T, h), "dHn1": mk(t, T, h), "dgamma1": mk(h, dt=f32), "dgamma2": mk(h, dt=f32)})
        self.ws = self.ctx.alloc_workspace(self.ctx.block_workspace_bytes(T, w.backward), device=device)

    def step(self):
        i, o, T = self.inp, self.out, self.w.tokens
        if self.compact:
            self.ctx.block_forward_compact(T, i["Y_attn"], i["W_o"], i["Y_mlp"], i["W_down"], i["R0s"], i["R0p"],
                                           i["gamma1"], None, i["gamma2"], None, o["Hn1s"], o["Hn1p"], o["X1"],
                                           o["rstd1"], None, o["Hn2s"], o["Hn2p"], o["X2"], o["rstd2"], None, self.ws)
            if self.w.backward:
                self.ctx.block_backward_compact(T, i["dX1"], i["dX2"], i["dHn2s"], i["dHn2p"], i["Y_attn"], i["W_o"],
                                                i["Y_mlp"], i["W_down"], o["Hn1s"], o["Hn1p"], o["rstd1"], None,
                                                o["Hn2s"], o["Hn2p"], o["rstd2"], None, i["gamma1"], i["gamma2"],
                                                o["dY_attn"], o["dW_o"], o["dY_mlp"], o["dW_down"], o["dR0s"],
                                                o["dR0p"], o["dHn1s"], o["dHn1p"], o["dgamma1"], None, o["dgamma2"],
                                                None, self.ws)
            return
        self.ctx.block_forward(T, i["Y_attn"], i["W_o"], i["Y_mlp"], i["W_down"], i["R0"], i["gamma1"], None,
                               i["gamma2"], None, o["Hn1"], o["X1"], o["rstd1"], None, o["Hn2"], o["X2"], o["rstd2"],
                               None, self.ws)
        if self.w.backward:
            self.ctx.block_backward(T, i["dX1"], i["dX2"], i["dHn2"], i["Y_attn"], i["W_o"], i["Y_mlp"], i["W_down"],
                                    o["Hn1"], o["rstd1"], None, o["Hn2"], o["rstd2"], None, i["gamma1"], i["gamma2"],
                                    o["dY_attn"], o["dW_o"], o["dY_mlp"], o["dW_down"], o["dR0"], o["dHn1"],
                                    o["dgamma1"], None, o["dgamma2"], None, self.ws)

    def touched_bytes(self):
        n = sum(v.numel() * v.element_size() for v in self.inp.values())
        return n + sum(v.numel() * v.element_size() for v in self.out.values())


class MlpRunner:
    """The whole tensor-parallel MLP: column-parallel gate|up + SwiGLU, then the MLP-down layer with partial
    channel-reduce (and the gradient of both), as two library calls per direction."""

    def __init__(self, w, device, compact=False):
        from paper_2506_19645_b200 import caat
        assert not compact
        self.caat, self.w, self.dev, self.compact = caat, w, device, False
        self.ctx = caat.Context(w.h, w.ffn, w.t, w.p, w.dtype)
        self.inp = synthetic.mlp_inputs(w, device=device)
        t, T, h, F = w.t, w.tokens, w.h, w.kr_mlp
        td, f32 = self.ctx.torch_dtype, torch.float32
        mk = lambda *s, dt=td: torch.empty(*s, dtype=dt, device=device)
        self.out = {"pre": mk(t, T, 2 * F), "Y": mk(t, T, F), "Hn": mk(t, T, h), "Xout": mk(t, T, h), "rstd": mk(t, T, dt=f32)}
        if w.backward:
            self.out.update({"dY": mk(t, T, F), "dB": mk(t, h, F, dt=f32), "dR": mk(t, T, h), "dgamma": mk(h, dt=f32),
                             "dX": mk(t, T, h), "dA": mk(t, 2 * F, h, dt=f32)})
        nbytes = max(self.ctx.workspace_bytes(caat.CAAT_MLP_DOWN, T, w.backward),
                     self.ctx.colpar_workspace_bytes(caat.CAAT_ACT_SWIGLU, 2 * F, T))
        self.ws = self.ctx.alloc_workspace(nbytes, device=device)

    def step(self):
        c, i, o, T, F = self.caat, self.inp, self.out, self.w.tokens, self.w.kr_mlp
        self.ctx.colpar_forward(c.CAAT_ACT_SWIGLU, 2 * F, T, i["X"], i["A"], o["pre"], o["Y"])
        self.ctx.rowpar_forward(c.CAAT_MLP_DOWN, T, o["Y"], i["B"], i["R"], i["gamma"], None, o["Hn"], o["Xout"], o["rstd"],
                                None, self.ws)
        if self.w.backward:
            self.ctx.rowpar_backward(c.CAAT_MLP_DOWN, T, i["dXout"], i["dHn"], o["Y"], i["B"], o["Hn"], o["rstd"], None,
                                     i["gamma"], o["dY"], o["dB"], o["dR"], o["dgamma"], None, self.ws)
            self.ctx.colpar_backward(c.CAAT_ACT_SWIGLU, 2 * F, T, o["dY"], i["X"], i["A"], o["pre"], o["dX"], o["dA"], self.ws)

    def touched_bytes(self):
        n = sum(v.numel() * v.element_size() for v in self.inp.values())
        return n + sum(v.numel() * v.element_size() for v in self.out.values())


# 8-GPU all-reduce bus bandwidth at 1 GiB measured on this pool's NVSwitch machines (nominal NVLink 5:
# 900 GB/s per direction per GPU); NCCL's convention: time = 2 (n - 1) / n * bytes / bus bandwidth.
NVLINK_ALLREDUCE_BUSBW_GBS = 725.0


def tp_projection(dev, name="block_7b", steps=20):
    """What the paper's claim looks like on this hardware: ONE GPU's share of a real t-GPU run of the block (one
    rank per GPU), timed with the library's two halves of every layer call and no collective, next to the time
    the four all-reduces of a step (Appendix C) would take for the analytic payload at the bandwidth above, not
    overlapped.  A projection, labelled as such: nothing here ran on more than one GPU."""
    from paper_2506_19645_b200 import caat
    w0 = synthetic.WORKLOADS[name]
    G, T, h = w0.t, w0.tokens, w0.h
    rows = []
    for p in (1.0, 0.75, 0.5, 0.25, 0.0):
        ctx = caat.Context(h, w0.ffn, 1, p, "bf16")
        ctx.set_option(caat.CAAT_OPT_TP_GROUPS, G)
        S = ctx.shared_channels
        if S % 8:
            continue
        layers = []
        for layer in (caat.CAAT_ATTN_OUT, caat.CAAT_MLP_DOWN):
            k = ctx.k_r(layer)
            d = synthetic.layer_inputs(1, T, h, k, "bf16", seed=layer, S=S, backward=True, device=dev)
            mk = lambda *sh, dt=torch.bfloat16: torch.empty(*sh, dtype=dt, device=dev)
            o = {"Hn": mk(1, T, h), "X": mk(1, T, h), "rstd": mk(1, T, dt=torch.float32), "dY": mk(1, T, k),
                 "dW": mk(1, h, k, dt=torch.float32), "dR": mk(1, T, h), "dg": mk(h, dt=torch.float32)}
            layers.append((layer, d, o))
        ws = ctx.alloc_workspace(ctx.block_workspace_bytes(T, True), device=dev)

        def step():
            for layer, d, o in layers:
                ctx.tp_forward_local(layer, T, d["Y"], d["W"], ws)
                ctx.tp_forward_finish(layer, T, d["R"], d["gamma"], None, o["Hn"], o["X"], o["rstd"], None, ws)
            for layer, d, o in reversed(layers):
                ctx.tp_backward_local(layer, T, d["dX"], d["dHn"], d["W"], o["Hn"], o["rstd"], None, d["gamma"], o["dR"],
                                      o["dg"], None, ws)
                ctx.tp_backward_finish(layer, T, d["Y"], d["W"], o["dR"], o["dY"], o["dW"], ws)

        for _ in range(3):
            step()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        compute_ms = e0.elapsed_time(e1) / steps
        ring = 2.0 * (G - 1) / G
        ar = lambda nbytes: ring * nbytes / (NVLINK_ALLREDUCE_BUSBW_GBS * 1e9) * 1e3
        fwd_ms = 2 * ar(T * S * 2)                       # two reduces per block forward, 16-bit payload
        bwd16_ms, bwd32_ms = 2 * ar(T * S * 2), 2 * ar(T * S * 4)
        rows.append({"p": p, "S": S, "compute_ms_per_gpu": compute_ms, "allreduce_ms_forward": fwd_ms,
                     "allreduce_ms_backward_16bit": bwd16_ms, "allreduce_ms_backward_fp32": bwd32_ms,
                     "step_ms_no_overlap": compute_ms + fwd_ms + bwd32_ms})
        del layers, ws
        torch.cuda.empty_cache()
    if rows:
        base = rows[0]["step_ms_no_overlap"]
        for r in rows:
            r["speedup_vs_p1"] = base / r["step_ms_no_overlap"]
    return {"workload": name, "gpus": G, "ranks_per_gpu": 1, "tokens": T,
            "allreduce_bus_bandwidth_gbs": NVLINK_ALLREDUCE_BUSBW_GBS,
            "note": "projection: measured one-GPU compute (two-halves calls, no collective) + analytic all-reduce "
                    "time (2 forward 16-bit + 2 backward fp32 reduces per block, ring factor 2(n-1)/n), no overlap; "
                    "not a multi-GPU measurement",
            "rows": rows}


def make_runner(w, device, compact=False):
    return MlpRunner(w, device, compact) if w.kind == "mlp" else BlockRunner(w, device, compact)


def capture_step(runner):
    """One step captured into a CUDA graph (launch-bound workloads: a decode step is tens of
    microseconds).  Returns (graph, kernels per step) or (None, 0) when capture is not possible."""
    from paper_2506_19645_b200 import caat
    try:
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            runner.step()                      # warm the side stream
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        l0 = caat.kernel_launches()
        with torch.cuda.graph(g, stream=side):
            runner.step()
        per_step = caat.kernel_launches() - l0
        g.replay()
        torch.cuda.synchronize()
        return g, int(per_step)
    except Exception as ex:  # noqa: BLE001
        sys.stderr.write(f"bench: CUDA graph capture failed ({ex}); timing eager launches\n")
        return None, 0


L2_BYTES = 126e6


def buffer_sets_needed(touched_bytes):
    """Steps that touch less than about twice the L2 would find their inputs cached from the step before:
    such workloads rotate over several buffer sets so that more than two L2s of other data pass between
    two uses of a set."""
    if touched_bytes >= 2 * L2_BYTES:
        return 1
    return min(16, int(2 * L2_BYTES // max(touched_bytes, 1)) + 2)


def time_steps(runner, steps, dist_on, graph=None):
    """Device time of exactly `steps` steps (ms), CUDA events on the launching stream.  `runner` and
    `graph` may be lists (buffer sets rotated step by step)."""
    runners = runner if isinstance(runner, list) else [runner]
    graphs = graph if isinstance(graph, list) else ([graph] if graph is not None else None)
    torch.cuda.synchronize()
    if dist_on:
        torch.distributed.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for q in range(steps):
        if graphs is not None:
            graphs[q % len(graphs)].replay()
        else:
            runners[q % len(runners)].step()
    e1.record()
    torch.cuda.synchronize()
    if dist_on:
        torch.distributed.barrier()
    return e0.elapsed_time(e1)


def e2e_leg(runner, steps):
    """Same step through the public API with HOST buffers: every step copies its inputs from pinned
    host memory and reads its results back to the host, all inside the timed region.  The three
    phases run on three streams over two sets of device buffers, so the copy of step s+1, the
    kernels of step s and the read-back of step s-1 overlap (PCIe moves both ways at once)."""
    runners = [runner, make_runner(runner.w, runner.dev, runner.compact)]
    inp_host = {k: v.cpu().pin_memory() for k, v in runner.inp.items()}
    out_host = [{k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in runner.out.items()} for _ in range(2)]
    h2d = sum(v.numel() * v.element_size() for v in inp_host.values())
    d2h = sum(v.numel() * v.element_size() for v in out_host[0].values())
    s_in, s_run, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [None, None]    # inputs of the buffer set are on the device
    ev_run = [None, None]   # its step has run
    ev_out = [None, None]   # its results are on the host

    def one(step):
        b = step & 1
        r = runners[b]
        with torch.cuda.stream(s_in):
            if ev_run[b] is not None:
                s_in.wait_event(ev_run[b])          # the previous step on this set no longer reads its inputs
            for k, v in inp_host.items():
                r.inp[k].copy_(v, non_blocking=True)
            ev_in[b] = s_in.record_event()
        with torch.cuda.stream(s_run):
            s_run.wait_event(ev_in[b])
            if ev_out[b] is not None:
                s_run.wait_event(ev_out[b])         # its previous results have left the device
            r.step()
            ev_run[b] = s_run.record_event()
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_run[b])
            for k, v in r.out.items():
                out_host[b][k].copy_(v, non_blocking=True)
            ev_out[b] = s_out.record_event()

    for q in range(2):
        one(q)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(s_in)
    for q in range(steps):
        one(q)
    s_out.wait_stream(s_in)
    s_out.wait_stream(s_run)
    e1.record(s_out)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    del runners[1]
    return ms, h2d, d2h


def oracle_sample_run(w, sample_tokens):
    """One block forward(+backward) of the fp64 oracle on `sample_tokens` tokens of the workload."""
    from oracle import caat_oracle as O
    ws = w.with_tokens(sample_tokens)
    S, alpha = ws.S, math.sqrt(ws.t)
    if w.kind == "mlp":
        d = {k: v.to(torch.float64).numpy() for k, v in synthetic.mlp_inputs(ws, device="cpu").items()}
        t0 = time.perf_counter()
        f = O.mlp_forward(d["X"], d["A"], d["B"], d["R"], d["gamma"], S=S, alpha=alpha)
        if w.backward:
            O.mlp_backward(d["dXout"], d["dHn"], d["X"], d["A"], d["B"], f["pre"], f["Y"], f["Hn"], f["rstd"], None,
                           d["gamma"], S=S, alpha=alpha)
        return time.perf_counter() - t0
    d = {k: v.to(torch.float64).numpy() for k, v in synthetic.block_inputs(ws, device="cpu").items()}
    t0 = time.perf_counter()
    f = O.block_forward(d["Y_attn"], d["W_o"], d["Y_mlp"], d["W_down"], d["R0"], d["gamma1"], d["gamma2"], S=S, alpha=alpha)
    if w.backward:
        O.block_backward(d["dX1"], d["dX2"], d["dHn2"], d["Y_attn"], d["W_o"], d["Y_mlp"], d["W_down"], f["Hn1"],
                         f["rstd1"], None, f["Hn2"], f["rstd2"], None, d["gamma1"], d["gamma2"], S=S, alpha=alpha)
    return time.perf_counter() - t0


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return len(os.sched_getaffinity(0))


def cpu_baseline(w, target_s=12.0):
    probe = min(256, w.tokens)
    tp = oracle_sample_run(w, probe)
    tp = min(tp, oracle_sample_run(w, probe))
    n = int(target_s / max(tp / probe, 1e-9))
    n = max(probe, min(w.tokens, n // 256 * 256 if n >= 256 else probe))
    ts = oracle_sample_run(w, n)
    return {"value": n / ts, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
            "sample": f"fp64 numpy oracle, block forward{'+backward' if w.backward else ''} on {n} of {w.tokens} tokens "
                      f"of {w.name} (all {w.t} ranks), {ts:.2f} s; host has {len(os.sched_getaffinity(0))} usable cores"}


def run_cuda(args):
    from paper_2506_19645_b200 import caat
    rank, local, world = replicas.rank_env()
    dist_on = world > 1
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if dist_on:
        torch.distributed.init_process_group("nccl", device_id=dev)
    w = synthetic.WORKLOADS[args.workload]
    if args.tokens > 0:
        w = w.with_tokens(args.tokens)
    compact = args.layout == "compact"
    runner = make_runner(w, dev, compact)
    warm = max(args.warmup, 3)
    for _ in range(warm):
        runner.step()
    torch.cuda.synchronize()
    assert runner.ctx.last_device_status() == caat.CAAT_OK

    # small working sets (decode: the weights are about one L2) rotate over several buffer sets
    nsets = buffer_sets_needed(runner.touched_bytes())
    rset = [runner] + [make_runner(w, dev, compact) for _ in range(nsets - 1)]
    for r in rset[1:]:
        r.step()
    torch.cuda.synchronize()
    # launch-bound steps (decode: tens of microseconds) are replayed from a CUDA graph
    graph, per_step = (None, 0)
    probe = time_steps(rset, 5, False) / 5
    if probe < 0.25 and not args.no_graph:
        caps = [capture_step(r) for r in rset]
        if all(g is not None for g, _ in caps):
            graph, per_step = [g for g, _ in caps], caps[0][1]
    sampler = ClockSampler(local)
    sampler.start()
    l0 = caat.kernel_launches()
    ms = time_steps(rset, args.steps, dist_on, graph)
    launches = per_step * args.steps if graph is not None else caat.kernel_launches() - l0
    # second pass of the same K steps with CUDA events around every kernel (per-kernel device times)
    caat.profile_begin(max(1024, launches + 64))
    ms_prof = time_steps(rset, args.steps, dist_on)
    prof = caat.profile_end()
    # small working sets: the same steps on ONE buffer set, i.e. with whatever fits staying in L2 (reported
    # separately; the headline figure is the rotated one)
    ms_warm_l2 = None
    if nsets > 1:
        ms_warm_l2 = time_steps(rset[:1], args.steps, False, graph[:1] if graph is not None else None) / args.steps
    del rset[1:]
    clocks = sampler.stop()
    ms = replicas.max_over_ranks(ms, dev)

    ms_step = ms / args.steps
    value = replicas.whole_job_rate(w.tokens, args.steps, world, ms)

    # end-to-end leg: every rank runs it at the same time (each GPU has its own host link); the job's figure is
    # all replicas' tokens over the slowest rank's time
    e2e = None
    try:
        if args.no_e2e:
            raise RuntimeError("skipped (--no-e2e)")
        if dist_on:
            torch.distributed.barrier()
        ems, h2d, d2h = e2e_leg(runner, max(4, min(args.steps, 8)))
        ems = replicas.max_over_ranks(ems, dev)
        e2e = {"value": world * w.tokens / (ems * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d * world,
               "d2h_bytes_per_step": d2h * world, "ms_per_step": ems,
               "overlap": "copy-in, kernels and read-back of consecutive steps on three streams, two buffer sets"}
    except Exception as ex:  # pinned-memory exhaustion on a small host
        if dist_on:
            replicas.max_over_ranks(0.0, dev)     # keep the ranks' collectives matched
        e2e = {"value": None, "unit": "tokens/s", "error": str(ex)[:200]}

    result = None
    if rank == 0:
        peaks = measured_peaks()
        work = step_work(w, compact)
        kernels = {}
        for kind, (kms, n) in prof.items():
            per_step_ms = kms / args.steps
            wk = work.get(kind)
            ent = {"ms_per_step": per_step_ms, "launches_per_step": n / args.steps, "share": kms / sum(v[0] for v in prof.values())}
            if wk:
                gbs = wk["bytes"] / (per_step_ms * 1e-3) / 1e9
                tfs = wk["flops"] / (per_step_ms * 1e-3) / 1e12
                t_hbm, t_tc = wk["bytes"] / (peaks["hbm_gbs"] * 1e9), wk["flops"] / (peaks["bf16_tflops"] * 1e12)
                if t_tc > t_hbm:
                    ent.update({"bound": "tensor", "achieved": tfs, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                "frac": tfs / peaks["bf16_tflops"]})
                else:
                    ent.update({"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                "frac": gbs / peaks["hbm_gbs"]})
                ent["gbs"], ent["tflops"] = gbs, tfs
            kernels[kind] = ent
        top = max((k for k in kernels if "frac" in kernels[k]), key=lambda k: kernels[k]["ms_per_step"])
        roof = {k: kernels[top][k] for k in ("bound", "achieved", "peak", "unit", "frac")}
        roof.update({"kernel": top, "traffic": recorded_traffic(top, w.name + ("@compact" if compact else "")), "peak_source": peaks["source"],
                     "timed": f"second pass of {args.steps} steps with CUDA events around every kernel launch "
                              f"({ms_prof / args.steps:.4f} ms/step with events)"})
        fl, by = paper_level_work(w, compact)
        t_roof = max(fl / (peaks["bf16_tflops"] * 1e12), by / (peaks["hbm_gbs"] * 1e9))
        ar = runner.ctx.allreduce_bytes(w.tokens, 2)
        result = {
            "metric": metric_name(w), "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": warm,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": w.dtype, "data": "synthetic",
            "config": {"workload": w.name, "t": w.t, "tokens": w.tokens, "h": w.h, "ffn": w.ffn, "p": w.p,
                       "S": w.S, "passes": "forward+backward" if w.backward else "forward",
                       "private_scale": "sqrt(t)", "norm": "rmsnorm", "parallelism": f"replicas x{world}",
                       "residual_layout": "compact (shared channels of the stream stored once)" if compact else "per rank [t,T,h]",
                       "launch": "cuda graph replay" if graph is not None else "eager",
                       "l2": (f"inputs+outputs touched per step {runner.touched_bytes() / 1e6:.0f} MB > 126 MB L2" if nsets == 1 else
                              f"{nsets} buffer sets rotated step by step: {runner.touched_bytes() / 1e6:.0f} MB touched per step, "
                              f"{(nsets - 1) * runner.touched_bytes() / 1e6:.0f} MB of other sets between two uses of a set (L2 126 MB)")},
            "clocks": clocks, "gpu_launches": int(launches), "e2e": e2e, "roofline": roof, "kernels": kernels,
            "path_roofline": {"flops_per_step": fl, "bytes_per_step": by, "roofline_ms": t_roof * 1e3,
                              "frac": t_roof * 1e3 / ms_step},
            "collective_bytes_analytic": {"per_reduce": ar, "reduces_per_step": 4 if w.backward else 2},
        }
        if ms_warm_l2 is not None:
            result["warm_l2"] = {"ms_per_step": ms_warm_l2, "tokens_per_s": w.tokens / (ms_warm_l2 * 1e-3),
                                 "note": "same steps on a single buffer set (operands that fit stay in the 126 MB L2); "
                                         "not the headline figure"}
    del runner
    torch.cuda.empty_cache()

    if rank == 0 and not args.no_sweep and world == 1:
        sweep = []
        for name in SWEEP:
            if name == w.name:
                continue
            try:
                r = make_runner(synthetic.WORKLOADS[name], dev)
                for _ in range(5):
                    r.step()
                k = max(3, min(args.steps, 30))
                sms = time_steps(r, k, False) / k
                fl, by = paper_level_work(r.w)
                peaks = measured_peaks()
                t_roof = max(fl / (peaks["bf16_tflops"] * 1e12), by / (peaks["hbm_gbs"] * 1e9)) * 1e3
                sweep.append({"workload": name, "p": r.w.p, "ms_per_step": sms, "tokens_per_s": r.w.tokens / (sms * 1e-3),
                              "path_roofline_frac": t_roof / sms,
                              "allreduce_payload_bytes": r.ctx.allreduce_bytes(r.w.tokens, 2)["payload_per_rank"]})
                del r
                torch.cuda.empty_cache()
                if r_w_compact_ok(synthetic.WORKLOADS[name]) and synthetic.WORKLOADS[name].kind == "block":
                    # the same block on the compact residual layout (shared channels of the stream stored once)
                    r = BlockRunner(synthetic.WORKLOADS[name], dev, True)
                    for _ in range(3):
                        r.step()
                    cms = time_steps(r, k, False) / k
                    sweep[-1]["compact_layout_ms_per_step"] = cms
                    sweep[-1]["compact_layout_tokens_per_s"] = r.w.tokens / (cms * 1e-3)
                    del r
                    torch.cuda.empty_cache()
            except Exception as ex:
                sweep.append({"workload": name, "error": str(ex)[:200]})
        result["sweep"] = sweep
        try:
            result["tp_projection"] = tp_projection(dev)
        except Exception as ex:  # noqa: BLE001
            result["tp_projection"] = {"error": str(ex)[:200]}
    if rank == 0:
        if not args.no_cpu and world == 1:
            result["cpu_baseline"] = cpu_baseline(w)
        else:
            result["cpu_baseline"] = None
        print(json.dumps(result), flush=True)
    if dist_on:
        torch.distributed.barrier()
        torch.distributed.destroy_process_group()


# --------------------------------------------------------------------------- the reference arm (oracle on host cores)
def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    w = synthetic.WORKLOADS[args.workload]
    probe = min(256, w.tokens)
    tp = min(oracle_sample_run(w, probe), oracle_sample_run(w, probe))
    budget = 150.0 / max(1, args.steps + args.warmup)            # seconds per step so the run ends within minutes
    n = int(min(budget, 1.0) / max(tp / probe, 1e-9))
    n = max(probe, min(w.tokens, n // 256 * 256 if n >= 256 else probe))
    for _ in range(args.warmup):
        oracle_sample_run(w, n)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_sample_run(w, n)
    dt = time.perf_counter() - t0
    value = n * args.steps / dt
    sample = (f"fp64 numpy oracle, block forward{'+backward' if w.backward else ''}, each step a sample of {n} of "
              f"{w.tokens} tokens of {w.name}; host has {len(os.sched_getaffinity(0))} usable cores")
    print(json.dumps({
        "impl": "reference", "metric": metric_name(w), "value": value, "unit": "tokens/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "t": w.t, "tokens": w.tokens, "h": w.h, "ffn": w.ffn, "p": w.p, "S": w.S,
                   "passes": "forward+backward" if w.backward else "forward", "sample_tokens": n},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synthetic.WORKLOADS))
    ap.add_argument("--no-sweep", action="store_true", help="skip the other workloads' tokens/s")
    ap.add_argument("--no-cpu", action="store_true", help="skip the timed CPU oracle baseline")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-graph", action="store_true", help="never replay launch-bound steps from a CUDA graph")
    ap.add_argument("--layout", default="per_rank", choices=["per_rank", "compact"],
                    help="residual-stream layout: per rank [t,T,h] (the benchmark's configuration) or compact")
    ap.add_argument("--tokens", type=int, default=0, help="override the workload's token count (profiling on a small case)")
    args = ap.parse_args()
    if args.steps < 1:
        raise SystemExit("--steps must be >= 1")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
