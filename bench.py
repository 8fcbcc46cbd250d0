#!/usr/bin/env python
"""Benchmark of the CAAT-Net row-parallel hot path on B200.

A step is one pass of the whole path over one batch of synthetic input: block forward
(attention-out layer, then MLP-down layer: GEMM + partial channel-reduce + residual +
norm) followed, for training workloads, by the block backward.  The t tensor-parallel
ranks are simulated as a batch dimension on one GPU.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]
  python -m torch.distributed.run ... bench.py --gpus N --mode tp      (real tensor parallelism, p sweep)

Prints ONE JSON line (rank 0).  With N > 1 (launched by torch.distributed.run) every GPU
runs an independent replica of the workload (the path as benchmarked has no cross-GPU
exchange step): weak scaling, no data-path collective; time is the max over ranks.
``--mode tp`` instead splits the tensor-parallel ranks over the GPUs and exchanges the
shared-channel slab with an all-reduce (the paper's partial channel-reduce).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2506_19645_b200 import replicas, synthetic  # noqa: E402

# The metric is quoted on no single configuration: the headline line is the largest one that fits a GPU.
DEFAULT_WORKLOAD = "block_7b"
METRIC = "CAAT block tokens/s (sim. TP=t, sync p) on 1 B200"


def metric_name(w):
    if w.kind == "mlp":
        return METRIC.replace("block", "MLP (column- + row-parallel half)")
    if w.kind == "layer":
        return METRIC.replace("block", "row-parallel layer")
    return METRIC


# every configuration the metric is defined on, lightest first: the 7B workloads run into the power cap and
# leave the GPU's clocks low for what follows
SWEEP = (["layer_fp32_small"] + [f"decode_7b_T{T}_p{p}" for T in (1, 8, 64) for p in ("100", "050")] +
         ["block_130m", "mlp_130m", "block_1p1b_p100", "block_1p1b_p075", "block_1p1b_p050", "block_1p1b_p025",
          "mlp_1p1b_p050", "block_7b", "mlp_7b"])


# --------------------------------------------------------------------------- peaks
def measured_peaks():
    """Roofline denominators: the copy bandwidth and the two cuBLAS bf16 figures measured on this machine (a burst
    figure for a kernel timed alone, a sustained one for kernels timed inside a long, power-capped step)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops_burst": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "of measured (MEASURED_PEAKS.json)"}
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_tflops_burst": 1590.0, "bf16_tflops_sustained": 1400.0,
                "source": "of fallback (earlier measurement on this pool)"}


def recorded_traffic(kernel: str, workload: str):
    """DRAM bytes per step of one kernel kind from a committed ncu capture (profiles/traffic.json), else None."""
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
        return {"sm_mhz": statistics.median(self.samples), "sm_min_mhz": min(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------- algorithmic work
def esize(w):
    return 4 if w.dtype == "f32" else 2


def layer_work(w, S, k_r, compact=False):
    """Work of ONE layer per kernel kind.  "bytes" is the ALGORITHMIC traffic of the step the kernel
    performs: tensors of the method read once and written once - no scratch (the GEMM's partial sums, the
    reduced gradient slab) and no saved statistics.  "bytes_interface" adds what the kernel's own interface
    makes it move on top (scratch in or out, rstd), for reference only.  compact: the residual stream and its
    gradient are stored shared-once + private-per-rank."""
    t, T, h, e = w.t, w.tokens, w.h, esize(w)
    K = k_r * t
    zsz = (T * S + t * T * (h - S)) * e            # split scratch: shared once, private per rank
    full = t * T * h * e
    stream = zsz if compact else full              # one tensor of the residual stream
    fl = 2.0 * T * K * h
    out = {
        "tc_gemm_forward": {"flops": fl, "bytes": (T * K + K * h) * e, "bytes_interface": (T * K + K * h) * e + zsz},
        # R in, Hn and X out
        "rows_forward": {"flops": 0.0, "bytes": 2 * stream + full, "bytes_interface": zsz + 2 * stream + full + t * T * 4},
    }
    if w.backward:
        # dX, Hn, dHn in, dR out; the interface also writes the reduced shared gradient gs [T, S] (compact: gs is
        # dRs, part of dR) and reads rstd
        gs = 0 if compact else T * S * e
        out["rows_backward"] = {"flops": 0.0, "bytes": full + 3 * stream, "bytes_interface": full + 3 * stream + gs + t * T * 4}
        # W in, dY out / Y in, dW (fp32) out; the gradient operand is dR and the slab, already counted above
        out["tc_gemm_dgrad"] = {"flops": fl, "bytes": (K * h + T * K) * e, "bytes_interface": zsz + (K * h + T * K) * e}
        out["tc_gemm_wgrad"] = {"flops": fl, "bytes": T * K * e + K * h * 4, "bytes_interface": zsz + T * K * e + K * h * 4}
    return out


def colpar_work(w):
    """Algorithmic work of the column-parallel MLP half (gate|up GEMM per rank + SwiGLU), e = 2 bytes."""
    t, T, h, F, e = w.t, w.tokens, w.h, w.kr_mlp, 2
    fl = 2.0 * t * T * h * 2 * F
    b_f = (t * T * h + t * 2 * F * h + t * T * 2 * F) * e
    out = {"tc_gemm_forward": {"flops": fl, "bytes": b_f, "bytes_interface": b_f},
           "activation": {"flops": 0.0, "bytes": t * T * 3 * F * e, "bytes_interface": t * T * 3 * F * e}}
    if w.backward:
        out["activation"]["bytes"] += t * T * 5 * F * e
        out["activation"]["bytes_interface"] += t * T * 5 * F * e
        b_d = (t * T * 2 * F + t * 2 * F * h + t * T * h) * e
        b_w = (t * T * 2 * F + t * T * h) * e + t * 2 * F * h * 4
        out["tc_gemm_dgrad"] = {"flops": fl, "bytes": b_d, "bytes_interface": b_d}
        out["tc_gemm_wgrad"] = {"flops": fl, "bytes": b_w, "bytes_interface": b_w}
    return out


def layer_widths(w):
    return (w.kr_mlp,) if w.kind in ("mlp", "layer") else (w.kr_attn, w.kr_mlp)


def step_work(w, S, compact=False):
    tot = {}
    parts = [layer_work(w, S, k_r, compact) for k_r in layer_widths(w)]
    if w.kind == "mlp":
        parts.append(colpar_work(w))
    for part in parts:
        for kind, v in part.items():
            a = tot.setdefault(kind, {"flops": 0.0, "bytes": 0.0, "bytes_interface": 0.0})
            for k in a:
                a[k] += v[k]
    if w.dtype == "f32":      # fp32 runs the CUDA-core GEMM (TF32 cannot meet the 1e-4 tolerance)
        tot["gemm_cuda_core"] = tot.pop("tc_gemm_forward")
    return tot


def paper_level_work(w, S, compact=False):
    """Whole-path algorithmic work per step (no scratch traffic): the roofline of the path."""
    t, T, h, e = w.t, w.tokens, w.h, esize(w)
    full = t * T * h
    stream = T * S + t * T * (h - S) if compact else full
    fl = by = 0.0
    if w.kind == "mlp":   # column-parallel half: X, A in; pre kept for the backward; dX, dA out
        F = w.kr_mlp
        fl += 2.0 * t * T * h * 2 * F * (3 if w.backward else 1)
        by += e * (full + t * 2 * F * h + t * T * 2 * F) + (e * (t * T * 2 * F + full) + 4 * t * 2 * F * h if w.backward else 0)
    for k_r in layer_widths(w):
        K = k_r * t
        fl += 2.0 * T * K * h
        by += e * (T * K + K * h + 2 * stream + full)
        if w.backward:
            fl += 4.0 * T * K * h
            by += e * (full + 3 * stream + 2 * T * K + K * h) + 4 * K * h
    return fl, by


# --------------------------------------------------------------------------- the CUDA arm
class BlockRunner:
    overlap = None     # --overlap / --no-overlap force CAAT_OPT_BLOCK_OVERLAP to 1 / 0; None: the library's own choice

    def __init__(self, w, device, compact=False):
        from paper_2506_19645_b200 import caat
        self.caat, self.w, self.dev, self.compact = caat, w, device, compact
        self.ctx = caat.Context(w.h, w.ffn, w.t, w.p, w.dtype)
        if BlockRunner.overlap is not None:
            self.ctx.set_option(caat.CAAT_OPT_BLOCK_OVERLAP, 1 if BlockRunner.overlap else 0)
        self.S = self.ctx.shared_channels
        self.inp = synthetic.block_inputs(w, self.S, device=device)
        t, T, h = w.t, w.tokens, w.h
        td = self.ctx.torch_dtype
        mk = lambda *s, dt=td: torch.empty(*s, dtype=dt, device=device)
        f32 = torch.float32
        if compact:
            # same synthetic block, with the (tied) shared channels of the stream kept once
            S, i = self.S, self.inp
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


class LayerRunner:
    """One MLP-down-like row-parallel layer, forward only (the small fp32 configuration)."""

    def __init__(self, w, device, compact=False):
        from paper_2506_19645_b200 import caat
        assert not compact and not w.backward
        self.caat, self.w, self.dev, self.compact = caat, w, device, False
        self.ctx = caat.Context(w.h, w.ffn, w.t, w.p, w.dtype)
        self.S = self.ctx.shared_channels
        d = synthetic.layer_inputs(w.t, w.tokens, w.h, w.kr_mlp, w.dtype, seed=w.seed, S=self.S, device=device)
        self.inp = {k: d[k] for k in ("Y", "W", "R", "gamma")}
        self.out = self.ctx.alloc_forward_outputs(w.tokens, device=device)
        self.out = {k: v for k, v in self.out.items() if v is not None}
        self.ws = self.ctx.alloc_workspace(self.ctx.workspace_bytes(caat.CAAT_MLP_DOWN, w.tokens, False), device=device)

    def step(self):
        i, o = self.inp, self.out
        self.ctx.rowpar_forward(self.caat.CAAT_MLP_DOWN, self.w.tokens, i["Y"], i["W"], i["R"], i["gamma"], None, o["Hn"],
                                o["X"], o["rstd"], None, self.ws)

    touched_bytes = BlockRunner.touched_bytes


class MlpRunner:
    """The whole tensor-parallel MLP: column-parallel gate|up + SwiGLU, then the MLP-down layer with partial
    channel-reduce (and the gradient of both), as two library calls per direction."""

    def __init__(self, w, device, compact=False):
        from paper_2506_19645_b200 import caat
        assert not compact
        self.caat, self.w, self.dev, self.compact = caat, w, device, False
        self.ctx = caat.Context(w.h, w.ffn, w.t, w.p, w.dtype)
        self.S = self.ctx.shared_channels
        self.inp = synthetic.mlp_inputs(w, self.S, device=device)
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

    touched_bytes = BlockRunner.touched_bytes


# The 8-GPU all-reduce bus bandwidth quoted for this pool's NVSwitch machines at a 1 GiB payload (nominal NVLink 5:
# 900 GB/s per direction per GPU).  NOT measured by this repository (no run here had more than one GPU); the
# payloads below are 17-134 MB, where a real collective reaches less, so the all-reduce times are lower bounds.
# NCCL's convention: time = 2 (n - 1) / n * bytes / bus bandwidth.
NVLINK_ALLREDUCE_BUSBW_GBS = 725.0


def tp_projection(dev, name="block_7b", steps=20):
    """What the paper's claim looks like on this hardware, PROJECTED: ONE GPU's share of a real t-GPU run of the
    two row-parallel sub-layers of a block (one rank per GPU; no attention, no column-parallel GEMMs), timed with
    the library's two halves of every layer call and no collective, next to the time the four all-reduces of a
    step (Appendix C) would take for the analytic payload at the bandwidth above, not overlapped.  Nothing here
    ran on more than one GPU; `bench.py --mode tp` is the measurement."""
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
    return {"title": "row-parallel sub-layers only, projected", "workload": name, "gpus": G, "ranks_per_gpu": 1, "tokens": T,
            "allreduce_bus_bandwidth_gbs": NVLINK_ALLREDUCE_BUSBW_GBS,
            "allreduce_bus_bandwidth_source": "figure quoted for this pool's 8-GPU NVSwitch machines at 1 GiB; nominal for "
                                              "this repository (never measured here), optimistic at these 17-134 MB payloads",
            "note": "projection: measured one-GPU compute of the two row-parallel sub-layers (two-halves calls, no "
                    "collective; no attention or column-parallel GEMMs, so not comparable with whole-model speed-ups) + "
                    "analytic all-reduce time (2 forward 16-bit + 2 backward fp32 reduces per block, ring factor "
                    "2(n-1)/n), no overlap; not a multi-GPU measurement",
            "rows": rows}


def library_gemm_yardstick(w, dev, secs=1.0):
    """Context for the GEMM fractions, NOT part of the path: the vendor library's batched GEMM (torch.bmm) on the
    workload's own shapes - t products [T, K_r] x [K_r, h] and their two gradient products per layer - each run back to
    back for about `secs` seconds, i.e. under the same power cap as the step.  The peak the fractions are quoted
    against comes from an 8192^3 product; the layer's shards are shorter in the contraction and write more output per
    flop, and this says how much of the gap the shapes themselves account for."""
    t, T, h = w.t, w.tokens, w.h
    out = {}
    bf = torch.bfloat16

    def sustained(fn, flops):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        n, t0 = 0, time.perf_counter()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        while True:
            for _ in range(5):
                fn()
            n += 5
            if time.perf_counter() - t0 > secs:
                break
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / n
        return ms, flops / (ms * 1e-3) / 1e12

    tot = {"forward": [0.0, 0.0], "dgrad": [0.0, 0.0], "wgrad": [0.0, 0.0]}
    for K in layer_widths(w):
        Y = torch.randn(t, T, K, device=dev, dtype=bf)
        W = torch.randn(t, h, K, device=dev, dtype=bf) * 0.02
        Gd = torch.randn(t, T, h, device=dev, dtype=bf)
        Z, dY, dW = torch.empty(t, T, h, device=dev, dtype=bf), torch.empty_like(Y), torch.empty_like(W)
        fl = 2.0 * t * T * K * h
        for kind, fn in (("forward", lambda: torch.bmm(Y, W.transpose(1, 2), out=Z)), ("dgrad", lambda: torch.bmm(Gd, W, out=dY)),
                         ("wgrad", lambda: torch.bmm(Gd.transpose(1, 2), Y, out=dW))):
            ms, _ = sustained(fn, fl)
            tot[kind][0] += ms
            tot[kind][1] += fl
        del Y, W, Gd, Z, dY, dW
        torch.cuda.empty_cache()
    for kind, (ms, fl) in tot.items():
        out[kind] = {"ms_per_step": ms, "tflops": fl / (ms * 1e-3) / 1e12}
    out["note"] = ("vendor-library batched GEMM (torch.bmm, bf16) on this workload's per-rank shapes, both layers, each "
                   f"product looped for about {secs:g} s; a yardstick for the shapes, not a step of the path")
    return out


def make_runner(w, device, compact=False):
    if w.kind == "mlp":
        return MlpRunner(w, device, compact)
    if w.kind == "layer":
        return LayerRunner(w, device, compact)
    return BlockRunner(w, device, compact)


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
    return min(128, int(2 * L2_BYTES // max(touched_bytes, 1)) + 2)


def time_steps(runner, steps, dist_on, graph=None, per_step=False):
    """Device time of exactly `steps` steps (ms), CUDA events on the launching stream.  `runner` and
    `graph` may be lists (buffer sets rotated step by step).  per_step: also an event after every step;
    returns (total, [per-step ms])."""
    runners = runner if isinstance(runner, list) else [runner]
    graphs = graph if isinstance(graph, list) else ([graph] if graph is not None else None)
    torch.cuda.synchronize()
    if dist_on:
        torch.distributed.barrier()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1 if per_step else 2)]
    ev[0].record()
    for q in range(steps):
        if graphs is not None:
            graphs[q % len(graphs)].replay()
        else:
            runners[q % len(runners)].step()
        if per_step:
            ev[q + 1].record()
    if not per_step:
        ev[1].record()
    torch.cuda.synchronize()
    if dist_on:
        torch.distributed.barrier()
    total = ev[0].elapsed_time(ev[-1])
    if per_step:
        return total, [ev[q].elapsed_time(ev[q + 1]) for q in range(steps)]
    return total


def step_stats(per_step_ms):
    s = sorted(per_step_ms)
    return {"median": statistics.median(s), "min": s[0], "max": s[-1], "n": len(s)}


def kernel_table(prof, work, steps, peaks):
    """Per kernel kind: device time per step from CUDA events around every launch, and the achieved rate on the
    kind's algorithmic work against the peak that bounds it (both bf16 denominators named)."""
    total = sum(v[0] for v in prof.values()) or 1.0
    kernels = {}
    for kind, (kms, n) in prof.items():
        per_step_ms = kms / steps
        ent = {"ms_per_step": per_step_ms, "launches_per_step": n / steps, "share": kms / total}
        wk = work.get(kind)
        if wk and per_step_ms > 0:
            sec = per_step_ms * 1e-3
            gbs, tfs = wk["bytes"] / sec / 1e9, wk["flops"] / sec / 1e12
            t_hbm = wk["bytes"] / (peaks["hbm_gbs"] * 1e9)
            t_tc = wk["flops"] / (peaks["bf16_tflops_sustained"] * 1e12)
            if t_tc > t_hbm:
                ent.update({"bound": "tensor", "achieved": tfs, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                            "frac": tfs / peaks["bf16_tflops_sustained"], "peak_name": "bf16_tflops_sustained",
                            "frac_of_burst_peak": tfs / peaks["bf16_tflops_burst"]})
            else:
                ent.update({"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                            "frac": gbs / peaks["hbm_gbs"], "peak_name": "hbm_gbs",
                            "interface_gbs": wk["bytes_interface"] / sec / 1e9})
            ent["algorithmic_bytes_per_step"], ent["flops_per_step"] = wk["bytes"], wk["flops"]
        kernels[kind] = ent
    return kernels


def path_roofline(w, S, compact, ms_step, peaks, kernels=None):
    """The whole step against its roofline: `roofline_ms` takes the step's algorithmic bytes and flops as if the
    HBM-bound kernels ran fully hidden behind the tensor-bound ones (the larger of the two totals); with the per-kernel
    table, `kernel_sum_roofline_ms` is the stricter companion: every kernel kind at the peak that bounds IT, one after
    the other, which is what a chain of dependent kernels can reach without running two of them side by side."""
    fl, by = paper_level_work(w, S, compact)
    t_hbm = by / (peaks["hbm_gbs"] * 1e9) * 1e3
    t_sus = fl / (peaks["bf16_tflops_sustained"] * 1e12) * 1e3
    t_bur = fl / (peaks["bf16_tflops_burst"] * 1e12) * 1e3
    out = {"flops_per_step": fl, "bytes_per_step": by, "bound": "tensor" if t_sus > t_hbm else "hbm",
           "roofline_ms": max(t_sus, t_hbm), "frac": max(t_sus, t_hbm) / ms_step,
           "roofline_ms_burst_peak": max(t_bur, t_hbm), "frac_burst_peak": max(t_bur, t_hbm) / ms_step,
           "hbm_ms": t_hbm, "tensor_ms_sustained": t_sus, "tensor_ms_burst": t_bur,
           "denominators": {"hbm_gbs": peaks["hbm_gbs"], "bf16_tflops_sustained": peaks["bf16_tflops_sustained"],
                            "bf16_tflops_burst": peaks["bf16_tflops_burst"], "source": peaks["source"]}}
    if kernels:
        t_sum = 0.0
        for ent in kernels.values():
            if "algorithmic_bytes_per_step" in ent:
                t_sum += max(ent["algorithmic_bytes_per_step"] / (peaks["hbm_gbs"] * 1e9),
                             ent["flops_per_step"] / (peaks["bf16_tflops_sustained"] * 1e12)) * 1e3
        out["kernel_sum_roofline_ms"] = t_sum
        out["frac_of_kernel_sum_roofline"] = t_sum / ms_step
    return out


def measure(w, dev, steps, warm, dist_on, compact=False, no_graph=False, kernels=True):
    """Everything the bench reports about one workload on this GPU: the timed pass of exactly `steps` steps, a pass
    with an event after every step (median / min), a pass with events around every kernel, and - for working sets
    that fit the L2 - the same steps on one buffer set.  Returns (dict, runner)."""
    from paper_2506_19645_b200 import caat
    runner = make_runner(w, dev, compact)
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
    graph, per_step = None, 0
    probe = time_steps(rset, 5, False) / 5
    if probe < 0.25 and not no_graph:
        caps = [capture_step(r) for r in rset]
        if all(g is not None for g, _ in caps):
            graph, per_step = [g for g, _ in caps], caps[0][1]
    l0 = caat.kernel_launches()
    ms = time_steps(rset, steps, dist_on, graph)
    launches = per_step * steps if graph is not None else caat.kernel_launches() - l0
    _, each = time_steps(rset, steps, False, graph, per_step=True)
    out = {"ms_total": ms, "launches": int(launches), "step_ms": step_stats(each), "nsets": nsets,
           "graph": graph is not None, "touched_bytes": runner.touched_bytes()}
    if kernels:
        # second pass of the same K steps with CUDA events around every kernel (per-kernel device times)
        caat.profile_begin(max(1024, (launches if graph is None else 64 * steps) + 64))
        ms_prof = time_steps(rset, steps, False)
        out["prof"], out["ms_prof"] = caat.profile_end(), ms_prof
    if nsets > 1:
        # the same steps on ONE buffer set, i.e. with whatever fits staying in L2 (reported separately)
        out["ms_warm_l2"] = time_steps(rset[:1], steps, False, graph[:1] if graph is not None else None) / steps
    del rset[1:], graph
    return out, runner


def l2_note(m):
    tb = m["touched_bytes"] / 1e6
    if m["nsets"] == 1:
        return f"inputs+outputs touched per step {tb:.0f} MB > 126 MB L2"
    return (f"{m['nsets']} buffer sets rotated step by step: {tb:.1f} MB touched per step, "
            f"{(m['nsets'] - 1) * tb:.0f} MB of other sets between two uses of a set (L2 126 MB)")


def e2e_leg(runner, steps):
    """Same step through the public API with HOST buffers: every step copies its inputs from pinned
    host memory and reads its results back to pinned host memory, all inside the timed region.  The three
    phases run on three streams over two sets of device buffers, so the copy of step s+1, the
    kernels of step s and the read-back of step s-1 overlap (PCIe moves both ways at once)."""
    runners = [runner, make_runner(runner.w, runner.dev, runner.compact)]
    inp_host = {k: v.cpu().pin_memory() for k, v in runner.inp.items()}
    # one host copy of the results: read-backs are serialised on their stream, each step overwrites the last
    out_host = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in runner.out.items()}
    h2d = sum(v.numel() * v.element_size() for v in inp_host.values())
    d2h = sum(v.numel() * v.element_size() for v in out_host.values())
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
                out_host[k].copy_(v, non_blocking=True)
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
    """One forward(+backward) of the fp64 oracle on `sample_tokens` tokens of the workload."""
    from oracle import caat_oracle as O
    ws = w.with_tokens(sample_tokens)
    S, alpha = O.shared_channels(ws.h, ws.p), math.sqrt(ws.t)
    if w.kind == "mlp":
        d = {k: v.to(torch.float64).numpy() for k, v in synthetic.mlp_inputs(ws, S, device="cpu").items()}
        t0 = time.perf_counter()
        f = O.mlp_forward(d["X"], d["A"], d["B"], d["R"], d["gamma"], S=S, alpha=alpha)
        if w.backward:
            O.mlp_backward(d["dXout"], d["dHn"], d["X"], d["A"], d["B"], f["pre"], f["Y"], f["Hn"], f["rstd"], None,
                           d["gamma"], S=S, alpha=alpha)
        return time.perf_counter() - t0
    if w.kind == "layer":
        d = {k: v.to(torch.float64).numpy() for k, v in
             synthetic.layer_inputs(ws.t, ws.tokens, ws.h, ws.kr_mlp, ws.dtype, seed=ws.seed, S=S).items()}
        t0 = time.perf_counter()
        O.rowpar_forward(d["Y"], d["W"], d["R"], d["gamma"], None, S=S, alpha=alpha)
        return time.perf_counter() - t0
    d = {k: v.to(torch.float64).numpy() for k, v in synthetic.block_inputs(ws, S, device="cpu").items()}
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


def passes(w):
    return "forward+backward" if w.backward else "forward"


def cpu_baseline(w, target_s=12.0):
    probe = min(256, w.tokens)
    tp = oracle_sample_run(w, probe)
    tp = min(tp, oracle_sample_run(w, probe))
    n = int(target_s / max(tp / probe, 1e-9))
    n = max(probe, min(w.tokens, n // 256 * 256 if n >= 256 else probe))
    ts = oracle_sample_run(w, n)
    return {"value": n / ts, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
            "sample": f"fp64 numpy oracle, {w.kind} {passes(w)} on {n} of {w.tokens} tokens "
                      f"of {w.name} (all {w.t} ranks), {ts:.2f} s; host has {len(os.sched_getaffinity(0))} usable cores"}


def config_of(w, S, world, compact, m):
    return {"workload": w.name, "t": w.t, "tokens": w.tokens, "h": w.h, "ffn": w.ffn, "p": w.p,
            "S": S, "passes": passes(w), "private_scale": "sqrt(t)", "norm": "rmsnorm", "parallelism": f"replicas x{world}",
            "residual_layout": "compact (shared channels of the stream stored once)" if compact else "per rank [t,T,h]",
            "launch": "cuda graph replay" if m["graph"] else "eager", "l2": l2_note(m),
            "block_forward_schedule": {None: "library's choice by shape (side by side unless the GEMM is much the longer kernel)",
                                       True: "row kernel of layer 1 beside the GEMM of layer 2 (two streams)",
                                       False: "kernels one after the other"}[BlockRunner.overlap]}


def sweep_entry(name, dev, steps, peaks):
    """One workload of the sweep with its own per-kernel table (same timing rules as the headline)."""
    w = synthetic.WORKLOADS[name]
    k = max(10, min(steps, 50)) if w.tokens > 64 else max(50, min(steps, 200))
    m, r = measure(w, dev, k, 5, False)
    S = r.S
    sms = m["ms_total"] / k
    ent = {"workload": name, "p": w.p, "S": S, "passes": passes(w), "dtype": w.dtype, "steps": k, "ms_per_step": sms,
           "step_ms": m["step_ms"], "tokens_per_s": w.tokens / (sms * 1e-3), "launch": "cuda graph replay" if m["graph"] else "eager",
           "l2": l2_note(m), "kernels": kernel_table(m["prof"], step_work(w, S), k, peaks),
           "allreduce_payload_bytes": r.ctx.allreduce_bytes(w.tokens, 2)["payload_per_rank"]}
    ent["path_roofline"] = path_roofline(w, S, False, sms, peaks, ent["kernels"])
    ent["path_roofline_frac"] = ent["path_roofline"]["frac"]
    if "ms_warm_l2" in m:
        ent["warm_l2"] = {"ms_per_step": m["ms_warm_l2"], "tokens_per_s": w.tokens / (m["ms_warm_l2"] * 1e-3),
                          "path_roofline_frac": ent["path_roofline"]["roofline_ms"] / m["ms_warm_l2"],
                          "note": "same steps on a single buffer set (operands that fit stay in the 126 MB L2); the "
                                  "entry's own figures are the rotated, cold-L2 ones"}
    del r
    torch.cuda.empty_cache()
    if w.kind == "block" and w.tokens > 64 and BlockRunner.overlap is None:
        # the same block with the forward's schedule forced either way (CAAT_OPT_BLOCK_OVERLAP = 0 / 1), same steps.
        # The kernel table above comes from the library's own schedule: where two kernels share the GPU their event
        # times include each other's slow-down, so the serial pass's table is printed as well.
        for flag, key in ((False, "serial_forward"), (True, "side_by_side_forward")):
            BlockRunner.overlap = flag
            try:
                m2, r2 = measure(w, dev, k, 3, False, kernels=not flag)
                ent[key + "_ms_per_step"] = m2["ms_total"] / k
                if not flag:
                    ent["kernels_serial_forward"] = kernel_table(m2["prof"], step_work(w, S), k, peaks)
                del r2
                torch.cuda.empty_cache()
            finally:
                BlockRunner.overlap = None
    if w.kind == "block" and w.tokens > 64 and S % 8 == 0:
        # the same block on the compact residual layout (shared channels of the stream stored once)
        r = BlockRunner(w, dev, True)
        for _ in range(3):
            r.step()
        cms = time_steps(r, k, False) / k
        ent["compact_layout_ms_per_step"] = cms
        ent["compact_layout_tokens_per_s"] = w.tokens / (cms * 1e-3)
        del r
        torch.cuda.empty_cache()
    return ent


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
    warm = max(args.warmup, 3)
    sampler = ClockSampler(local)
    sampler.start()
    m, runner = measure(w, dev, args.steps, warm, dist_on, compact, args.no_graph)
    clocks = sampler.stop()
    S = runner.S
    ms = replicas.max_over_ranks(m["ms_total"], dev)
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
               "overlap": "copy-in, kernels and read-back of consecutive steps on three streams, two device buffer sets, "
                          "pinned host memory both ways"}
    except Exception as ex:  # pinned-memory exhaustion on a small host
        if dist_on:
            replicas.max_over_ranks(0.0, dev)     # keep the ranks' collectives matched
        e2e = {"value": None, "unit": "tokens/s", "h2d_bytes_per_step": None, "d2h_bytes_per_step": None,
               "error": "end-to-end leg not measured (host could not pin the step's buffers, or skipped): " + str(ex)[:200]}

    result = None
    if rank == 0:
        peaks = measured_peaks()
        kernels = kernel_table(m["prof"], step_work(w, S, compact), args.steps, peaks)
        top = max((k for k in kernels if "frac" in kernels[k]), key=lambda k: kernels[k]["ms_per_step"])
        roof = {k: kernels[top][k] for k in ("bound", "achieved", "peak", "unit", "frac", "peak_name")}
        if "frac_of_burst_peak" in kernels[top]:
            roof["frac_of_burst_peak"] = kernels[top]["frac_of_burst_peak"]
        roof.update({"kernel": top, "traffic": recorded_traffic(top, w.name + ("@compact" if compact else "")),
                     "peak_source": peaks["source"] + ("; sustained bf16 figure: the kernel is timed inside a long step"
                                                       if roof["bound"] == "tensor" else ""),
                     "timed": f"pass of {args.steps} steps with CUDA events around every kernel launch "
                              f"({m['ms_prof'] / args.steps:.4f} ms/step with events); achieved = the kind's algorithmic "
                              f"work per step / its event time per step"})
        ar = runner.ctx.allreduce_bytes(w.tokens, 2)
        result = {
            "metric": metric_name(w), "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": warm,
            "ms_per_step": ms_step, "step_ms": m["step_ms"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": w.dtype, "data": "synthetic", "config": config_of(w, S, world, compact, m),
            "clocks": clocks, "gpu_launches": m["launches"], "e2e": e2e, "roofline": roof, "kernels": kernels,
            "path_roofline": path_roofline(w, S, compact, ms_step, peaks, kernels),
            "collective_bytes_analytic": {"per_reduce": ar, "reduces_per_step": 4 if w.backward else 2},
        }
        if "ms_warm_l2" in m:
            result["warm_l2"] = {"ms_per_step": m["ms_warm_l2"], "tokens_per_s": w.tokens / (m["ms_warm_l2"] * 1e-3),
                                 "note": "same steps on a single buffer set (operands that fit stay in the 126 MB L2); "
                                         "not the headline figure"}
    del runner
    torch.cuda.empty_cache()

    if rank == 0 and world == 1 and not args.no_sweep and w.kind == "block" and w.backward and w.dtype == "bf16":
        try:
            result["library_gemm_same_shapes"] = library_gemm_yardstick(w, dev)
            for kind, v in result["library_gemm_same_shapes"].items():
                k = "tc_gemm_" + kind
                if isinstance(v, dict) and k in result["kernels"] and "achieved" in result["kernels"][k]:
                    result["kernels"][k]["vs_library_gemm_same_shapes"] = result["kernels"][k]["achieved"] / v["tflops"]
        except Exception as ex:  # noqa: BLE001
            result["library_gemm_same_shapes"] = {"error": str(ex)[:200]}
            torch.cuda.empty_cache()

    if rank == 0 and not args.no_sweep and world == 1:
        sweep = []
        peaks = measured_peaks()
        for name in SWEEP:
            if name == w.name and not compact:
                continue
            try:
                sweep.append(sweep_entry(name, dev, args.steps, peaks))
            except Exception as ex:  # noqa: BLE001
                sweep.append({"workload": name, "error": str(ex)[:200]})
                torch.cuda.empty_cache()
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
    from oracle import caat_oracle as O
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
    sample = (f"fp64 numpy oracle, {w.kind} {passes(w)}, each step a sample of {n} of "
              f"{w.tokens} tokens of {w.name}; host has {len(os.sched_getaffinity(0))} usable cores")
    print(json.dumps({
        "impl": "reference", "metric": metric_name(w), "value": value, "unit": "tokens/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "t": w.t, "tokens": w.tokens, "h": w.h, "ffn": w.ffn, "p": w.p,
                   "S": O.shared_channels(w.h, w.p), "passes": passes(w), "sample_tokens": n},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--mode", default="replicas", choices=["replicas", "tp"],
                    help="replicas: one independent replica of the workload per GPU (the benchmark); tp: the "
                         "tensor-parallel ranks split over the GPUs, all-reduce of the shared-channel slab, p sweep")
    ap.add_argument("--tp-exchange", default="nccl", choices=["nccl", "push"],
                    help="--mode tp: the slab exchange - a library all-reduce, or the package's own kernels over peer memory")
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synthetic.WORKLOADS))
    ap.add_argument("--no-sweep", action="store_true", help="skip the other workloads' tokens/s")
    ap.add_argument("--no-cpu", action="store_true", help="skip the timed CPU oracle baseline")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-graph", action="store_true", help="never replay launch-bound steps from a CUDA graph")
    ap.add_argument("--no-overlap", action="store_true",
                    help="block forward: run the layers' kernels one after the other (CAAT_OPT_BLOCK_OVERLAP = 0)")
    ap.add_argument("--overlap", action="store_true",
                    help="block forward: run the first layer's row kernel beside the second layer's GEMM on two streams "
                         "(CAAT_OPT_BLOCK_OVERLAP = 1); default: the library chooses by shape")
    ap.add_argument("--layout", default="per_rank", choices=["per_rank", "compact"],
                    help="residual-stream layout: per rank [t,T,h] (the benchmark's configuration) or compact")
    ap.add_argument("--tokens", type=int, default=0, help="override the workload's token count (profiling on a small case)")
    args = ap.parse_args()
    if args.steps < 1:
        raise SystemExit("--steps must be >= 1")
    BlockRunner.overlap = True if args.overlap else (False if args.no_overlap else None)
    if args.impl == "reference":
        run_reference(args)
    elif args.mode == "tp":
        from paper_2506_19645_b200 import tp_bench
        tp_bench.run(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
