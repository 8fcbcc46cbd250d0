"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random tensors and names shapes.  It imports neither the
CUDA binding nor the oracle, so both sides of a parity test can be fed from it;
the channel partition S is not computed here: callers pass the value their side
computed (the library's ``caat_shared_channels`` or the oracle's
``shared_channels``) to say how many leading residual channels to tie.

Recipe: one ``torch.Generator`` per workload seeded with the workload's seed;
tensors are drawn in fp32 in the fixed order ``Y_attn, W_o, Y_mlp, W_down, R,
dX1, dX2, dHn2`` and then cast to the run's storage dtype.  Activations,
residual and upstream gradients ~ N(0, 1); weights ~ N(0, std 0.02); norm gain
1 (bias 0).  By default the residual's shared channels are identical on every
rank, which is the structure a real network with partially synchronised
activations has (the embedding is replicated and every later shared channel is
a rank sum).
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    t: int          # tensor-parallel ranks simulated as a batch dimension
    tokens: int     # T = batch x sequence
    h: int          # hidden size
    ffn: int        # MLP inner width (total, over all ranks)
    p: float        # synchronisation factor
    dtype: str      # "f32" | "bf16"  (storage type; accumulation is fp32)
    kind: str       # "layer" (one MLP-down-like layer) | "block" (attention-out + MLP-down) |
                    # "mlp" (column-parallel gate/up + SwiGLU, then the MLP-down layer)
    backward: bool
    seed: int = 0

    @property
    def kr_attn(self) -> int:
        return self.h // self.t

    @property
    def kr_mlp(self) -> int:
        return self.ffn // self.t

    def with_tokens(self, tokens: int) -> "Workload":
        return replace(self, tokens=tokens)


def _w(name, t, T, h, ffn, p, dtype, kind, backward):
    return Workload(name, t, T, h, ffn, p, dtype, kind, backward, 0)


WORKLOADS = {
    w.name: w for w in [
        _w("layer_fp32_small", 2, 128, 256, 1024, 0.5, "f32", "layer", False),
        _w("block_130m", 4, 8 * 2048, 768, 3072, 0.5, "bf16", "block", True),
        _w("block_1p1b_p100", 8, 8 * 2048, 2048, 5632, 1.0, "bf16", "block", True),
        _w("block_1p1b_p075", 8, 8 * 2048, 2048, 5632, 0.75, "bf16", "block", True),
        _w("block_1p1b_p050", 8, 8 * 2048, 2048, 5632, 0.5, "bf16", "block", True),
        _w("block_1p1b_p025", 8, 8 * 2048, 2048, 5632, 0.25, "bf16", "block", True),
        _w("block_7b", 8, 4 * 4096, 4096, 11008, 0.5, "bf16", "block", True),
    ] + [
        _w(f"decode_7b_T{T}_p{int(p * 100):03d}", 8, T, 4096, 11008, p, "bf16", "block", False)
        for T in (1, 8, 64) for p in (1.0, 0.5)
    ] + [
        # the whole tensor-parallel MLP of the same models: column-parallel half + row-parallel half
        _w("mlp_130m", 4, 8 * 2048, 768, 3072, 0.5, "bf16", "mlp", True),
        _w("mlp_1p1b_p050", 8, 8 * 2048, 2048, 5632, 0.5, "bf16", "mlp", True),
        _w("mlp_7b", 8, 4 * 4096, 4096, 11008, 0.5, "bf16", "mlp", True),
    ]
}


def torch_dtype(dtype: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]


def _randn(gen, shape, std, dtype, device):
    x = torch.randn(shape, generator=gen, dtype=torch.float32, device=device)
    if std != 1.0:
        x.mul_(std)
    return x.to(dtype)


def tie_shared_channels(R: torch.Tensor, S: int) -> torch.Tensor:
    """Copy rank 0's shared channels of a [t, T, h] tensor onto every rank (in place)."""
    if S > 0 and R.shape[0] > 1:
        R[1:, :, :S] = R[0:1, :, :S]
    return R


def layer_inputs(t, tokens, h, k_r, dtype="bf16", seed=0, S=0, backward=False,
                 tied_residual=True, device="cpu", weight_std=0.02) -> dict:
    """Inputs of one row-parallel sub-layer: Y [t,T,K_r], W [t,h,K_r], R [t,T,h], gamma, beta
    and, for the backward, dX [t,T,h] and dHn [t,T,h]."""
    td = torch_dtype(dtype)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    out = {
        "Y": _randn(gen, (t, tokens, k_r), 1.0, td, device),
        "W": _randn(gen, (t, h, k_r), weight_std, td, device),
        "R": _randn(gen, (t, tokens, h), 1.0, td, device),
        "gamma": torch.ones(h, dtype=td, device=device),
        "beta": torch.zeros(h, dtype=td, device=device),
    }
    if tied_residual:
        tie_shared_channels(out["R"], S)
    if backward:
        out["dX"] = _randn(gen, (t, tokens, h), 1.0, td, device)
        out["dHn"] = _randn(gen, (t, tokens, h), 1.0, td, device)
    return out


def mlp_inputs(w: Workload, S: int, tied_residual=True, device="cpu", weight_std=0.02) -> dict:
    """Inputs of a whole MLP: per-rank normalised input X [t,T,h], gate|up weights A [t, 2 ffn/t, h],
    down weights B [t, h, ffn/t], residual R, gain, and the upstream gradients of the backward."""
    td = torch_dtype(w.dtype)
    gen = torch.Generator(device=device)
    gen.manual_seed(w.seed)
    t, T, h, F = w.t, w.tokens, w.h, w.kr_mlp
    out = {
        "X": _randn(gen, (t, T, h), 1.0, td, device),
        "A": _randn(gen, (t, 2 * F, h), weight_std, td, device),
        "B": _randn(gen, (t, h, F), weight_std, td, device),
        "R": _randn(gen, (t, T, h), 1.0, td, device),
        "gamma": torch.ones(h, dtype=td, device=device),
    }
    if tied_residual:
        tie_shared_channels(out["R"], S)
    if w.backward:
        out["dXout"] = _randn(gen, (t, T, h), 1.0, td, device)
        out["dHn"] = _randn(gen, (t, T, h), 1.0, td, device)
    return out


def block_inputs(w: Workload, S: int, tied_residual=True, device="cpu", weight_std=0.02) -> dict:
    """Inputs of a block (attention-out then MLP-down) in the fixed drawing order; S = the caller's number of
    shared channels (the leading S channels of R0 are tied across ranks)."""
    td = torch_dtype(w.dtype)
    gen = torch.Generator(device=device)
    gen.manual_seed(w.seed)
    t, T, h = w.t, w.tokens, w.h
    out = {
        "Y_attn": _randn(gen, (t, T, w.kr_attn), 1.0, td, device),
        "W_o": _randn(gen, (t, h, w.kr_attn), weight_std, td, device),
        "Y_mlp": _randn(gen, (t, T, w.kr_mlp), 1.0, td, device),
        "W_down": _randn(gen, (t, h, w.kr_mlp), weight_std, td, device),
        "R0": _randn(gen, (t, T, h), 1.0, td, device),
        "gamma1": torch.ones(h, dtype=td, device=device),
        "gamma2": torch.ones(h, dtype=td, device=device),
    }
    if tied_residual:
        tie_shared_channels(out["R0"], S)
    if w.backward:
        out["dX1"] = _randn(gen, (t, T, h), 1.0, td, device)
        out["dX2"] = _randn(gen, (t, T, h), 1.0, td, device)
        out["dHn2"] = _randn(gen, (t, T, h), 1.0, td, device)
    return out


def small_integers(shape, lo, hi, dtype="bf16", seed=0, device="cpu") -> torch.Tensor:
    """Integer-valued tensor in [lo, hi]; exact in bf16 for small magnitudes."""
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    return torch.randint(lo, hi + 1, shape, generator=gen, device=device).to(torch_dtype(dtype))
