"""fp64 CPU oracle for the CAAT-Net row-parallel hot path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA path is checked against.  It shares no code with the CUDA path and is
imported only by the tests, by the smoke check and by the benchmark's
CPU-baseline leg.  Nothing in the product path may call it.

Everything is numpy float64.  Inputs are expected to be already rounded to the
run's storage type by the caller (the harness) and widened to float64, so the
oracle and the GPU see the same values.

Notation (paper's symbols in brackets):
  t        tensor-parallel ranks               [r, M; rank index m]
  T        tokens                              [b x t, s]
  h        hidden size                         [h]
  K_r      per-rank contraction width          [f / r]
  S        shared channels = floor(h * p)      [floor(hp), Eq. A3]
  alpha    private-channel scale, 1 or sqrt(t) [sqrt(r), Section 4 "Private channel scaling"]
  Y[m]     rank m's input  [T, K_r]            [Y_m, H_m]
  W[m]     rank m's weight shard stored out x in, [h, K_r]   [B~_{klm} as W[m][l][k]]
  Zt[m]    rank m's partial output [T, h]      [Z~_{ilm}]
  R[m]     residual entering the add           [R, R_m]
  Hn[m]    Z[m] + R[m], the new residual stream
  X[m]     Norm(Hn[m])                         [X_m, Eq. 9]

Pins (see tests/test_oracle_pins.py): the two-device closed form of Eq. 8, a
brute-force index-notation evaluation of Eq. A3, p=1 against an unsharded
library matmul plus library norms, p=0 independence, rank-permutation
invariance, the variance law of Eq. 14-15, central finite differences and the
p=1 reduce-before-norm equivalence of Section 4 for the backward, and the
closed forms of Appendix C for the byte counts.  The compact-layout functions
(shared part of the residual stream stored once) are pinned by their own finite
differences, by equality with the per-rank forward on a tied residual, and by the
rank-sum relation between a tied variable's gradient and its copies' gradients.
The column-parallel half (colpar_*, mlp_*) is pinned by library silu / autograd, by
finite differences, and by the textbook identity that with identical inputs on every
rank the concatenated shards equal the unsharded layer (Section 3, Eq. 2-3).

Parity unpinned (the paper fixes no value; these are this build's documented
choices): eps, the norm kind per model, the default of alpha, the dtype of dW.
The paper prints no worked numeric example of the operator, so no pin is a
printed value; all pins are closed forms, invariants and special cases.
"""
from __future__ import annotations

import math

import numpy as np

RMSNORM = 0
LAYERNORM = 1


# --------------------------------------------------------------------------
# F0: partition  (Section 3: the first h*p channels are shared; Eq. A3 floor(hp))
# --------------------------------------------------------------------------
def shared_channels(h: int, p: float) -> int:
    """S = floor(h * p) evaluated in IEEE double, as Eq. A3 writes it."""
    if not (0.0 <= p <= 1.0):
        raise ValueError("p must lie in [0, 1]")
    return int(math.floor(float(h) * float(p)))


def private_scale(t: int, enabled: bool = True) -> float:
    """Section 4, private channel scaling: sqrt(r) when on, 1 when off."""
    return math.sqrt(float(t)) if enabled else 1.0


# --------------------------------------------------------------------------
# F1: per-rank GEMM  (Eq. A3 first line / Eq. A5 second line)
# --------------------------------------------------------------------------
def rank_partials(Y: np.ndarray, W: np.ndarray) -> np.ndarray:
    """Zt[m, i, l] = sum_k Y[m, i, k] * W[m, l, k]."""
    Y = np.asarray(Y, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    t = Y.shape[0]
    return np.stack([Y[m] @ W[m].T for m in range(t)], axis=0)


# --------------------------------------------------------------------------
# F2 + F3: partial channel-reduce with private scaling  (Eq. A3 cases; Section 4)
# --------------------------------------------------------------------------
def partial_channel_reduce(Zt: np.ndarray, S: int, alpha: float = 1.0) -> np.ndarray:
    """Z[m, i, l] = sum_m' Zt[m', i, l] for l < S, alpha * Zt[m, i, l] for l >= S.

    The rank sum runs m' = 0 .. t-1 in that order.
    """
    Zt = np.asarray(Zt, dtype=np.float64)
    t = Zt.shape[0]
    Z = np.empty_like(Zt)
    if S > 0:
        Zs = np.zeros_like(Zt[0, :, :S])
        for m in range(t):
            Zs = Zs + Zt[m, :, :S]
        for m in range(t):
            Z[m, :, :S] = Zs
    Z[:, :, S:] = alpha * Zt[:, :, S:]
    return Z


# --------------------------------------------------------------------------
# F5: per-rank norm over all h channels of that rank  (Eq. 9; RMSNorm / LayerNorm)
# --------------------------------------------------------------------------
def norm_forward(Hn: np.ndarray, gamma: np.ndarray, beta, eps: float, norm: int):
    """Returns X, rstd, mean (mean is None for RMSNorm). Statistics per (rank, token)."""
    Hn = np.asarray(Hn, dtype=np.float64)
    gamma = np.asarray(gamma, dtype=np.float64)
    if norm == RMSNORM:
        ms = np.mean(Hn * Hn, axis=-1)
        rstd = 1.0 / np.sqrt(ms + eps)
        X = Hn * rstd[..., None] * gamma
        return X, rstd, None
    if norm == LAYERNORM:
        mu = np.mean(Hn, axis=-1)
        c = Hn - mu[..., None]
        var = np.mean(c * c, axis=-1)
        rstd = 1.0 / np.sqrt(var + eps)
        X = c * rstd[..., None] * gamma
        if beta is not None:
            X = X + np.asarray(beta, dtype=np.float64)
        return X, rstd, mu
    raise ValueError("unknown norm kind")


# --------------------------------------------------------------------------
# Forward of one row-parallel sub-layer  (F1..F5)
# --------------------------------------------------------------------------
def rowpar_forward(Y, W, R, gamma, beta=None, *, S: int, alpha: float = 1.0,
                   eps: float = 1e-5, norm: int = RMSNORM) -> dict:
    Zt = rank_partials(Y, W)                                  # F1
    Z = partial_channel_reduce(Zt, S, alpha)                  # F2, F3
    Hn = Z + np.asarray(R, dtype=np.float64)                  # F4 (Eq. 9 argument)
    X, rstd, mean = norm_forward(Hn, gamma, beta, eps, norm)  # F5
    return {"Zt": Zt, "Z": Z, "Hn": Hn, "X": X, "rstd": rstd, "mean": mean}


# --------------------------------------------------------------------------
# B1: norm backward (textbook) + residual gradient
# --------------------------------------------------------------------------
def norm_backward(dX, Hn, rstd, mean, gamma, norm: int) -> np.ndarray:
    """Gradient of X = Norm(Hn) w.r.t. Hn contracted with dX, per (rank, token) row."""
    dX = np.asarray(dX, dtype=np.float64)
    Hn = np.asarray(Hn, dtype=np.float64)
    rstd = np.asarray(rstd, dtype=np.float64)[..., None]
    gamma = np.asarray(gamma, dtype=np.float64)
    dxh = dX * gamma
    if norm == RMSNORM:
        xh = Hn * rstd
        c = np.mean(dxh * xh, axis=-1, keepdims=True)
        return rstd * (dxh - xh * c)
    if norm == LAYERNORM:
        mu = np.asarray(mean, dtype=np.float64)[..., None]
        xh = (Hn - mu) * rstd
        c1 = np.mean(dxh, axis=-1, keepdims=True)
        c2 = np.mean(dxh * xh, axis=-1, keepdims=True)
        return rstd * (dxh - c1 - xh * c2)
    raise ValueError("unknown norm kind")


def normalized(Hn, rstd, mean, norm: int) -> np.ndarray:
    """x_hat, the normalised row before gain and bias."""
    Hn = np.asarray(Hn, dtype=np.float64)
    rstd = np.asarray(rstd, dtype=np.float64)[..., None]
    if norm == RMSNORM:
        return Hn * rstd
    return (Hn - np.asarray(mean, dtype=np.float64)[..., None]) * rstd


def residual_stream_gradient(dX, dHn, Hn, rstd, mean, gamma, norm: int) -> np.ndarray:
    """B1/B2: g[m] = NormBwd(dX[m]) + dHn[m]; this is also dR[m] (not reduced over ranks)."""
    g = norm_backward(dX, Hn, rstd, mean, gamma, norm)
    if dHn is not None:
        g = g + np.asarray(dHn, dtype=np.float64)
    return g


def norm_param_gradients(dX, Hn, rstd, mean, norm: int):
    """B3: dgamma[l] = sum_m sum_i dX*x_hat ; dbeta[l] = sum_m sum_i dX (LayerNorm only).

    Summed over ranks as Section 4 requires for replicated norm parameters.
    """
    dX = np.asarray(dX, dtype=np.float64)
    xh = normalized(Hn, rstd, mean, norm)
    dgamma = np.sum(dX * xh, axis=(0, 1))
    dbeta = np.sum(dX, axis=(0, 1)) if norm == LAYERNORM else None
    return dgamma, dbeta


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round to bfloat16 (8 significand bits, round to nearest even) and widen back to float64.
    Written on the bit pattern of the float32 value: add 0x7FFF plus the last kept bit, drop 16 bits."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    out = (r & 0xFFFFFFFF).astype(np.uint32).view(np.float32).astype(np.float64)
    return np.where(np.isfinite(f), out, f.astype(np.float64))


def backward_partial_channel_reduce(g, S: int, alpha: float = 1.0, reduce_mode: int = 0) -> np.ndarray:
    """B4: the reduce placed after the norm's backward (operation 'h' of Fig. 2b).

    dZt[m, i, l] = sum_m' g[m', i, l] for l < S, alpha * g[m, i, l] for l >= S.
    It is the transpose of the forward partial channel-reduce.

    reduce_mode models the precision of the rank sum that Section 4 discusses (16-bit runs only):
      0  exact sum of the ranks' gradients (what fp32 accumulation approximates),
      1  every rank's term rounded to bfloat16 first (a 16-bit all-reduce payload), summed exactly,
      2  terms rounded to bfloat16 and the running sum rounded to bfloat16 after every addition,
         m ascending (accumulation in 16 bit).
    """
    g = np.asarray(g, dtype=np.float64)
    if reduce_mode == 0:
        return partial_channel_reduce(g, S, alpha)
    t = g.shape[0]
    dZt = np.empty_like(g)
    acc = np.zeros_like(g[0, :, :S])
    for m in range(t):
        acc = acc + round_bf16(g[m, :, :S])
        if reduce_mode == 2:
            acc = round_bf16(acc)
    for m in range(t):
        dZt[m, :, :S] = acc
    dZt[:, :, S:] = alpha * g[:, :, S:]
    return dZt


def data_gradient(dZt, W) -> np.ndarray:
    """B5: dY[m, i, k] = sum_l dZt[m, i, l] * W[m, l, k]."""
    W = np.asarray(W, dtype=np.float64)
    return np.stack([dZt[m] @ W[m] for m in range(dZt.shape[0])], axis=0)


def weight_gradient(dZt, Y) -> np.ndarray:
    """B6: dW[m, l, k] = sum_i dZt[m, i, l] * Y[m, i, k]."""
    Y = np.asarray(Y, dtype=np.float64)
    return np.stack([dZt[m].T @ Y[m] for m in range(dZt.shape[0])], axis=0)


def rowpar_backward(dX, dHn, Y, W, Hn, rstd, mean, gamma, *, S: int, alpha: float = 1.0,
                    norm: int = RMSNORM, reduce_mode: int = 0) -> dict:
    """Exact gradient of rowpar_forward w.r.t. (Y, W, R, gamma, beta), contracted with
    upstream dX (through the norm) and dHn (through the residual stream)."""
    g = residual_stream_gradient(dX, dHn, Hn, rstd, mean, gamma, norm)   # B1
    dgamma, dbeta = norm_param_gradients(dX, Hn, rstd, mean, norm)       # B3
    dZt = backward_partial_channel_reduce(g, S, alpha, reduce_mode)      # B4
    dY = data_gradient(dZt, W)                                           # B5
    dW = weight_gradient(dZt, Y)                                         # B6
    return {"g": g, "dR": g, "dZt": dZt, "dY": dY, "dW": dW, "dgamma": dgamma, "dbeta": dbeta}


# --------------------------------------------------------------------------
# V2: block = attention-out sub-layer then MLP-down sub-layer (two reduces per block,
# Appendix C), chained only through the residual stream.
# --------------------------------------------------------------------------
def block_forward(Y_attn, W_o, Y_mlp, W_down, R0, gamma1, gamma2, beta1=None, beta2=None, *,
                  S: int, alpha: float = 1.0, eps: float = 1e-5, norm: int = RMSNORM) -> dict:
    f1 = rowpar_forward(Y_attn, W_o, R0, gamma1, beta1, S=S, alpha=alpha, eps=eps, norm=norm)
    f2 = rowpar_forward(Y_mlp, W_down, f1["Hn"], gamma2, beta2, S=S, alpha=alpha, eps=eps, norm=norm)
    return {"Hn1": f1["Hn"], "X1": f1["X"], "rstd1": f1["rstd"], "mean1": f1["mean"],
            "Hn2": f2["Hn"], "X2": f2["X"], "rstd2": f2["rstd"], "mean2": f2["mean"]}


def block_backward(dX1, dX2, dHn2, Y_attn, W_o, Y_mlp, W_down, Hn1, rstd1, mean1, Hn2, rstd2,
                   mean2, gamma1, gamma2, *, S: int, alpha: float = 1.0, norm: int = RMSNORM) -> dict:
    b2 = rowpar_backward(dX2, dHn2, Y_mlp, W_down, Hn2, rstd2, mean2, gamma2, S=S, alpha=alpha, norm=norm)
    b1 = rowpar_backward(dX1, b2["dR"], Y_attn, W_o, Hn1, rstd1, mean1, gamma1, S=S, alpha=alpha, norm=norm)
    return {"dY_attn": b1["dY"], "dW_o": b1["dW"], "dY_mlp": b2["dY"], "dW_down": b2["dW"],
            "dR0": b1["dR"], "dHn1": b2["dR"], "dgamma1": b1["dgamma"], "dgamma2": b2["dgamma"],
            "dbeta1": b1["dbeta"], "dbeta2": b2["dbeta"]}


# --------------------------------------------------------------------------
# Compact ("logical devices on one GPU", Section 3.2) residual layout.  When every rank holds
# the same values on the shared channels of the residual stream - which the partial
# channel-reduce guarantees from the first layer on, if the stream entering the network is
# tied - those channels are ONE variable stored once:
#     Rs [T, S]  shared part          Rp [t, T, h - S]  private part of every rank
# The forward is the same map as rowpar_forward applied to R[m] = [Rs | Rp[m]]; the backward
# below is the gradient of that map with Rs (and Hns) treated as single variables, written
# out on its own (it does not go through rowpar_backward).
# --------------------------------------------------------------------------
def rowpar_forward_compact(Y, W, Rs, Rp, gamma, beta=None, *, S: int, alpha: float = 1.0,
                           eps: float = 1e-5, norm: int = RMSNORM) -> dict:
    Zt = rank_partials(Y, W)                                       # F1
    t, T, h = Zt.shape
    Zs = np.zeros((T, S))                                          # F2: rank sum, m ascending
    for m in range(t):
        Zs = Zs + Zt[m, :, :S]
    Hns = Zs + np.asarray(Rs, dtype=np.float64)                    # F4 on the shared channels, once
    Hnp = alpha * Zt[:, :, S:] + np.asarray(Rp, dtype=np.float64)  # F3 + F4 on the private channels
    X = np.empty((t, T, h))
    rstd = np.empty((t, T))
    mean = np.empty((t, T)) if norm == LAYERNORM else None
    for m in range(t):                                             # F5: statistics over all h channels of rank m
        row = np.concatenate([Hns, Hnp[m]], axis=1)
        X[m], rstd[m], mu = norm_forward(row, gamma, beta, eps, norm)
        if norm == LAYERNORM:
            mean[m] = mu
    return {"Hns": Hns, "Hnp": Hnp, "X": X, "rstd": rstd, "mean": mean}


def rowpar_backward_compact(dX, dHns, dHnp, Y, W, Hns, Hnp, rstd, mean, gamma, *, S: int,
                            alpha: float = 1.0, norm: int = RMSNORM) -> dict:
    """Gradient of rowpar_forward_compact contracted with dX (through every rank's norm), dHns
    (on the shared part of the outgoing stream, one variable) and dHnp (private parts).

    Hns feeds the norm of EVERY rank, so its gradient collects all ranks' norm backward: that
    rank sum is the backward partial channel-reduce (operation 'h' of Fig. 2b, after the norm
    backward).  Because Hns = sum_m Zt[m][:, :S] + Rs, the same tensor is the gradient of Rs
    and of the shared columns of every rank's Zt.
    """
    dX = np.asarray(dX, dtype=np.float64)
    Hns = np.asarray(Hns, dtype=np.float64)
    Hnp = np.asarray(Hnp, dtype=np.float64)
    t, T, h = dX.shape
    gs = np.zeros((T, S)) if dHns is None else np.asarray(dHns, dtype=np.float64).copy()
    gp = np.empty((t, T, h - S))
    dgamma = np.zeros(h)
    dbeta = np.zeros(h) if norm == LAYERNORM else None
    for m in range(t):
        row = np.concatenate([Hns, Hnp[m]], axis=1)
        mu = None if mean is None else np.asarray(mean, dtype=np.float64)[m]
        n_m = norm_backward(dX[m], row, np.asarray(rstd, dtype=np.float64)[m], mu, gamma, norm)   # B1
        gs = gs + n_m[:, :S]                                   # B4, m ascending, in full precision
        gp[m] = n_m[:, S:]
        dgamma += np.sum(dX[m] * normalized(row, np.asarray(rstd, dtype=np.float64)[m], mu, norm), axis=0)   # B3
        if norm == LAYERNORM:
            dbeta += np.sum(dX[m], axis=0)
    if dHnp is not None:
        gp = gp + np.asarray(dHnp, dtype=np.float64)
    dZt = np.empty((t, T, h))
    for m in range(t):
        dZt[m, :, :S] = gs
        dZt[m, :, S:] = alpha * gp[m]                          # private channels carry alpha
    return {"dRs": gs, "dRp": gp, "dZt": dZt, "dY": data_gradient(dZt, W), "dW": weight_gradient(dZt, Y),
            "dgamma": dgamma, "dbeta": dbeta}


def block_forward_compact(Y_attn, W_o, Y_mlp, W_down, R0s, R0p, gamma1, gamma2, beta1=None, beta2=None, *,
                          S: int, alpha: float = 1.0, eps: float = 1e-5, norm: int = RMSNORM) -> dict:
    f1 = rowpar_forward_compact(Y_attn, W_o, R0s, R0p, gamma1, beta1, S=S, alpha=alpha, eps=eps, norm=norm)
    f2 = rowpar_forward_compact(Y_mlp, W_down, f1["Hns"], f1["Hnp"], gamma2, beta2, S=S, alpha=alpha, eps=eps, norm=norm)
    return {"Hn1s": f1["Hns"], "Hn1p": f1["Hnp"], "X1": f1["X"], "rstd1": f1["rstd"], "mean1": f1["mean"],
            "Hn2s": f2["Hns"], "Hn2p": f2["Hnp"], "X2": f2["X"], "rstd2": f2["rstd"], "mean2": f2["mean"]}


def block_backward_compact(dX1, dX2, dHn2s, dHn2p, Y_attn, W_o, Y_mlp, W_down, Hn1s, Hn1p, rstd1, mean1,
                           Hn2s, Hn2p, rstd2, mean2, gamma1, gamma2, *, S: int, alpha: float = 1.0,
                           norm: int = RMSNORM) -> dict:
    b2 = rowpar_backward_compact(dX2, dHn2s, dHn2p, Y_mlp, W_down, Hn2s, Hn2p, rstd2, mean2, gamma2,
                                 S=S, alpha=alpha, norm=norm)
    b1 = rowpar_backward_compact(dX1, b2["dRs"], b2["dRp"], Y_attn, W_o, Hn1s, Hn1p, rstd1, mean1, gamma1,
                                 S=S, alpha=alpha, norm=norm)
    return {"dY_attn": b1["dY"], "dW_o": b1["dW"], "dY_mlp": b2["dY"], "dW_down": b2["dW"],
            "dR0s": b1["dRs"], "dR0p": b1["dRp"], "dHn1s": b2["dRs"], "dHn1p": b2["dRp"],
            "dgamma1": b1["dgamma"], "dgamma2": b2["dgamma"], "dbeta1": b1["dbeta"], "dbeta2": b2["dbeta"]}


# --------------------------------------------------------------------------
# Column-parallel half in front of the row-parallel layer (Section 3, "Y_m = sigma(X_m A_m)";
# Eq. A3, inner sum).  With partially synchronised activations every rank has its OWN input X_m
# (the per-rank norm output), so the layer is a batch of t independent products.
#   A[m]   rank m's weight shard stored out x in, [N, h]        [A~_{jkm} as A[m][k][j]]
#   NONE     out = X_m A_m^T                       (QKV projection: N = 3 h / t)
#   SILU     Y   = silu(X_m A_m^T)                 (an elementwise sigma, as Eq. A3 writes it)
#   SWIGLU   Y   = silu(G) * U,  [G | U] = X_m A_m^T,  N = 2 F  (the gated MLP of the Llama models
#            the paper trains; rows [0, F) of A_m are the gate, rows [F, 2F) the up projection)
# --------------------------------------------------------------------------
ACT_NONE = 0
ACT_SILU = 1
ACT_SWIGLU = 2


def silu(x: np.ndarray) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    return x / (1.0 + np.exp(-x))


def silu_grad(x: np.ndarray) -> np.ndarray:
    """d silu / dx = s (1 + x (1 - s)), s = logistic(x)."""
    x = np.asarray(x, dtype=np.float64)
    sg = 1.0 / (1.0 + np.exp(-x))
    return sg * (1.0 + x * (1.0 - sg))


def colpar_forward(X, A, act: int = ACT_NONE) -> dict:
    """pre[m] = X[m] A[m]^T; Y = act(pre).  Returns pre (saved for the backward) and Y."""
    pre = rank_partials(X, A)                    # the same batched product as F1, other operands
    if act == ACT_NONE:
        return {"pre": pre, "Y": pre}
    if act == ACT_SILU:
        return {"pre": pre, "Y": silu(pre)}
    if act == ACT_SWIGLU:
        F = pre.shape[2] // 2
        return {"pre": pre, "Y": silu(pre[:, :, :F]) * pre[:, :, F:]}
    raise ValueError("unknown activation")


def colpar_backward(dY, X, A, pre, act: int = ACT_NONE) -> dict:
    """Gradient of colpar_forward contracted with dY: dpre (through the activation), then
    dX[m] = dpre[m] A[m] and dA[m] = dpre[m]^T X[m], rank by rank (no cross-rank term:
    each rank's X_m is its own variable)."""
    dY = np.asarray(dY, dtype=np.float64)
    pre = np.asarray(pre, dtype=np.float64)
    if act == ACT_NONE:
        dpre = dY
    elif act == ACT_SILU:
        dpre = dY * silu_grad(pre)
    elif act == ACT_SWIGLU:
        F = pre.shape[2] // 2
        G, U = pre[:, :, :F], pre[:, :, F:]
        dpre = np.concatenate([dY * U * silu_grad(G), dY * silu(G)], axis=2)
    else:
        raise ValueError("unknown activation")
    return {"dpre": dpre, "dX": data_gradient(dpre, A), "dA": weight_gradient(dpre, X)}


def mlp_forward(X, A, B, R, gamma, beta=None, *, act: int = ACT_SWIGLU, S: int, alpha: float = 1.0,
                eps: float = 1e-5, norm: int = RMSNORM) -> dict:
    """A whole tensor-parallel MLP with partial channel-reduce (Eq. A3): column-parallel half on the
    per-rank inputs, then the row-parallel half with reduce, scaling, residual and norm."""
    c = colpar_forward(X, A, act)
    r = rowpar_forward(c["Y"], B, R, gamma, beta, S=S, alpha=alpha, eps=eps, norm=norm)
    return {"pre": c["pre"], "Y": c["Y"], "Hn": r["Hn"], "X": r["X"], "rstd": r["rstd"], "mean": r["mean"]}


def mlp_backward(dXout, dHn, X, A, B, pre, Y, Hn, rstd, mean, gamma, *, act: int = ACT_SWIGLU, S: int,
                 alpha: float = 1.0, norm: int = RMSNORM) -> dict:
    r = rowpar_backward(dXout, dHn, Y, B, Hn, rstd, mean, gamma, S=S, alpha=alpha, norm=norm)
    c = colpar_backward(r["dY"], X, A, pre, act)
    return {"dX": c["dX"], "dA": c["dA"], "dB": r["dW"], "dR": r["dR"], "dgamma": r["dgamma"], "dbeta": r["dbeta"]}


# --------------------------------------------------------------------------
# V3: analytic collective bytes  (Appendix C payload P(p); Appendix D volume law)
# --------------------------------------------------------------------------
def allreduce_bytes(tokens: int, h: int, t: int, S: int, elem_bytes: int = 2) -> dict:
    """Bytes a real tensor-parallel system would move for ONE partial channel-reduce.

    payload_per_rank:     tokens * S * e   (each device sends and receives that many activations)
    payload_per_rank_p1:  tokens * h * e   (the full all-reduce, p = 1)
    ring_wire_per_rank:   2 (t-1)/t * payload  (reduce-scatter + all-gather halves)
    """
    payload = tokens * S * elem_bytes
    payload_p1 = tokens * h * elem_bytes
    ring_num = 2 * (t - 1) * payload
    return {"payload_per_rank": payload, "payload_per_rank_p1": payload_p1,
            "ring_wire_per_rank": ring_num // t if ring_num % t == 0 else ring_num / t,
            "norm_grad_sync_bytes": h * 4}


def speedup_model(h: int, s: int, r: int, C: float, p: float) -> float:
    """Appendix C: (T(1) - T(p)) / T(1) with T = G/C' + P, written directly from
    G = (24 s h^2 + 4 s^2 h) / r, P(p) = 2 s h p and compute/communication ratio C."""
    G = (24.0 * s * h * h + 4.0 * s * s * h) / r
    t1 = G / C + 2.0 * s * h * 1.0
    tp = G / C + 2.0 * s * h * p
    return (t1 - tp) / t1
