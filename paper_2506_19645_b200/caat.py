"""Thin ctypes binding of libcaat.so (the C ABI declared in include/caat.h).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  PyTorch is used for device memory (``torch.empty``), ``data_ptr()`` and the
current CUDA stream.  There is no CPU fallback: without the built library the import
fails, and without a CUDA device the compute calls raise.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_double, c_int, c_size_t, c_uint, c_ulonglong, c_void_p

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libcaat.so")

CAAT_F32, CAAT_BF16 = 0, 1
CAAT_ATTN_OUT, CAAT_MLP_DOWN = 0, 1
(CAAT_OK, CAAT_EINVAL, CAAT_ESHAPE, CAAT_EALIGN, CAAT_EWORKSPACE, CAAT_EUNSUPPORTED, CAAT_ECUDA,
 CAAT_ETIMEOUT, CAAT_ELIMIT) = range(9)
CAAT_NOALLOC_SCRATCH_BYTES = 32 * 1024 * 1024
(CAAT_OPT_NORM, CAAT_OPT_EPS, CAAT_OPT_PRIVATE_SCALE, CAAT_OPT_SHARED_CHANNELS, CAAT_OPT_GEMM, CAAT_OPT_ROWS,
 CAAT_OPT_DECODE, CAAT_OPT_BACKWARD_REDUCE, CAAT_OPT_TP_GROUPS, CAAT_OPT_BLOCK_OVERLAP) = range(10)
RMSNORM, LAYERNORM = 0, 1
CAAT_MAX_PEERS, CAAT_TP_FLAG_BYTES = 8, 256


class caat_peers(Structure):
    """Mirror of the C struct: the GPUs of a slab exchange as this GPU addresses their buffers."""
    _fields_ = [("world", c_int), ("rank", c_int), ("recv", c_void_p * CAAT_MAX_PEERS),
                ("slab", c_void_p * CAAT_MAX_PEERS), ("flags", c_void_p * CAAT_MAX_PEERS)]
CAAT_ACT_NONE, CAAT_ACT_SILU, CAAT_ACT_SWIGLU = 0, 1, 2

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2506_19645_b200.build` "
                      "(there is no fallback path)")
lib = ctypes.CDLL(LIB_PATH)

_P = c_void_p
_sigs = {
    "caat_create": (c_int, [c_int, c_int, c_int, c_double, c_int, POINTER(c_void_p)]),
    "caat_set_option": (c_int, [_P, c_int, c_double]),
    "caat_destroy": (None, [_P]),
    "caat_shared_channels": (c_int, [_P]),
    "caat_private_scale": (c_double, [_P]),
    "caat_workspace_bytes": (c_size_t, [_P, c_int, c_int, c_int]),
    "caat_block_workspace_bytes": (c_size_t, [_P, c_int, c_int]),
    "caat_strerror": (c_char_p, [c_int]),
    "caat_last_cuda_error": (c_char_p, []),
    "caat_rowpar_forward": (c_int, [_P, c_int, c_int] + [_P] * 9 + [_P, c_size_t, _P]),
    "caat_rowpar_forward_noalloc": (c_int, [_P, c_int, c_int] + [_P] * 9 + [_P]),
    "caat_rowpar_backward": (c_int, [_P, c_int, c_int] + [_P] * 13 + [_P, c_size_t, _P]),
    "caat_block_forward": (c_int, [_P, c_int] + [_P] * 17 + [_P, c_size_t, _P]),
    "caat_block_backward": (c_int, [_P, c_int] + [_P] * 25 + [_P, c_size_t, _P]),
    "caat_rowpar_forward_compact": (c_int, [_P, c_int, c_int] + [_P] * 11 + [_P, c_size_t, _P]),
    "caat_rowpar_backward_compact": (c_int, [_P, c_int, c_int] + [_P] * 16 + [_P, c_size_t, _P]),
    "caat_block_forward_compact": (c_int, [_P, c_int] + [_P] * 20 + [_P, c_size_t, _P]),
    "caat_block_backward_compact": (c_int, [_P, c_int] + [_P] * 30 + [_P, c_size_t, _P]),
    "caat_colpar_workspace_bytes": (c_size_t, [_P, c_int, c_int, c_int]),
    "caat_colpar_forward": (c_int, [_P, c_int, c_int, c_int] + [_P] * 4 + [_P]),
    "caat_colpar_backward": (c_int, [_P, c_int, c_int, c_int] + [_P] * 6 + [_P, c_size_t, _P]),
    "caat_tp_slab": (c_int, [_P, c_int, c_int, c_int, POINTER(c_size_t), POINTER(c_int), POINTER(c_int)]),
    "caat_tp_forward_local": (c_int, [_P, c_int, c_int] + [_P] * 2 + [_P, c_size_t, _P]),
    "caat_tp_forward_finish": (c_int, [_P, c_int, c_int] + [_P] * 7 + [_P, c_size_t, _P]),
    "caat_tp_backward_local": (c_int, [_P, c_int, c_int] + [_P] * 10 + [_P, c_size_t, _P]),
    "caat_tp_backward_finish": (c_int, [_P, c_int, c_int] + [_P] * 5 + [_P, c_size_t, _P]),
    "caat_tp_exchange_bytes": (c_int, [_P, c_int, c_int, c_int, POINTER(c_size_t), POINTER(c_int)]),
    "caat_tp_exchange_scatter": (c_int, [_P, c_int, c_int, c_int, POINTER(caat_peers), c_uint, _P, c_size_t, _P]),
    "caat_tp_exchange_reduce": (c_int, [_P, c_int, c_int, POINTER(caat_peers), c_uint, _P]),
    "caat_tp_exchange_wait": (c_int, [_P, POINTER(caat_peers), c_uint, _P]),
    "caat_tp_exchange": (c_int, [_P, c_int, c_int, c_int, POINTER(caat_peers), c_uint, _P, c_size_t, _P]),
    "caat_tp_forward_local_push": (c_int, [_P, c_int, c_int, _P, _P, POINTER(caat_peers), c_uint, _P, c_size_t, _P]),
    "caat_tp_backward_local_push": (c_int, [_P, c_int, c_int] + [_P] * 10 + [POINTER(caat_peers), c_uint, _P, c_size_t, _P]),
    "caat_allreduce_bytes": (c_int, [_P, c_int, c_int] + [POINTER(c_ulonglong)] * 3),
    "caat_last_device_status": (c_int, [_P, _P]),
    "caat_kernel_launches": (c_ulonglong, []),
    "caat_profile_begin": (c_int, [c_int]),
    "caat_profile_end": (c_int, [c_int, POINTER(c_double), POINTER(c_ulonglong)]),
    "caat_kernel_kind_name": (c_char_p, [c_int]),
}
for _name, (_res, _args) in _sigs.items():
    _f = getattr(lib, _name)
    _f.restype = _res
    _f.argtypes = _args
EXPORTED = tuple(_sigs)


class CaatError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib.caat_strerror(status).decode()
        if status == CAAT_ECUDA:
            msg += ": " + lib.caat_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} (status {status})")


def _check(status: int, where: str):
    if status != CAAT_OK:
        raise CaatError(status, where)


def _dtype_code(dtype) -> int:
    if dtype == "bf16" or dtype is torch.bfloat16:
        return CAAT_BF16
    if dtype == "f32" or dtype is torch.float32:
        return CAAT_F32
    raise ValueError(f"unsupported dtype {dtype!r}")


def _ptr(x, dtype=None, shape=None, name="tensor"):
    """Device pointer of a contiguous CUDA tensor (None -> NULL), with shape/dtype checks."""
    if x is None:
        return None
    if not isinstance(x, torch.Tensor) or not x.is_cuda:
        raise TypeError(f"{name}: expected a CUDA tensor (the library has no host path)")
    if not x.is_contiguous():
        raise ValueError(f"{name}: must be contiguous")
    if dtype is not None and x.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {x.dtype}")
    if shape is not None and tuple(x.shape) != tuple(shape):
        raise ValueError(f"{name}: expected shape {tuple(shape)}, got {tuple(x.shape)}")
    if x.numel() == 0:
        return None
    return x.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


class Context:
    """Owns a ``caat_ctx``.  Methods carry the names of the C entry points without the prefix."""

    def __init__(self, h: int, ffn: int, t: int, p: float, dtype="bf16"):
        self._h = c_void_p()
        self.h, self.ffn, self.t, self.p = h, ffn, t, p
        self.dtype_code = _dtype_code(dtype)
        self.torch_dtype = torch.bfloat16 if self.dtype_code == CAAT_BF16 else torch.float32
        self.norm = RMSNORM
        self.groups = 1
        _check(lib.caat_create(h, ffn, t, float(p), self.dtype_code, byref(self._h)), "caat_create")

    def __del__(self):
        # at interpreter shutdown the module globals may already be gone
        if getattr(self, "_h", None) is not None and self._h.value and lib is not None:
            lib.caat_destroy(self._h)
            self._h = c_void_p()

    # ---- options / queries
    def set_option(self, opt: int, value: float):
        _check(lib.caat_set_option(self._h, opt, float(value)), "caat_set_option")
        if opt == CAAT_OPT_NORM:
            self.norm = int(value)
        if opt == CAAT_OPT_TP_GROUPS:
            self.groups = int(value)
        return self

    @property
    def shared_channels(self) -> int:
        return lib.caat_shared_channels(self._h)

    @property
    def private_scale(self) -> float:
        return lib.caat_private_scale(self._h)

    def k_r(self, layer: int) -> int:
        return (self.h if layer == CAAT_ATTN_OUT else self.ffn) // (self.t * self.groups)

    def workspace_bytes(self, layer: int, tokens: int, backward: bool) -> int:
        return lib.caat_workspace_bytes(self._h, layer, tokens, 1 if backward else 0)

    def block_workspace_bytes(self, tokens: int, backward: bool) -> int:
        return lib.caat_block_workspace_bytes(self._h, tokens, 1 if backward else 0)

    def allreduce_bytes(self, tokens: int, elem_bytes: int = 2) -> dict:
        a, b, c = c_ulonglong(), c_ulonglong(), c_ulonglong()
        _check(lib.caat_allreduce_bytes(self._h, tokens, elem_bytes, byref(a), byref(b), byref(c)),
               "caat_allreduce_bytes")
        return {"payload_per_rank": a.value, "payload_per_rank_p1": b.value, "ring_wire_per_rank": c.value}

    def last_device_status(self) -> int:
        return lib.caat_last_device_status(self._h, _stream())

    # ---- compute: raw entry points (caller passes every buffer)
    def rowpar_forward(self, layer, tokens, Y, W, R, gamma, beta, Hn, X, rstd, mean, workspace):
        td, t, h, k = self.torch_dtype, self.t, self.h, self.k_r(layer)
        st = lib.caat_rowpar_forward(
            self._h, layer, tokens,
            _ptr(Y, td, (t, tokens, k), "Y"), _ptr(W, td, (t, h, k), "W"), _ptr(R, td, (t, tokens, h), "R"),
            _ptr(gamma, td, (h,), "gamma"), _ptr(beta, td, (h,), "beta"),
            _ptr(Hn, td, (t, tokens, h), "Hn"), _ptr(X, td, (t, tokens, h), "X"),
            _ptr(rstd, torch.float32, (t, tokens), "rstd"), _ptr(mean, torch.float32, (t, tokens), "mean"),
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel() if workspace is not None else 0,
            _stream())
        _check(st, "caat_rowpar_forward")

    def rowpar_forward_noalloc(self, layer, tokens, Y, W, R, gamma, beta, Hn, X, rstd, mean):
        """caat_rowpar_forward without a caller workspace: for callers that cannot allocate device
        memory when the layer runs.  Scratch is the library's built-in array (32 MiB); larger
        problems raise CaatError(CAAT_ELIMIT).  Calls on one device must not overlap on the GPU."""
        td, t, h, k = self.torch_dtype, self.t, self.h, self.k_r(layer)
        st = lib.caat_rowpar_forward_noalloc(
            self._h, layer, tokens,
            _ptr(Y, td, (t, tokens, k), "Y"), _ptr(W, td, (t, h, k), "W"), _ptr(R, td, (t, tokens, h), "R"),
            _ptr(gamma, td, (h,), "gamma"), _ptr(beta, td, (h,), "beta"),
            _ptr(Hn, td, (t, tokens, h), "Hn"), _ptr(X, td, (t, tokens, h), "X"),
            _ptr(rstd, torch.float32, (t, tokens), "rstd"), _ptr(mean, torch.float32, (t, tokens), "mean"),
            _stream())
        _check(st, "caat_rowpar_forward_noalloc")

    def rowpar_backward(self, layer, tokens, dX, dHn, Y, W, Hn, rstd, mean, gamma, dY, dW, dR, dgamma, dbeta,
                        workspace):
        td, t, h, k = self.torch_dtype, self.t, self.h, self.k_r(layer)
        f32 = torch.float32
        st = lib.caat_rowpar_backward(
            self._h, layer, tokens,
            _ptr(dX, td, (t, tokens, h), "dX"), _ptr(dHn, td, (t, tokens, h), "dHn"),
            _ptr(Y, td, (t, tokens, k), "Y"), _ptr(W, td, (t, h, k), "W"), _ptr(Hn, td, (t, tokens, h), "Hn"),
            _ptr(rstd, f32, (t, tokens), "rstd"), _ptr(mean, f32, (t, tokens), "mean"), _ptr(gamma, td, (h,), "gamma"),
            _ptr(dY, td, (t, tokens, k), "dY"), _ptr(dW, f32, (t, h, k), "dW"), _ptr(dR, td, (t, tokens, h), "dR"),
            _ptr(dgamma, f32, (h,), "dgamma"), _ptr(dbeta, f32, (h,), "dbeta"),
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel() if workspace is not None else 0,
            _stream())
        _check(st, "caat_rowpar_backward")

    def block_forward(self, tokens, Y_attn, W_o, Y_mlp, W_down, R0, gamma1, beta1, gamma2, beta2,
                      Hn1, X1, rstd1, mean1, Hn2, X2, rstd2, mean2, workspace):
        td, t, h = self.torch_dtype, self.t, self.h
        ka, km = self.k_r(CAAT_ATTN_OUT), self.k_r(CAAT_MLP_DOWN)
        f32 = torch.float32
        act = (t, tokens, h)
        st = lib.caat_block_forward(
            self._h, tokens,
            _ptr(Y_attn, td, (t, tokens, ka), "Y_attn"), _ptr(W_o, td, (t, h, ka), "W_o"),
            _ptr(Y_mlp, td, (t, tokens, km), "Y_mlp"), _ptr(W_down, td, (t, h, km), "W_down"),
            _ptr(R0, td, act, "R0"), _ptr(gamma1, td, (h,), "gamma1"), _ptr(beta1, td, (h,), "beta1"),
            _ptr(gamma2, td, (h,), "gamma2"), _ptr(beta2, td, (h,), "beta2"),
            _ptr(Hn1, td, act, "Hn1"), _ptr(X1, td, act, "X1"), _ptr(rstd1, f32, (t, tokens), "rstd1"),
            _ptr(mean1, f32, (t, tokens), "mean1"),
            _ptr(Hn2, td, act, "Hn2"), _ptr(X2, td, act, "X2"), _ptr(rstd2, f32, (t, tokens), "rstd2"),
            _ptr(mean2, f32, (t, tokens), "mean2"),
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel() if workspace is not None else 0,
            _stream())
        _check(st, "caat_block_forward")

    def block_backward(self, tokens, dX1, dX2, dHn2, Y_attn, W_o, Y_mlp, W_down, Hn1, rstd1, mean1, Hn2, rstd2,
                       mean2, gamma1, gamma2, dY_attn, dW_o, dY_mlp, dW_down, dR0, dHn1, dgamma1, dbeta1,
                       dgamma2, dbeta2, workspace):
        td, t, h = self.torch_dtype, self.t, self.h
        ka, km = self.k_r(CAAT_ATTN_OUT), self.k_r(CAAT_MLP_DOWN)
        f32 = torch.float32
        act = (t, tokens, h)
        st = lib.caat_block_backward(
            self._h, tokens,
            _ptr(dX1, td, act, "dX1"), _ptr(dX2, td, act, "dX2"), _ptr(dHn2, td, act, "dHn2"),
            _ptr(Y_attn, td, (t, tokens, ka), "Y_attn"), _ptr(W_o, td, (t, h, ka), "W_o"),
            _ptr(Y_mlp, td, (t, tokens, km), "Y_mlp"), _ptr(W_down, td, (t, h, km), "W_down"),
            _ptr(Hn1, td, act, "Hn1"), _ptr(rstd1, f32, (t, tokens), "rstd1"), _ptr(mean1, f32, (t, tokens), "mean1"),
            _ptr(Hn2, td, act, "Hn2"), _ptr(rstd2, f32, (t, tokens), "rstd2"), _ptr(mean2, f32, (t, tokens), "mean2"),
            _ptr(gamma1, td, (h,), "gamma1"), _ptr(gamma2, td, (h,), "gamma2"),
            _ptr(dY_attn, td, (t, tokens, ka), "dY_attn"), _ptr(dW_o, f32, (t, h, ka), "dW_o"),
            _ptr(dY_mlp, td, (t, tokens, km), "dY_mlp"), _ptr(dW_down, f32, (t, h, km), "dW_down"),
            _ptr(dR0, td, act, "dR0"), _ptr(dHn1, td, act, "dHn1"),
            _ptr(dgamma1, f32, (h,), "dgamma1"), _ptr(dbeta1, f32, (h,), "dbeta1"),
            _ptr(dgamma2, f32, (h,), "dgamma2"), _ptr(dbeta2, f32, (h,), "dbeta2"),
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel() if workspace is not None else 0,
            _stream())
        _check(st, "caat_block_backward")

    # ---- compact residual layout: shared part [T, S] once, private parts [t, T, h - S]
    def rowpar_forward_compact(self, layer, tokens, Y, W, Rs, Rp, gamma, beta, Hns, Hnp, X, rstd, mean, workspace):
        td, t, h, k, S = self.torch_dtype, self.t, self.h, self.k_r(layer), self.shared_channels
        sh, pr, f32 = (tokens, S), (t, tokens, h - S), torch.float32
        st = lib.caat_rowpar_forward_compact(
            self._h, layer, tokens,
            _ptr(Y, td, (t, tokens, k), "Y"), _ptr(W, td, (t, h, k), "W"), _ptr(Rs, td, sh, "Rs"), _ptr(Rp, td, pr, "Rp"),
            _ptr(gamma, td, (h,), "gamma"), _ptr(beta, td, (h,), "beta"),
            _ptr(Hns, td, sh, "Hns"), _ptr(Hnp, td, pr, "Hnp"), _ptr(X, td, (t, tokens, h), "X"),
            _ptr(rstd, f32, (t, tokens), "rstd"), _ptr(mean, f32, (t, tokens), "mean"),
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel() if workspace is not None else 0,
            _stream())
        _check(st, "caat_rowpar_forward_compact")

    def rowpar_backward_compact(self, layer, tokens, dX, dHns, dHnp, Y, W, Hns, Hnp, rstd, mean, gamma, dY, dW,
                                dRs, dRp, dgamma, dbeta, workspace):
        td, t, h, k, S = self.torch_dtype, self.t, self.h, self.k_r(layer), self.shared_channels
        sh, pr, f32 = (tokens, S), (t, tokens, h - S), torch.float32
        st = lib.caat_rowpar_backward_compact(
            self._h, layer, tokens,
            _ptr(dX, td, (t, tokens, h), "dX"), _ptr(dHns, td, sh, "dHns"), _ptr(dHnp, td, pr, "dHnp"),
            _ptr(Y, td, (t, tokens, k), "Y"), _ptr(W, td, (t, h, k), "W"),
            _ptr(Hns, td, sh, "Hns"), _ptr(Hnp, td, pr, "Hnp"),
            _ptr(rstd, f32, (t, tokens), "rstd"), _ptr(mean, f32, (t, tokens), "mean"), _ptr(gamma, td, (h,), "gamma"),
            _ptr(dY, td, (t, tokens, k), "dY"), _ptr(dW, f32, (t, h, k), "dW"),
            _ptr(dRs, td, sh, "dRs"), _ptr(dRp, td, pr, "dRp"),
            _ptr(dgamma, f32, (h,), "dgamma"), _ptr(dbeta, f32, (h,), "dbeta"),
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel() if workspace is not None else 0,
            _stream())
        _check(st, "caat_rowpar_backward_compact")

    def block_forward_compact(self, tokens, Y_attn, W_o, Y_mlp, W_down, R0s, R0p, gamma1, beta1, gamma2, beta2,
                              Hn1s, Hn1p, X1, rstd1, mean1, Hn2s, Hn2p, X2, rstd2, mean2, workspace):
        td, t, h, S = self.torch_dtype, self.t, self.h, self.shared_channels
        ka, km = self.k_r(CAAT_ATTN_OUT), self.k_r(CAAT_MLP_DOWN)
        sh, pr, act, st2, f32 = (tokens, S), (t, tokens, h - S), (t, tokens, h), (t, tokens), torch.float32
        st = lib.caat_block_forward_compact(
            self._h, tokens,
            _ptr(Y_attn, td, (t, tokens, ka), "Y_attn"), _ptr(W_o, td, (t, h, ka), "W_o"),
            _ptr(Y_mlp, td, (t, tokens, km), "Y_mlp"), _ptr(W_down, td, (t, h, km), "W_down"),
            _ptr(R0s, td, sh, "R0s"), _ptr(R0p, td, pr, "R0p"),
            _ptr(gamma1, td, (h,), "gamma1"), _ptr(beta1, td, (h,), "beta1"),
            _ptr(gamma2, td, (h,), "gamma2"), _ptr(beta2, td, (h,), "beta2"),
            _ptr(Hn1s, td, sh, "Hn1s"), _ptr(Hn1p, td, pr, "Hn1p"), _ptr(X1, td, act, "X1"),
            _ptr(rstd1, f32, st2, "rstd1"), _ptr(mean1, f32, st2, "mean1"),
            _ptr(Hn2s, td, sh, "Hn2s"), _ptr(Hn2p, td, pr, "Hn2p"), _ptr(X2, td, act, "X2"),
            _ptr(rstd2, f32, st2, "rstd2"), _ptr(mean2, f32, st2, "mean2"),
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel() if workspace is not None else 0,
            _stream())
        _check(st, "caat_block_forward_compact")

    def block_backward_compact(self, tokens, dX1, dX2, dHn2s, dHn2p, Y_attn, W_o, Y_mlp, W_down, Hn1s, Hn1p, rstd1,
                               mean1, Hn2s, Hn2p, rstd2, mean2, gamma1, gamma2, dY_attn, dW_o, dY_mlp, dW_down,
                               dR0s, dR0p, dHn1s, dHn1p, dgamma1, dbeta1, dgamma2, dbeta2, workspace):
        td, t, h, S = self.torch_dtype, self.t, self.h, self.shared_channels
        ka, km = self.k_r(CAAT_ATTN_OUT), self.k_r(CAAT_MLP_DOWN)
        sh, pr, act, st2, f32 = (tokens, S), (t, tokens, h - S), (t, tokens, h), (t, tokens), torch.float32
        st = lib.caat_block_backward_compact(
            self._h, tokens,
            _ptr(dX1, td, act, "dX1"), _ptr(dX2, td, act, "dX2"), _ptr(dHn2s, td, sh, "dHn2s"), _ptr(dHn2p, td, pr, "dHn2p"),
            _ptr(Y_attn, td, (t, tokens, ka), "Y_attn"), _ptr(W_o, td, (t, h, ka), "W_o"),
            _ptr(Y_mlp, td, (t, tokens, km), "Y_mlp"), _ptr(W_down, td, (t, h, km), "W_down"),
            _ptr(Hn1s, td, sh, "Hn1s"), _ptr(Hn1p, td, pr, "Hn1p"), _ptr(rstd1, f32, st2, "rstd1"), _ptr(mean1, f32, st2, "mean1"),
            _ptr(Hn2s, td, sh, "Hn2s"), _ptr(Hn2p, td, pr, "Hn2p"), _ptr(rstd2, f32, st2, "rstd2"), _ptr(mean2, f32, st2, "mean2"),
            _ptr(gamma1, td, (h,), "gamma1"), _ptr(gamma2, td, (h,), "gamma2"),
            _ptr(dY_attn, td, (t, tokens, ka), "dY_attn"), _ptr(dW_o, f32, (t, h, ka), "dW_o"),
            _ptr(dY_mlp, td, (t, tokens, km), "dY_mlp"), _ptr(dW_down, f32, (t, h, km), "dW_down"),
            _ptr(dR0s, td, sh, "dR0s"), _ptr(dR0p, td, pr, "dR0p"), _ptr(dHn1s, td, sh, "dHn1s"), _ptr(dHn1p, td, pr, "dHn1p"),
            _ptr(dgamma1, f32, (h,), "dgamma1"), _ptr(dbeta1, f32, (h,), "dbeta1"),
            _ptr(dgamma2, f32, (h,), "dgamma2"), _ptr(dbeta2, f32, (h,), "dbeta2"),
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel() if workspace is not None else 0,
            _stream())
        _check(st, "caat_block_backward_compact")

    # ---- column-parallel half: pre = X A^T per rank, Y = act(pre)
    def colpar_workspace_bytes(self, act: int, n_out: int, tokens: int) -> int:
        return int(lib.caat_colpar_workspace_bytes(self._h, act, n_out, tokens))

    def colpar_forward(self, act, n_out, tokens, X, A, pre, Y):
        td, t, h = self.torch_dtype, self.t, self.h
        wy = n_out // 2 if act == CAAT_ACT_SWIGLU else n_out
        st = lib.caat_colpar_forward(
            self._h, act, n_out, tokens,
            _ptr(X, td, (t, tokens, h), "X"), _ptr(A, td, (t, n_out, h), "A"), _ptr(pre, td, (t, tokens, n_out), "pre"),
            _ptr(Y, td, (t, tokens, wy), "Y"), _stream())
        _check(st, "caat_colpar_forward")

    def colpar_backward(self, act, n_out, tokens, dY, X, A, pre, dX, dA, workspace):
        td, t, h = self.torch_dtype, self.t, self.h
        wy = n_out // 2 if act == CAAT_ACT_SWIGLU else n_out
        st = lib.caat_colpar_backward(
            self._h, act, n_out, tokens,
            _ptr(dY, td, (t, tokens, wy), "dY"), _ptr(X, td, (t, tokens, h), "X"), _ptr(A, td, (t, n_out, h), "A"),
            _ptr(pre, td, (t, tokens, n_out), "pre"), _ptr(dX, td, (t, tokens, h), "dX"),
            _ptr(dA, torch.float32, (t, n_out, h), "dA"),
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel() if workspace is not None else 0,
            _stream())
        _check(st, "caat_colpar_backward")

    # ---- real tensor parallelism: the halves of a layer call around the caller's all-reduce
    def tp_slab(self, layer, tokens, backward, workspace):
        """The [tokens, S] slab of `workspace` that the caller all-reduces between the two halves (a view)."""
        off, rows, cols = c_size_t(), c_int(), c_int()
        _check(lib.caat_tp_slab(self._h, layer, tokens, 1 if backward else 0, byref(off), byref(rows), byref(cols)),
               "caat_tp_slab")
        es = 2 if self.dtype_code == CAAT_BF16 else 4
        nbytes = rows.value * cols.value * es
        return workspace[off.value:off.value + nbytes].view(self.torch_dtype).view(rows.value, cols.value)

    def tp_forward_local(self, layer, tokens, Y, W, workspace):
        td, t, h, k = self.torch_dtype, self.t, self.h, self.k_r(layer)
        _check(lib.caat_tp_forward_local(
            self._h, layer, tokens, _ptr(Y, td, (t, tokens, k), "Y"), _ptr(W, td, (t, h, k), "W"),
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel(), _stream()), "caat_tp_forward_local")

    def tp_forward_finish(self, layer, tokens, R, gamma, beta, Hn, X, rstd, mean, workspace):
        td, t, h = self.torch_dtype, self.t, self.h
        _check(lib.caat_tp_forward_finish(
            self._h, layer, tokens, _ptr(R, td, (t, tokens, h), "R"), _ptr(gamma, td, (h,), "gamma"),
            _ptr(beta, td, (h,), "beta"), _ptr(Hn, td, (t, tokens, h), "Hn"), _ptr(X, td, (t, tokens, h), "X"),
            _ptr(rstd, torch.float32, (t, tokens), "rstd"), _ptr(mean, torch.float32, (t, tokens), "mean"),
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel(), _stream()), "caat_tp_forward_finish")

    def tp_backward_local(self, layer, tokens, dX, dHn, W, Hn, rstd, mean, gamma, dR, dgamma, dbeta, workspace):
        td, t, h, k = self.torch_dtype, self.t, self.h, self.k_r(layer)
        f32 = torch.float32
        _check(lib.caat_tp_backward_local(
            self._h, layer, tokens, _ptr(dX, td, (t, tokens, h), "dX"), _ptr(dHn, td, (t, tokens, h), "dHn"),
            _ptr(W, td, (t, h, k), "W"), _ptr(Hn, td, (t, tokens, h), "Hn"), _ptr(rstd, f32, (t, tokens), "rstd"),
            _ptr(mean, f32, (t, tokens), "mean"), _ptr(gamma, td, (h,), "gamma"), _ptr(dR, td, (t, tokens, h), "dR"),
            _ptr(dgamma, f32, (h,), "dgamma"), _ptr(dbeta, f32, (h,), "dbeta"),
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel(), _stream()), "caat_tp_backward_local")

    def tp_backward_finish(self, layer, tokens, Y, W, dR, dY, dW, workspace):
        td, t, h, k = self.torch_dtype, self.t, self.h, self.k_r(layer)
        _check(lib.caat_tp_backward_finish(
            self._h, layer, tokens, _ptr(Y, td, (t, tokens, k), "Y"), _ptr(W, td, (t, h, k), "W"),
            _ptr(dR, td, (t, tokens, h), "dR"), _ptr(dY, td, (t, tokens, k), "dY"),
            _ptr(dW, torch.float32, (t, h, k), "dW"),
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel(), _stream()), "caat_tp_backward_finish")

    # ---- the slab exchange over peer memory (the library's own kernels instead of a collective)
    def tp_exchange_bytes(self, layer, tokens, world):
        """(bytes of one GPU's receive buffer, tokens per owner)."""
        n, sl = c_size_t(), c_int()
        _check(lib.caat_tp_exchange_bytes(self._h, layer, tokens, world, byref(n), byref(sl)), "caat_tp_exchange_bytes")
        return n.value, sl.value

    @staticmethod
    def make_peers(rank, recv_ptrs, slab_ptrs, flag_ptrs):
        """caat_peers from device addresses (ints), one per GPU of the group, as THIS GPU addresses them."""
        pe = caat_peers()
        pe.world, pe.rank = len(flag_ptrs), rank
        for q in range(pe.world):
            pe.recv[q] = recv_ptrs[q] if recv_ptrs else None
            pe.slab[q] = slab_ptrs[q] if slab_ptrs else None
            pe.flags[q] = flag_ptrs[q]
        return pe

    def tp_exchange_scatter(self, layer, tokens, backward, peers, epoch, workspace):
        _check(lib.caat_tp_exchange_scatter(self._h, layer, tokens, 1 if backward else 0, byref(peers), epoch,
                                            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel(), _stream()),
               "caat_tp_exchange_scatter")

    def tp_exchange_reduce(self, layer, tokens, peers, epoch):
        _check(lib.caat_tp_exchange_reduce(self._h, layer, tokens, byref(peers), epoch, _stream()), "caat_tp_exchange_reduce")

    def tp_exchange_wait(self, peers, epoch):
        _check(lib.caat_tp_exchange_wait(self._h, byref(peers), epoch, _stream()), "caat_tp_exchange_wait")

    def tp_exchange(self, layer, tokens, backward, peers, epoch, workspace):
        _check(lib.caat_tp_exchange(self._h, layer, tokens, 1 if backward else 0, byref(peers), epoch,
                                    _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel(), _stream()),
               "caat_tp_exchange")

    def tp_forward_local_push(self, layer, tokens, Y, W, peers, epoch, workspace):
        td, t, h, k = self.torch_dtype, self.t, self.h, self.k_r(layer)
        _check(lib.caat_tp_forward_local_push(
            self._h, layer, tokens, _ptr(Y, td, (t, tokens, k), "Y"), _ptr(W, td, (t, h, k), "W"), byref(peers), epoch,
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel(), _stream()), "caat_tp_forward_local_push")

    def tp_backward_local_push(self, layer, tokens, dX, dHn, W, Hn, rstd, mean, gamma, dR, dgamma, dbeta, peers, epoch,
                               workspace):
        td, t, h, k = self.torch_dtype, self.t, self.h, self.k_r(layer)
        f32 = torch.float32
        _check(lib.caat_tp_backward_local_push(
            self._h, layer, tokens, _ptr(dX, td, (t, tokens, h), "dX"), _ptr(dHn, td, (t, tokens, h), "dHn"),
            _ptr(W, td, (t, h, k), "W"), _ptr(Hn, td, (t, tokens, h), "Hn"), _ptr(rstd, f32, (t, tokens), "rstd"),
            _ptr(mean, f32, (t, tokens), "mean"), _ptr(gamma, td, (h,), "gamma"), _ptr(dR, td, (t, tokens, h), "dR"),
            _ptr(dgamma, f32, (h,), "dgamma"), _ptr(dbeta, f32, (h,), "dbeta"), byref(peers), epoch,
            _ptr(workspace, torch.uint8, None, "workspace"), workspace.numel(), _stream()), "caat_tp_backward_local_push")

    # ---- buffer helpers (torch.empty only; no arithmetic)
    def alloc_workspace(self, nbytes: int, device="cuda"):
        return torch.empty(max(int(nbytes), 16), dtype=torch.uint8, device=device)

    def alloc_forward_outputs(self, tokens: int, device="cuda") -> dict:
        td, t, h = self.torch_dtype, self.t, self.h
        out = {"Hn": torch.empty((t, tokens, h), dtype=td, device=device),
               "X": torch.empty((t, tokens, h), dtype=td, device=device),
               "rstd": torch.empty((t, tokens), dtype=torch.float32, device=device),
               "mean": torch.empty((t, tokens), dtype=torch.float32, device=device) if self.norm == LAYERNORM else None}
        return out

    def alloc_backward_outputs(self, layer: int, tokens: int, device="cuda") -> dict:
        td, t, h, k = self.torch_dtype, self.t, self.h, self.k_r(layer)
        return {"dY": torch.empty((t, tokens, k), dtype=td, device=device),
                "dW": torch.empty((t, h, k), dtype=torch.float32, device=device),
                "dR": torch.empty((t, tokens, h), dtype=td, device=device),
                "dgamma": torch.empty((h,), dtype=torch.float32, device=device),
                "dbeta": torch.empty((h,), dtype=torch.float32, device=device) if self.norm == LAYERNORM else None}


def kernel_launches() -> int:
    return int(lib.caat_kernel_launches())


CAAT_K_COUNT = 10


def profile_begin(max_launches: int = 65536):
    _check(lib.caat_profile_begin(max_launches), "caat_profile_begin")


def profile_end() -> dict:
    """{kernel kind name: (milliseconds, timed launches)} for the kinds that ran."""
    ms = (c_double * CAAT_K_COUNT)()
    n = (c_ulonglong * CAAT_K_COUNT)()
    _check(lib.caat_profile_end(CAAT_K_COUNT, ms, n), "caat_profile_end")
    return {lib.caat_kernel_kind_name(k).decode(): (ms[k], int(n[k])) for k in range(CAAT_K_COUNT) if n[k]}
