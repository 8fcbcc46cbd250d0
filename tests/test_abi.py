"""Host-side checks of the C ABI: the library loads, exports every declared symbol, and
rejects bad arguments before any launch.  No GPU needed: no compute call reaches a kernel."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def caat():
    from paper_2506_19645_b200 import build
    build.build()
    from paper_2506_19645_b200 import caat as m
    return m


def test_exports_every_declared_symbol(caat):
    header = open(os.path.join(ROOT, "include", "caat.h")).read()
    declared = set(re.findall(r"\b(caat_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(caat.lib, name), f"libcaat.so does not export {name}"
    assert declared == set(caat.EXPORTED), declared ^ set(caat.EXPORTED)


def test_create_validation_and_partition(caat):
    h = ctypes.c_void_p()
    assert caat.lib.caat_create(768, 3072, 4, 0.5, caat.CAAT_BF16, ctypes.byref(h)) == caat.CAAT_OK
    assert caat.lib.caat_shared_channels(h) == 384
    assert caat.lib.caat_private_scale(h) == pytest.approx(2.0)
    caat.lib.caat_destroy(h)
    assert caat.lib.caat_create(768, 3072, 5, 0.5, caat.CAAT_BF16, ctypes.byref(h)) == caat.CAAT_ESHAPE
    assert caat.lib.caat_create(768, 3072, 4, 1.5, caat.CAAT_BF16, ctypes.byref(h)) == caat.CAAT_EINVAL
    assert caat.lib.caat_create(768, 3072, 4, 0.5, 7, ctypes.byref(h)) == caat.CAAT_EINVAL
    assert caat.lib.caat_create(768, 3072, 4, 0.5, caat.CAAT_BF16, None) == caat.CAAT_EINVAL
    assert caat.lib.caat_shared_channels(None) == -1
    for hh, p, S in [(256, 0.5, 128), (2048, 0.75, 1536), (2048, 0.25, 512), (4096, 1.0, 4096), (4096, 0.0, 0),
                     (10, 0.35, 3), (4096, 0.703125, 2880), (4096, 0.7, 2867)]:
        c = caat.Context(hh, 4 * hh, 2, p, "bf16")
        assert c.shared_channels == S      # floor(h p), Eq. A3


def test_options(caat):
    c = caat.Context(512, 2048, 8, 0.5, "bf16")
    assert c.private_scale == pytest.approx(8 ** 0.5)
    c.set_option(caat.CAAT_OPT_PRIVATE_SCALE, 1.0)
    assert c.private_scale == 1.0
    c.set_option(caat.CAAT_OPT_SHARED_CHANNELS, 100)
    assert c.shared_channels == 100
    with pytest.raises(caat.CaatError) as e:
        c.set_option(caat.CAAT_OPT_SHARED_CHANNELS, 513)
    assert e.value.status == caat.CAAT_ESHAPE
    with pytest.raises(caat.CaatError):
        c.set_option(caat.CAAT_OPT_NORM, 2)
    with pytest.raises(caat.CaatError):
        c.set_option(99, 0)
    assert caat.lib.caat_strerror(caat.CAAT_EWORKSPACE).decode().startswith("workspace")


def test_workspace_and_argument_errors_before_launch(caat):
    c = caat.Context(768, 3072, 4, 0.5, "bf16")
    T = 256        # above the few-token (decode) threshold, whose forward scratch holds fp32 planes
    need = c.workspace_bytes(caat.CAAT_MLP_DOWN, T, False)
    assert need >= T * 384 * 2 + 4 * T * 384 * 2
    assert c.workspace_bytes(caat.CAAT_MLP_DOWN, T, True) > need
    assert c.workspace_bytes(caat.CAAT_MLP_DOWN, 0, False) == 0
    fake = 0x10000  # never dereferenced: validation fails first
    f = caat.lib.caat_rowpar_forward
    args = [c._h, caat.CAAT_MLP_DOWN, T] + [fake] * 9
    assert f(*args[:3], None, *args[4:], fake, need, None) == caat.CAAT_EINVAL
    assert f(*args, fake, need - 1, None) == caat.CAAT_EWORKSPACE
    assert f(*args, None, need, None) == caat.CAAT_EWORKSPACE
    bad = list(args); bad[5] = fake + 2
    assert f(*bad, fake, need, None) == caat.CAAT_EALIGN
    assert f(c._h, 5, T, *args[3:], fake, need, None) == caat.CAAT_EINVAL
    assert f(c._h, caat.CAAT_MLP_DOWN, 0, *args[3:], fake, need, None) == caat.CAAT_ESHAPE
    odd = caat.Context(36, 72, 2, 0.5, "bf16")     # h not a multiple of 8
    assert caat.lib.caat_rowpar_forward(odd._h, 0, T, *([fake] * 9), fake, 1 << 20, None) == caat.CAAT_EUNSUPPORTED
    ln = caat.Context(768, 3072, 4, 0.5, "bf16").set_option(caat.CAAT_OPT_NORM, 1)
    a2 = [ln._h, caat.CAAT_MLP_DOWN, T] + [fake] * 8 + [None]      # mean missing under LayerNorm
    assert f(*a2, fake, need, None) == caat.CAAT_EINVAL
    b = caat.lib.caat_rowpar_backward
    bargs = [c._h, caat.CAAT_MLP_DOWN, T] + [fake] * 13
    assert b(*bargs, fake, 16, None) == caat.CAAT_EWORKSPACE
    bargs2 = list(bargs); bargs2[3] = None
    assert b(*bargs2, fake, 1 << 30, None) == caat.CAAT_EINVAL


def test_binding_refuses_host_tensors(caat):
    import torch
    c = caat.Context(256, 1024, 2, 0.5, "f32")
    x = torch.zeros(2, 4, 512)
    with pytest.raises(TypeError):
        c.rowpar_forward(caat.CAAT_MLP_DOWN, 4, x, x, x, x, None, x, x, x, None, x)


def test_allreduce_bytes_matches_closed_form(caat):
    # Appendix C: tokens*h*p activations per device per reduce; Appendix D: cut by 100(1-p) %.
    c = caat.Context(4096, 11008, 8, 0.5, "bf16")
    a = c.allreduce_bytes(16384, 2)
    assert a["payload_per_rank"] == 16384 * 2048 * 2 == 67108864
    assert a["payload_per_rank_p1"] == 16384 * 4096 * 2
    assert a["ring_wire_per_rank"] == 2 * 7 * 67108864 // 8
    from oracle import caat_oracle as O
    o = O.allreduce_bytes(16384, 4096, 8, 2048, 2)
    assert o["payload_per_rank"] == a["payload_per_rank"] and o["ring_wire_per_rank"] == a["ring_wire_per_rank"]


def test_tensor_parallel_groups_and_slab(caat):
    # CAAT_OPT_TP_GROUPS: this context holds t of t*G ranks; K_r and alpha follow; the slab is the dense [T, S] block
    ctx = caat.Context(4096, 11008, 1, 0.5, "bf16")
    ctx.set_option(caat.CAAT_OPT_TP_GROUPS, 8)
    assert ctx.k_r(caat.CAAT_ATTN_OUT) == 512 and ctx.k_r(caat.CAAT_MLP_DOWN) == 1376
    assert ctx.private_scale == pytest.approx(8 ** 0.5)
    with pytest.raises(caat.CaatError) as e:
        ctx.set_option(caat.CAAT_OPT_TP_GROUPS, 3)              # 3 does not divide h
    assert e.value.status == caat.CAAT_ESHAPE
    with pytest.raises(caat.CaatError):
        ctx.set_option(caat.CAAT_OPT_TP_GROUPS, 0)
    off, rows, cols = ctypes.c_size_t(), ctypes.c_int(), ctypes.c_int()
    for backward in (0, 1):
        st = caat.lib.caat_tp_slab(ctx._h, caat.CAAT_MLP_DOWN, 300, backward, ctypes.byref(off), ctypes.byref(rows),
                                   ctypes.byref(cols))
        assert st == caat.CAAT_OK and (rows.value, cols.value) == (300, 2048) and off.value % 16 == 0
        assert off.value + 300 * 2048 * 2 <= ctx.workspace_bytes(caat.CAAT_MLP_DOWN, 300, True)
    # analytic ring bytes count the GPUs of the group
    ar = ctx.allreduce_bytes(300, 2)
    assert ar["payload_per_rank"] == 300 * 2048 * 2 and ar["ring_wire_per_rank"] == 2 * 7 * ar["payload_per_rank"] // 8
    # no packed slab off the tensor-core path: fp32, or a partition that is not a multiple of 8
    c32 = caat.Context(256, 1024, 2, 0.5, "f32")
    assert caat.lib.caat_tp_slab(c32._h, caat.CAAT_MLP_DOWN, 64, 0, None, None, None) == caat.CAAT_EUNSUPPORTED
    odd = caat.Context(4096, 11008, 8, 0.5, "bf16").set_option(caat.CAAT_OPT_SHARED_CHANNELS, 100)
    assert caat.lib.caat_tp_slab(odd._h, caat.CAAT_MLP_DOWN, 64, 0, None, None, None) == caat.CAAT_EUNSUPPORTED
    # the halves reject a missing workspace before any launch
    assert caat.lib.caat_tp_forward_local(ctx._h, caat.CAAT_MLP_DOWN, 300, None, None, None, 0, None) == caat.CAAT_EWORKSPACE


def test_block_workspace_and_schedule_option(caat):
    # the block calls' scratch: both layers' forward regions side by side, never less than one layer's full need
    ctx = caat.Context(2048, 5632, 8, 0.5, "bf16")
    A, M = caat.CAAT_ATTN_OUT, caat.CAAT_MLP_DOWN
    for T in (300, 16384):
        for backward in (False, True):
            one = max(ctx.workspace_bytes(A, T, backward), ctx.workspace_bytes(M, T, backward))
            both = ctx.block_workspace_bytes(T, backward)
            assert both >= one
            assert both >= ctx.workspace_bytes(A, T, False) + ctx.workspace_bytes(M, T, False)
    assert caat.lib.caat_block_workspace_bytes(None, 16, 0) == 0
    assert caat.lib.caat_block_workspace_bytes(ctx._h, 0, 0) == 0
    for v in (0, 1, 2):
        ctx.set_option(caat.CAAT_OPT_BLOCK_OVERLAP, v)
    with pytest.raises(caat.CaatError) as e:
        ctx.set_option(caat.CAAT_OPT_BLOCK_OVERLAP, 3)
    assert e.value.status == caat.CAAT_EINVAL


def test_exchange_geometry_and_argument_errors(caat):
    # the slab exchange over peer memory: slices of tokens per owner, receive-buffer size, arguments checked on the host
    ctx = caat.Context(4096, 11008, 1, 0.5, "bf16")
    ctx.set_option(caat.CAAT_OPT_TP_GROUPS, 8)
    M = caat.CAAT_MLP_DOWN
    assert ctx.tp_exchange_bytes(M, 16384, 8) == (8 * 2048 * 2048 * 2, 2048)       # [world][slice][S] 16-bit
    assert ctx.tp_exchange_bytes(M, 1000, 4)[1] == 256                              # ceil(1000/4) = 250 -> 8-row units
    assert ctx.tp_exchange_bytes(M, 4097, 2)[1] == 2304                             # 2049 -> whole 256-row pair tiles
    assert ctx.tp_exchange_bytes(M, 130, 8)[1] == 24
    n = ctypes.c_size_t()
    assert caat.lib.caat_tp_exchange_bytes(ctx._h, M, 64, 9, ctypes.byref(n), None) == caat.CAAT_EINVAL      # > CAAT_MAX_PEERS
    assert caat.lib.caat_tp_exchange_bytes(ctx._h, M, 0, 2, ctypes.byref(n), None) == caat.CAAT_ESHAPE
    c32 = caat.Context(256, 1024, 2, 0.5, "f32")
    assert caat.lib.caat_tp_exchange_bytes(c32._h, M, 64, 2, ctypes.byref(n), None) == caat.CAAT_EUNSUPPORTED
    pe = caat.caat_peers()
    pe.world, pe.rank = 2, 2                                                        # rank outside the group
    assert caat.lib.caat_tp_exchange_wait(ctx._h, ctypes.byref(pe), 1, None) == caat.CAAT_EINVAL
    pe.rank = 0                                                                     # no flag words given
    assert caat.lib.caat_tp_exchange_wait(ctx._h, ctypes.byref(pe), 1, None) == caat.CAAT_EINVAL
    pe.flags[0] = pe.flags[1] = 0x1008                                              # not 16-byte aligned
    assert caat.lib.caat_tp_exchange_wait(ctx._h, ctypes.byref(pe), 1, None) == caat.CAAT_EALIGN
    assert caat.lib.caat_tp_exchange_reduce(ctx._h, M, 64, None, 1, None) == caat.CAAT_EINVAL
    assert ctypes.sizeof(caat.caat_peers) == 8 + 3 * 8 * caat.CAAT_MAX_PEERS         # the C struct's layout
