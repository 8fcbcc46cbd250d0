"""Pins for the fp64 oracle: every check here compares the oracle with something other than
itself - a hand-worked closed form, a brute-force index-notation evaluation, a library
routine on a special case, an invariant, finite differences or a closed form of the paper.
CPU only."""
import itertools
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import caat_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def _rand_layer(rng, t, T, h, K_r, backward=False):
    d = {"Y": rng.standard_normal((t, T, K_r)), "W": rng.standard_normal((t, h, K_r)) * 0.3,
         "R": rng.standard_normal((t, T, h)), "gamma": 1.0 + 0.2 * rng.standard_normal(h),
         "beta": 0.1 * rng.standard_normal(h)}
    if backward:
        d["dX"] = rng.standard_normal((t, T, h))
        d["dHn"] = rng.standard_normal((t, T, h))
    return d


# ---------------------------------------------------------------- F0 partition
def test_partition_floor_hp():
    # Eq. A3: shared channels are l < floor(h p).
    assert O.shared_channels(256, 0.5) == 128
    assert O.shared_channels(768, 0.5) == 384
    assert [O.shared_channels(2048, p) for p in (1.0, 0.75, 0.5, 0.25)] == [2048, 1536, 1024, 512]
    assert O.shared_channels(4096, 0.5) == 2048
    assert O.shared_channels(4096, 0.0) == 0
    assert O.shared_channels(4096, 1.0) == 4096
    assert O.shared_channels(10, 0.35) == 3       # floor, not round
    assert O.shared_channels(4096, 90 * 2.0 ** -7) == 2880   # the p = 90 * 2^-7 example of Section 5
    with pytest.raises(ValueError):
        O.shared_channels(8, 1.5)


def test_private_scale_is_sqrt_t():
    assert O.private_scale(2) == pytest.approx(math.sqrt(2.0))
    assert O.private_scale(8) == pytest.approx(math.sqrt(8.0))
    assert O.private_scale(8, enabled=False) == 1.0


# ---------------------------------------------------------------- forward: closed forms
def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split("=")
            out[k.strip()] = np.array([float(x) for x in v.split()])
    return out


def test_two_device_worked_example():
    g = _read_golden("two_device_closed_form.txt")
    Y = np.stack([g["Y1"][None, :], g["Y2"][None, :]])                     # [2, 1, 2]
    B = [np.stack([g["B1_row0"], g["B1_row1"]]), np.stack([g["B2_row0"], g["B2_row1"]])]
    W = np.stack([b.T for b in B])                                         # [2, h, K_r], out x in
    R = np.stack([g["R1"][None, :], g["R2"][None, :]])
    out = O.rowpar_forward(Y, W, R, np.ones(4), None, S=2, alpha=1.0, eps=0.0, norm=O.RMSNORM)
    np.testing.assert_array_equal(out["Z"][0, 0], g["Z1"])
    np.testing.assert_array_equal(out["Z"][1, 0], g["Z2"])
    np.testing.assert_array_equal(out["Hn"][0, 0], g["Hn1"])
    np.testing.assert_array_equal(out["Hn"][1, 0], g["Hn2"])
    np.testing.assert_allclose(out["rstd"][:, 0], [g["meansq1"][0] ** -0.5, g["meansq2"][0] ** -0.5], rtol=1e-15)
    np.testing.assert_allclose(out["X"][0, 0], g["Hn1"] / math.sqrt(g["meansq1"][0]), rtol=1e-15)
    ln = O.rowpar_forward(Y, W, R, np.ones(4), np.zeros(4), S=2, alpha=1.0, eps=0.0, norm=O.LAYERNORM)
    np.testing.assert_allclose(ln["mean"][:, 0], [g["mean1"][0], g["mean2"][0]], rtol=1e-15)
    np.testing.assert_allclose(ln["rstd"][:, 0], [g["var1"][0] ** -0.5, g["var2"][0] ** -0.5], rtol=1e-15)
    np.testing.assert_allclose(ln["X"][1, 0], (g["Hn2"] - g["mean2"][0]) / math.sqrt(g["var2"][0]), rtol=1e-14)


def test_two_device_block_matrix_form():
    # Eq. 7-8 with random blocks: B_m = [B_1m | B_2m]; Z_1 = [Y_1 B_11 + Y_2 B_12, Y_1 B_21], Z_2 likewise.
    rng = _rng(1)
    T, h, K_r, S = 5, 6, 3, 4
    Y1, Y2 = rng.standard_normal((T, K_r)), rng.standard_normal((T, K_r))
    B11, B21 = rng.standard_normal((K_r, S)), rng.standard_normal((K_r, h - S))
    B12, B22 = rng.standard_normal((K_r, S)), rng.standard_normal((K_r, h - S))
    Z1 = np.concatenate([Y1 @ B11 + Y2 @ B12, Y1 @ B21], axis=1)
    Z2 = np.concatenate([Y1 @ B11 + Y2 @ B12, Y2 @ B22], axis=1)
    W = np.stack([np.concatenate([B11, B21], axis=1).T, np.concatenate([B12, B22], axis=1).T])
    Z = O.partial_channel_reduce(O.rank_partials(np.stack([Y1, Y2]), W), S, 1.0)
    np.testing.assert_allclose(Z[0], Z1, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(Z[1], Z2, rtol=1e-13, atol=1e-13)


def test_brute_force_index_notation():
    # Eq. A3 evaluated entry by entry with Python loops (sigma(X A) replaced by the given Y).
    rng = _rng(2)
    t, T, h, K_r = 3, 2, 5, 4
    d = _rand_layer(rng, t, T, h, K_r)
    for S, alpha in itertools.product((0, 2, 5), (1.0, math.sqrt(t))):
        out = O.rowpar_forward(d["Y"], d["W"], d["R"], d["gamma"], None, S=S, alpha=alpha, eps=1e-5)
        for m, i, l in itertools.product(range(t), range(T), range(h)):
            zt = [sum(d["Y"][mm, i, k] * d["W"][mm, l, k] for k in range(K_r)) for mm in range(t)]
            z = sum(zt) if l < S else alpha * zt[m]
            assert out["Z"][m, i, l] == pytest.approx(z, rel=1e-12, abs=1e-12)
            assert out["Hn"][m, i, l] == pytest.approx(z + d["R"][m, i, l], rel=1e-12, abs=1e-12)
        for m, i in itertools.product(range(t), range(T)):
            ms = sum(out["Hn"][m, i, l] ** 2 for l in range(h)) / h
            for l in range(h):
                x = out["Hn"][m, i, l] / math.sqrt(ms + 1e-5) * d["gamma"][l]
                assert out["X"][m, i, l] == pytest.approx(x, rel=1e-12, abs=1e-12)


# ---------------------------------------------------------------- forward: special cases
@pytest.mark.parametrize("norm", [O.RMSNORM, O.LAYERNORM])
def test_p1_equals_unsharded_library(norm):
    # p = 1: a vanilla transformer.  Unsharded Y [T, K] @ W [h, K]^T + R, then the library norm.
    rng = _rng(3)
    t, T, h, K_r = 4, 7, 12, 5
    d = _rand_layer(rng, t, T, h, K_r)
    R = np.broadcast_to(d["R"][0], (t, T, h)).copy()
    out = O.rowpar_forward(d["Y"], d["W"], R, d["gamma"], d["beta"], S=h, alpha=math.sqrt(t), eps=1e-5, norm=norm)
    Ycat = np.concatenate([d["Y"][m] for m in range(t)], axis=1)          # [T, K]
    Wcat = np.concatenate([d["W"][m] for m in range(t)], axis=1)          # [h, K]
    Hn = torch.from_numpy(Ycat) @ torch.from_numpy(Wcat).T + torch.from_numpy(R[0])
    if norm == O.RMSNORM:
        X = F.rms_norm(Hn, (h,), torch.from_numpy(d["gamma"]), eps=1e-5)
    else:
        X = F.layer_norm(Hn, (h,), torch.from_numpy(d["gamma"]), torch.from_numpy(d["beta"]), eps=1e-5)
    for m in range(t):   # every rank holds the same, fully synchronised, result
        np.testing.assert_allclose(out["Hn"][m], Hn.numpy(), rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(out["X"][m], X.numpy(), rtol=1e-11, atol=1e-12)


def test_p0_no_cross_rank_mixing():
    # No shared channels: an ensemble. Changing rank 1's inputs leaves every other rank bitwise unchanged.
    rng = _rng(4)
    t, T, h, K_r = 3, 4, 8, 6
    d = _rand_layer(rng, t, T, h, K_r)
    a = O.rowpar_forward(d["Y"], d["W"], d["R"], d["gamma"], None, S=0, alpha=math.sqrt(t))
    Y2, W2, R2 = d["Y"].copy(), d["W"].copy(), d["R"].copy()
    Y2[1] += 1.0; W2[1] *= -2.0; R2[1] += 3.0
    b = O.rowpar_forward(Y2, W2, R2, d["gamma"], None, S=0, alpha=math.sqrt(t))
    for m in (0, 2):
        assert np.array_equal(a["X"][m], b["X"][m]) and np.array_equal(a["Hn"][m], b["Hn"][m])
    assert not np.array_equal(a["X"][1], b["X"][1])
    # and with shared channels the other ranks DO change, but only through the shared channels' sum
    c = O.rowpar_forward(d["Y"], d["W"], d["R"], d["gamma"], None, S=3, alpha=1.0)
    e = O.rowpar_forward(Y2, W2, d["R"], d["gamma"], None, S=3, alpha=1.0)
    assert not np.array_equal(c["Hn"][0][:, :3], e["Hn"][0][:, :3])
    assert np.array_equal(c["Hn"][0][:, 3:], e["Hn"][0][:, 3:])


def test_rank_permutation_invariance_exact():
    # Integer inputs: sums are exact, so shared sums do not depend on the order of the ranks
    # and private outputs follow their rank.
    rng = _rng(5)
    t, T, h, K_r, S = 4, 6, 8, 5, 3
    Y = rng.integers(-3, 4, (t, T, K_r)).astype(float)
    W = rng.integers(-2, 3, (t, h, K_r)).astype(float)
    R = rng.integers(-4, 5, (t, T, h)).astype(float)
    perm = np.array([2, 0, 3, 1])
    a = O.rowpar_forward(Y, W, R, np.ones(h), None, S=S, alpha=1.0)
    b = O.rowpar_forward(Y[perm], W[perm], R[perm], np.ones(h), None, S=S, alpha=1.0)
    assert np.array_equal(a["Z"][perm], b["Z"])
    assert np.array_equal(a["Hn"][perm], b["Hn"])
    assert np.array_equal(a["Z"][0, :, :S], b["Z"][3, :, :S])


def test_fingerprint_inputs():
    # Y_m == (m+1), W_m selects input 0 for every output: shared = t(t+1)/2, private = alpha (m+1).
    t, T, h, K_r, S = 5, 3, 7, 4, 4
    Y = np.stack([np.full((T, K_r), m + 1.0) for m in range(t)])
    W = np.zeros((t, h, K_r)); W[:, :, 0] = 1.0
    Z = O.partial_channel_reduce(O.rank_partials(Y, W), S, 2.0)
    assert np.all(Z[:, :, :S] == t * (t + 1) / 2)
    for m in range(t):
        assert np.all(Z[m, :, S:] == 2.0 * (m + 1))


def test_variance_law_pins_alpha_location():
    # Eq. 14-15: shared variance t sigma^2, private sigma^2; equal after multiplying private by sqrt(t).
    rng = _rng(6)
    t, T, h, K_r, S = 4, 4096, 32, 64, 16
    Y = rng.standard_normal((t, T, K_r)); W = rng.standard_normal((t, h, K_r)) / math.sqrt(K_r)
    Zt = O.rank_partials(Y, W)
    Z1 = O.partial_channel_reduce(Zt, S, 1.0)
    Zs = O.partial_channel_reduce(Zt, S, O.private_scale(t))
    assert Z1[:, :, :S].var() / Z1[:, :, S:].var() == pytest.approx(t, rel=0.08)
    assert Zs[:, :, :S].var() / Zs[:, :, S:].var() == pytest.approx(1.0, rel=0.08)
    # the scale acts on the layer output before the residual add
    R = rng.standard_normal((t, T, h))
    out = O.rowpar_forward(Y, W, R, np.ones(h), None, S=S, alpha=O.private_scale(t))
    np.testing.assert_allclose(out["Hn"] - R, Zs, rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- backward
def _loss(d, Gx, Gh, S, alpha, norm):
    out = O.rowpar_forward(d["Y"], d["W"], d["R"], d["gamma"], d["beta"], S=S, alpha=alpha, eps=1e-5, norm=norm)
    return float(np.sum(Gx * out["X"]) + np.sum(Gh * out["Hn"]))


@pytest.mark.parametrize("norm", [O.RMSNORM, O.LAYERNORM])
@pytest.mark.parametrize("S,alpha", [(0, 2.0), (3, 1.0), (3, math.sqrt(3.0)), (6, 1.7)])
def test_backward_matches_finite_differences(norm, S, alpha):
    rng = _rng(7)
    t, T, h, K_r = 3, 2, 6, 4
    d = _rand_layer(rng, t, T, h, K_r, backward=True)
    Gx, Gh = d["dX"], d["dHn"]
    f = O.rowpar_forward(d["Y"], d["W"], d["R"], d["gamma"], d["beta"], S=S, alpha=alpha, eps=1e-5, norm=norm)
    b = O.rowpar_backward(Gx, Gh, d["Y"], d["W"], f["Hn"], f["rstd"], f["mean"], d["gamma"], S=S, alpha=alpha, norm=norm)
    step = 1e-6
    checks = [("Y", b["dY"]), ("W", b["dW"]), ("R", b["dR"]), ("gamma", b["dgamma"])]
    if norm == O.LAYERNORM:
        checks.append(("beta", b["dbeta"]))
    for name, grad in checks:
        num = np.zeros_like(d[name])
        it = np.nditer(d[name], flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = d[name][idx]
            d[name][idx] = keep + step; lp = _loss(d, Gx, Gh, S, alpha, norm)
            d[name][idx] = keep - step; lm = _loss(d, Gx, Gh, S, alpha, norm)
            d[name][idx] = keep
            num[idx] = (lp - lm) / (2 * step)
        scale = max(1.0, np.abs(num).max())
        assert np.abs(num - grad).max() / scale < 2e-7, name


def _torch_forward(Y, W, R, gamma, beta, S, alpha, norm):
    """An independent forward graph made of library ops only, for autograd."""
    t, T, h = R.shape
    Zt = torch.einsum("mik,mlk->mil", Y, W)
    Zs = Zt[:, :, :S].sum(dim=0, keepdim=True).expand(t, T, S)
    Hn = torch.cat([Zs, alpha * Zt[:, :, S:]], dim=2) + R
    if norm == O.RMSNORM:
        X = F.rms_norm(Hn, (h,), gamma, eps=1e-5)
    else:
        X = F.layer_norm(Hn, (h,), gamma, beta, eps=1e-5)
    return Hn, X


@pytest.mark.parametrize("norm", [O.RMSNORM, O.LAYERNORM])
def test_backward_matches_autograd(norm):
    rng = _rng(8)
    t, T, h, K_r, S, alpha = 4, 9, 16, 6, 8, 2.0
    d = _rand_layer(rng, t, T, h, K_r, backward=True)
    tt = {k: torch.tensor(v, requires_grad=k in ("Y", "W", "R", "gamma", "beta")) for k, v in d.items()}
    Hn, X = _torch_forward(tt["Y"], tt["W"], tt["R"], tt["gamma"], tt["beta"], S, alpha, norm)
    ((tt["dX"] * X).sum() + (tt["dHn"] * Hn).sum()).backward()
    f = O.rowpar_forward(d["Y"], d["W"], d["R"], d["gamma"], d["beta"], S=S, alpha=alpha, eps=1e-5, norm=norm)
    b = O.rowpar_backward(d["dX"], d["dHn"], d["Y"], d["W"], f["Hn"], f["rstd"], f["mean"], d["gamma"],
                          S=S, alpha=alpha, norm=norm)
    np.testing.assert_allclose(b["dY"], tt["Y"].grad.numpy(), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(b["dW"], tt["W"].grad.numpy(), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(b["dR"], tt["R"].grad.numpy(), rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(b["dgamma"], tt["gamma"].grad.numpy(), rtol=1e-10, atol=1e-11)
    if norm == O.LAYERNORM:
        np.testing.assert_allclose(b["dbeta"], tt["beta"].grad.numpy(), rtol=1e-10, atol=1e-11)


def test_backward_p1_reduce_before_or_after_norm():
    # Section 4: with full synchronisation, reducing the gradients after the norm's backward
    # (plus summing norm-parameter gradients over ranks) equals reducing them before it.
    rng = _rng(9)
    t, T, h, K_r = 4, 5, 10, 3
    d = _rand_layer(rng, t, T, h, K_r, backward=True)
    R = np.broadcast_to(d["R"][0], (t, T, h)).copy()
    f = O.rowpar_forward(d["Y"], d["W"], R, d["gamma"], None, S=h, alpha=1.0, eps=1e-5)
    b = O.rowpar_backward(d["dX"], d["dHn"], d["Y"], d["W"], f["Hn"], f["rstd"], None, d["gamma"], S=h, alpha=1.0)
    # single-device textbook graph: one Hn, upstream gradient = sum over ranks (reduce BEFORE the norm)
    Hn = torch.tensor(f["Hn"][0], requires_grad=True)
    gamma = torch.tensor(d["gamma"], requires_grad=True)
    X = F.rms_norm(Hn, (h,), gamma, eps=1e-5)
    ((torch.tensor(d["dX"].sum(0)) * X).sum() + (torch.tensor(d["dHn"].sum(0)) * Hn).sum()).backward()
    for m in range(t):
        np.testing.assert_allclose(b["dZt"][m], Hn.grad.numpy(), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(b["dgamma"], gamma.grad.numpy(), rtol=1e-11, atol=1e-12)
    # the per-rank residual gradients are partial contributions whose rank sum is the logical gradient
    np.testing.assert_allclose(b["dR"].sum(0), Hn.grad.numpy(), rtol=1e-11, atol=1e-12)


def test_backward_reduce_is_transpose_of_forward_reduce():
    # <PCR(a), b> == <a, PCR(b)> : the backward reduction sits at the forward one's place.
    rng = _rng(10)
    a, b = rng.standard_normal((3, 4, 7)), rng.standard_normal((3, 4, 7))
    lhs = np.sum(O.partial_channel_reduce(a, 3, 1.5) * b)
    rhs = np.sum(a * O.backward_partial_channel_reduce(b, 3, 1.5))
    assert lhs == pytest.approx(rhs, rel=1e-13)


# ---------------------------------------------------------------- block
def test_block_chains_through_residual_and_matches_finite_differences():
    rng = _rng(11)
    t, T, h, ka, km, S, alpha = 2, 2, 4, 2, 3, 2, math.sqrt(2.0)
    inp = {"Y_attn": rng.standard_normal((t, T, ka)), "W_o": rng.standard_normal((t, h, ka)) * 0.4,
           "Y_mlp": rng.standard_normal((t, T, km)), "W_down": rng.standard_normal((t, h, km)) * 0.4,
           "R0": rng.standard_normal((t, T, h)), "gamma1": 1 + 0.1 * rng.standard_normal(h),
           "gamma2": 1 + 0.1 * rng.standard_normal(h)}
    G1, G2, Gh = (rng.standard_normal((t, T, h)) for _ in range(3))

    def fwd():
        return O.block_forward(inp["Y_attn"], inp["W_o"], inp["Y_mlp"], inp["W_down"], inp["R0"],
                               inp["gamma1"], inp["gamma2"], S=S, alpha=alpha)

    def loss():
        o = fwd()
        return float(np.sum(G1 * o["X1"]) + np.sum(G2 * o["X2"]) + np.sum(Gh * o["Hn2"]))

    o = fwd()
    l1 = O.rowpar_forward(inp["Y_attn"], inp["W_o"], inp["R0"], inp["gamma1"], None, S=S, alpha=alpha)
    l2 = O.rowpar_forward(inp["Y_mlp"], inp["W_down"], l1["Hn"], inp["gamma2"], None, S=S, alpha=alpha)
    assert np.array_equal(o["X1"], l1["X"]) and np.array_equal(o["Hn2"], l2["Hn"]) and np.array_equal(o["X2"], l2["X"])
    b = O.block_backward(G1, G2, Gh, inp["Y_attn"], inp["W_o"], inp["Y_mlp"], inp["W_down"], o["Hn1"], o["rstd1"],
                         None, o["Hn2"], o["rstd2"], None, inp["gamma1"], inp["gamma2"], S=S, alpha=alpha)
    pairs = [("Y_attn", "dY_attn"), ("W_o", "dW_o"), ("Y_mlp", "dY_mlp"), ("W_down", "dW_down"),
             ("R0", "dR0"), ("gamma1", "dgamma1"), ("gamma2", "dgamma2")]
    step = 1e-6
    for name, gname in pairs:
        num = np.zeros_like(inp[name])
        it = np.nditer(inp[name], flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = inp[name][idx]
            inp[name][idx] = keep + step; lp = loss()
            inp[name][idx] = keep - step; lm = loss()
            inp[name][idx] = keep
            num[idx] = (lp - lm) / (2 * step)
        assert np.abs(num - b[gname]).max() / max(1.0, np.abs(num).max()) < 2e-7, name


# ---------------------------------------------------------------- column-parallel half
def test_silu_and_its_derivative_match_the_library():
    x = np.linspace(-12, 12, 4001)
    xt = torch.tensor(x, requires_grad=True)
    y = F.silu(xt)
    y.sum().backward()
    np.testing.assert_allclose(O.silu(x), y.detach().numpy(), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(O.silu_grad(x), xt.grad.numpy(), rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("act", [O.ACT_NONE, O.ACT_SILU, O.ACT_SWIGLU])
def test_colpar_shards_concatenate_to_the_unsharded_layer(act):
    # Section 3 (standard tensor parallelism): with the SAME input on every rank, the column shards'
    # outputs side by side are the unsharded sigma(X A)
    rng = _rng(41)
    t, T, h, N = 4, 7, 10, 6
    Xs = rng.standard_normal((T, h))
    A = rng.standard_normal((t, N, h)) * 0.5
    out = O.colpar_forward(np.broadcast_to(Xs, (t, T, h)), A, act)["Y"]
    if act == O.ACT_SWIGLU:
        Fh = N // 2
        gate = np.concatenate([A[m, :Fh] for m in range(t)], 0)       # [t Fh, h]
        up = np.concatenate([A[m, Fh:] for m in range(t)], 0)
        ref = F.silu(torch.tensor(Xs @ gate.T)).numpy() * (Xs @ up.T)
    else:
        full = np.concatenate([A[m] for m in range(t)], 0)
        pre = Xs @ full.T
        ref = pre if act == O.ACT_NONE else F.silu(torch.tensor(pre)).numpy()
    np.testing.assert_allclose(np.concatenate([out[m] for m in range(t)], 1), ref, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("act", [O.ACT_NONE, O.ACT_SILU, O.ACT_SWIGLU])
def test_colpar_backward_matches_autograd(act):
    rng = _rng(42)
    t, T, h, N = 3, 5, 8, 6
    X, A = rng.standard_normal((t, T, h)), rng.standard_normal((t, N, h)) * 0.5
    dY = rng.standard_normal((t, T, N // 2 if act == O.ACT_SWIGLU else N))
    Xt, At = torch.tensor(X, requires_grad=True), torch.tensor(A, requires_grad=True)
    pre = torch.einsum("mik,mlk->mil", Xt, At)
    if act == O.ACT_NONE:
        Y = pre
    elif act == O.ACT_SILU:
        Y = F.silu(pre)
    else:
        Y = F.silu(pre[:, :, :N // 2]) * pre[:, :, N // 2:]
    (Y * torch.tensor(dY)).sum().backward()
    f = O.colpar_forward(X, A, act)
    np.testing.assert_allclose(f["Y"], Y.detach().numpy(), rtol=1e-12, atol=1e-13)
    b = O.colpar_backward(dY, X, A, f["pre"], act)
    np.testing.assert_allclose(b["dX"], Xt.grad.numpy(), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(b["dA"], At.grad.numpy(), rtol=1e-11, atol=1e-12)


def test_mlp_backward_matches_finite_differences():
    rng = _rng(43)
    t, T, h, Fh, S, alpha = 2, 2, 4, 3, 2, math.sqrt(2.0)
    d = {"X": rng.standard_normal((t, T, h)), "A": rng.standard_normal((t, 2 * Fh, h)) * 0.5,
         "B": rng.standard_normal((t, h, Fh)) * 0.5, "R": rng.standard_normal((t, T, h)),
         "gamma": 1 + 0.1 * rng.standard_normal(h)}
    Gx, Gh = rng.standard_normal((t, T, h)), rng.standard_normal((t, T, h))

    def fwd():
        return O.mlp_forward(d["X"], d["A"], d["B"], d["R"], d["gamma"], S=S, alpha=alpha)

    def loss():
        o = fwd()
        return float(np.sum(Gx * o["X"]) + np.sum(Gh * o["Hn"]))

    o = fwd()
    b = O.mlp_backward(Gx, Gh, d["X"], d["A"], d["B"], o["pre"], o["Y"], o["Hn"], o["rstd"], None, d["gamma"], S=S, alpha=alpha)
    step = 1e-6
    for name, gname in (("X", "dX"), ("A", "dA"), ("B", "dB"), ("R", "dR"), ("gamma", "dgamma")):
        num = np.zeros_like(d[name])
        it = np.nditer(d[name], flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = d[name][idx]
            d[name][idx] = keep + step; lp = loss()
            d[name][idx] = keep - step; lm = loss()
            d[name][idx] = keep
            num[idx] = (lp - lm) / (2 * step)
        assert np.abs(num - b[gname]).max() / max(1.0, np.abs(num).max()) < 2e-7, name


# ---------------------------------------------------------------- precision models of the backward reduce
def test_round_bf16_matches_library_cast():
    rng = _rng(31)
    x = np.concatenate([rng.standard_normal(4096) * 10.0 ** rng.integers(-6, 6, 4096),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e38, 1e-40])])
    ref = torch.tensor(x, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(O.round_bf16(x), ref)
    # ties go to the even significand: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert O.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert O.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6


def test_reduce_precision_models():
    rng = _rng(32)
    t, T, h, S = 16, 64, 32, 16
    g = rng.standard_normal((t, T, h))
    exact = O.backward_partial_channel_reduce(g, S, 2.0)
    wire = O.backward_partial_channel_reduce(g, S, 2.0, reduce_mode=1)
    acc16 = O.backward_partial_channel_reduce(g, S, 2.0, reduce_mode=2)
    # private channels are untouched by the model; shared ones are identical on every rank
    for r in (wire, acc16):
        np.testing.assert_array_equal(r[:, :, S:], exact[:, :, S:])
        assert all(np.array_equal(r[0, :, :S], r[m, :, :S]) for m in range(t))
    # mode 1 is the exact sum of rounded terms; mode 2 stays on the bfloat16 grid
    np.testing.assert_allclose(wire[0, :, :S], O.round_bf16(g[:, :, :S]).sum(0), rtol=0, atol=1e-12)
    np.testing.assert_array_equal(acc16[0, :, :S], O.round_bf16(acc16[0, :, :S]))
    # error bounds: each rounding is at most half a unit in the last place (2^-9 relative)
    e1 = np.abs(wire - exact)[0, :, :S]
    assert e1.max() <= 2.0 ** -9 * np.abs(g[:, :, :S]).sum(0).max() * 1.0001
    e2 = np.abs(acc16 - exact)[0, :, :S]
    assert e1.mean() < e2.mean()          # accumulating in 16 bit loses more than a 16-bit payload
    # a value already on the grid, one rank: both models are exact
    one = O.round_bf16(rng.standard_normal((1, 4, 8)))
    np.testing.assert_array_equal(O.backward_partial_channel_reduce(one, 8, 1.0, reduce_mode=2), one)


# ---------------------------------------------------------------- compact residual layout
def _rand_compact(rng, t, T, h, K_r, S):
    return {"Y": rng.standard_normal((t, T, K_r)), "W": rng.standard_normal((t, h, K_r)) * 0.3,
            "Rs": rng.standard_normal((T, S)), "Rp": rng.standard_normal((t, T, h - S)),
            "gamma": 1.0 + 0.2 * rng.standard_normal(h), "beta": 0.1 * rng.standard_normal(h)}


@pytest.mark.parametrize("norm", [O.RMSNORM, O.LAYERNORM])
def test_compact_forward_is_per_rank_forward_on_tied_residual(norm):
    # the compact form is the per-rank map evaluated on R[m] = [Rs | Rp[m]]
    rng = _rng(21)
    t, T, h, K_r, S, alpha = 3, 5, 12, 4, 8, math.sqrt(3.0)
    d = _rand_compact(rng, t, T, h, K_r, S)
    R = np.concatenate([np.broadcast_to(d["Rs"], (t, T, S)), d["Rp"]], axis=2)
    ref = O.rowpar_forward(d["Y"], d["W"], R, d["gamma"], d["beta"], S=S, alpha=alpha, norm=norm)
    out = O.rowpar_forward_compact(d["Y"], d["W"], d["Rs"], d["Rp"], d["gamma"], d["beta"], S=S, alpha=alpha, norm=norm)
    for m in range(t):
        np.testing.assert_allclose(out["Hns"], ref["Hn"][m, :, :S], rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(out["Hnp"], ref["Hn"][:, :, S:], rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(out["X"], ref["X"], rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(out["rstd"], ref["rstd"], rtol=1e-13)


@pytest.mark.parametrize("norm", [O.RMSNORM, O.LAYERNORM])
@pytest.mark.parametrize("S,alpha", [(0, 2.0), (4, 1.0), (4, math.sqrt(3.0)), (6, 1.7)])
def test_compact_backward_matches_finite_differences(norm, S, alpha):
    rng = _rng(22)
    t, T, h, K_r = 3, 2, 6, 4
    d = _rand_compact(rng, t, T, h, K_r, S)
    Gx, Gs, Gp = rng.standard_normal((t, T, h)), rng.standard_normal((T, S)), rng.standard_normal((t, T, h - S))

    def loss():
        o = O.rowpar_forward_compact(d["Y"], d["W"], d["Rs"], d["Rp"], d["gamma"], d["beta"], S=S, alpha=alpha, norm=norm)
        return float(np.sum(Gx * o["X"]) + np.sum(Gs * o["Hns"]) + np.sum(Gp * o["Hnp"]))

    f = O.rowpar_forward_compact(d["Y"], d["W"], d["Rs"], d["Rp"], d["gamma"], d["beta"], S=S, alpha=alpha, norm=norm)
    b = O.rowpar_backward_compact(Gx, Gs, Gp, d["Y"], d["W"], f["Hns"], f["Hnp"], f["rstd"], f["mean"], d["gamma"],
                                  S=S, alpha=alpha, norm=norm)
    checks = [("Y", b["dY"]), ("W", b["dW"]), ("Rs", b["dRs"]), ("Rp", b["dRp"]), ("gamma", b["dgamma"])]
    if norm == O.LAYERNORM:
        checks.append(("beta", b["dbeta"]))
    step = 1e-6
    for name, grad in checks:
        if d[name].size == 0:
            assert grad.size == 0
            continue
        num = np.zeros_like(d[name])
        it = np.nditer(d[name], flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = d[name][idx]
            d[name][idx] = keep + step; lp = loss()
            d[name][idx] = keep - step; lm = loss()
            d[name][idx] = keep
            num[idx] = (lp - lm) / (2 * step)
        assert np.abs(num - grad).max() / max(1.0, np.abs(num).max()) < 2e-7, name


def test_compact_backward_is_rank_sum_of_per_rank_backward():
    # per-rank copies of a tied variable: the gradient of the single variable is the sum of the
    # copies' gradients, for ANY split of the upstream dHns over the copies
    rng = _rng(23)
    t, T, h, K_r, S, alpha = 4, 3, 16, 5, 8, 2.0
    d = _rand_compact(rng, t, T, h, K_r, S)
    Gx, Gs, Gp = rng.standard_normal((t, T, h)), rng.standard_normal((T, S)), rng.standard_normal((t, T, h - S))
    f = O.rowpar_forward_compact(d["Y"], d["W"], d["Rs"], d["Rp"], d["gamma"], None, S=S, alpha=alpha)
    b = O.rowpar_backward_compact(Gx, Gs, Gp, d["Y"], d["W"], f["Hns"], f["Hnp"], f["rstd"], None, d["gamma"], S=S, alpha=alpha)
    split = rng.standard_normal((t, 1, 1)); split = split / split.sum()
    dHn = np.concatenate([split * Gs[None], Gp], axis=2)
    Hn = np.concatenate([np.broadcast_to(f["Hns"], (t, T, S)), f["Hnp"]], axis=2)
    ref = O.rowpar_backward(Gx, dHn, d["Y"], d["W"], Hn, f["rstd"], None, d["gamma"], S=S, alpha=alpha)
    np.testing.assert_allclose(b["dRs"], ref["dR"][:, :, :S].sum(0), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(b["dRp"], ref["dR"][:, :, S:], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(b["dY"], ref["dY"], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(b["dW"], ref["dW"], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(b["dgamma"], ref["dgamma"], rtol=1e-11, atol=1e-12)


def test_compact_block_matches_finite_differences():
    rng = _rng(24)
    t, T, h, ka, km, S, alpha = 2, 2, 4, 2, 3, 2, math.sqrt(2.0)
    inp = {"Y_attn": rng.standard_normal((t, T, ka)), "W_o": rng.standard_normal((t, h, ka)) * 0.4,
           "Y_mlp": rng.standard_normal((t, T, km)), "W_down": rng.standard_normal((t, h, km)) * 0.4,
           "R0s": rng.standard_normal((T, S)), "R0p": rng.standard_normal((t, T, h - S)),
           "gamma1": 1 + 0.1 * rng.standard_normal(h), "gamma2": 1 + 0.1 * rng.standard_normal(h)}
    G1, G2 = rng.standard_normal((t, T, h)), rng.standard_normal((t, T, h))
    Gs, Gp = rng.standard_normal((T, S)), rng.standard_normal((t, T, h - S))

    def fwd():
        return O.block_forward_compact(inp["Y_attn"], inp["W_o"], inp["Y_mlp"], inp["W_down"], inp["R0s"], inp["R0p"],
                                       inp["gamma1"], inp["gamma2"], S=S, alpha=alpha)

    def loss():
        o = fwd()
        return float(np.sum(G1 * o["X1"]) + np.sum(G2 * o["X2"]) + np.sum(Gs * o["Hn2s"]) + np.sum(Gp * o["Hn2p"]))

    o = fwd()
    b = O.block_backward_compact(G1, G2, Gs, Gp, inp["Y_attn"], inp["W_o"], inp["Y_mlp"], inp["W_down"], o["Hn1s"],
                                 o["Hn1p"], o["rstd1"], None, o["Hn2s"], o["Hn2p"], o["rstd2"], None, inp["gamma1"],
                                 inp["gamma2"], S=S, alpha=alpha)
    pairs = [("Y_attn", "dY_attn"), ("W_o", "dW_o"), ("Y_mlp", "dY_mlp"), ("W_down", "dW_down"),
             ("R0s", "dR0s"), ("R0p", "dR0p"), ("gamma1", "dgamma1"), ("gamma2", "dgamma2")]
    step = 1e-6
    for name, gname in pairs:
        num = np.zeros_like(inp[name])
        it = np.nditer(inp[name], flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = inp[name][idx]
            inp[name][idx] = keep + step; lp = loss()
            inp[name][idx] = keep - step; lm = loss()
            inp[name][idx] = keep
            num[idx] = (lp - lm) / (2 * step)
        assert np.abs(num - b[gname]).max() / max(1.0, np.abs(num).max()) < 2e-7, name


# ---------------------------------------------------------------- analytic bytes
def test_allreduce_bytes_closed_forms():
    # Appendix C: per block forward the payload is P(p) = 2 s h p activations per device (two reduces).
    s, h, t = 2048, 4096, 8
    for p in (1.0, 0.75, 0.5, 0.25, 0.0):
        S = O.shared_channels(h, p)
        a = O.allreduce_bytes(s, h, t, S, elem_bytes=1)
        assert 2 * a["payload_per_rank"] == 2 * s * h * p
        assert a["payload_per_rank_p1"] == s * h
        # Appendix D: traffic is cut by 100 (1 - p) percent
        assert 1.0 - a["payload_per_rank"] / a["payload_per_rank_p1"] == pytest.approx(1.0 - p)
        assert a["ring_wire_per_rank"] == pytest.approx(2 * (t - 1) / t * s * S)
    assert O.allreduce_bytes(16384, 768, 4, 384, 2)["payload_per_rank"] == 16384 * 384 * 2
    assert O.allreduce_bytes(1, 4096, 8, 4096, 2)["norm_grad_sync_bytes"] == 4096 * 4


def test_collective_byte_counts_are_the_sizes_of_the_tensors_the_method_exchanges():
    # Not the formulas again: the payload is the storage size of the slab the forward really sums over the ranks (the
    # shared columns of one rank's partial output), and the norm-parameter synchronisation (Eq. 10-11, Section 4) is
    # the storage size of the fp32 gradient of gamma that the backward really produces.
    t, T, h, K, S = 4, 37, 96, 8, 40
    rng = np.random.default_rng(3)
    Y, W = rng.standard_normal((t, T, K)), rng.standard_normal((t, h, K))
    R, gamma = rng.standard_normal((t, T, h)), 1 + 0.1 * rng.standard_normal(h)
    f = O.rowpar_forward(Y, W, R, gamma, None, S=S, alpha=2.0)
    slab = f["Zt"][0][:, :S]                                           # what one rank contributes to the reduce
    b = O.rowpar_backward(rng.standard_normal((t, T, h)), None, Y, W, f["Hn"], f["rstd"], None, gamma, S=S, alpha=2.0)
    for e, dt in ((2, np.float16), (4, np.float32)):
        a = O.allreduce_bytes(T, h, t, S, e)
        assert a["payload_per_rank"] == slab.astype(dt).nbytes
        assert a["payload_per_rank_p1"] == f["Zt"][0].astype(dt).nbytes
        assert a["norm_grad_sync_bytes"] == b["dgamma"].astype(np.float32).nbytes
    # the private scale acts on exactly the columns the reduce leaves out: alpha times the rank's own partial there
    assert np.array_equal(f["Z"][1][:, S:], 2.0 * f["Zt"][1][:, S:])
    assert np.allclose(f["Z"][1][:, :S], f["Zt"][:, :, :S].sum(0))


def test_speedup_model_closed_form():
    # Appendix C: (T(1) - T(p)) / T(1) = (1 - p) / (1 + (12 h + 2 s) / (C r)).
    for h, s, r, C, p in [(4096, 2048, 8, 3000.0, 0.5), (768, 1024, 16, 500.0, 0.25), (2048, 2048, 4, 8000.0, 0.75)]:
        assert O.speedup_model(h, s, r, C, p) == pytest.approx((1 - p) / (1 + (12 * h + 2 * s) / (C * r)), rel=1e-12)
