"""Pins of the fp64 CPU oracle against what the definitions and the mathematics fix (CPU only).

Each test is chosen so that a plausible mistake in oracle.c (dropped term, flipped kernel, wrong pad or
stride index, transposed operand, biased/unbiased mix-up, sign error in a gradient) fails at least one.
Nothing here uses the CUDA library.
"""
import math

import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(20260925)


# --------------------------------------------------------------------------- independent brute force (python loops)
def brute_conv(x, w, stride):
    N, H, W, C = x.shape
    K, k, _, _ = w.shape
    P = k // 2
    Ho = (H + 2 * P - k) // stride + 1
    Wo = (W + 2 * P - k) // stride + 1
    xp = np.zeros((N, H + 2 * P, W + 2 * P, C))
    xp[:, P:P + H, P:P + W, :] = x  # explicit zero padding instead of bounds tests
    y = np.zeros((N, Ho, Wo, K))
    for n in range(N):
        for p in range(Ho):
            for q in range(Wo):
                for co in range(K):
                    patch = xp[n, p * stride:p * stride + k, q * stride:q * stride + k, :]
                    y[n, p, q, co] = float((patch * w[co]).sum())
    return y


def brute_dgrad_scatter(dy, w, xshape, stride):
    N, H, W, C = xshape
    K, k, _, _ = w.shape
    P = k // 2
    dxp = np.zeros((N, H + 2 * P, W + 2 * P, C))
    for n in range(dy.shape[0]):
        for p in range(dy.shape[1]):
            for q in range(dy.shape[2]):
                for co in range(K):
                    dxp[n, p * stride:p * stride + k, q * stride:q * stride + k, :] += dy[n, p, q, co] * w[co]
    return dxp[:, P:P + H, P:P + W, :]


def brute_wgrad_scatter(x, dy, k, stride):
    N, H, W, C = x.shape
    K = dy.shape[-1]
    P = k // 2
    xp = np.zeros((N, H + 2 * P, W + 2 * P, C))
    xp[:, P:P + H, P:P + W, :] = x
    dw = np.zeros((K, k, k, C))
    for n in range(dy.shape[0]):
        for p in range(dy.shape[1]):
            for q in range(dy.shape[2]):
                patch = xp[n, p * stride:p * stride + k, q * stride:q * stride + k, :]
                for co in range(K):
                    dw[co] += dy[n, p, q, co] * patch
    return dw


SHAPES = [  # N, H, W, Cin, Cout, k, stride
    (2, 7, 6, 3, 4, 3, 2),
    (1, 5, 5, 2, 3, 3, 2),
    (2, 6, 5, 4, 2, 3, 1),
    (1, 4, 7, 5, 3, 1, 1),
    (2, 5, 6, 3, 2, 1, 2),
    (1, 1, 1, 2, 2, 3, 1),
]


@pytest.mark.parametrize("N,H,W,C,K,k,s", SHAPES)
def test_conv_fwd_brute_force(N, H, W, C, K, k, s):
    x = RNG.normal(size=(N, H, W, C))
    w = RNG.normal(size=(K, k, k, C))
    np.testing.assert_allclose(oracle.conv_fwd(x, w, s), brute_conv(x, w, s), rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("N,H,W,C,K,k,s", SHAPES)
def test_dgrad_wgrad_brute_force_scatter(N, H, W, C, K, k, s):
    x = RNG.normal(size=(N, H, W, C))
    w = RNG.normal(size=(K, k, k, C))
    Ho, Wo = oracle.out_extent(H, k, s), oracle.out_extent(W, k, s)
    dy = RNG.normal(size=(N, Ho, Wo, K))
    np.testing.assert_allclose(oracle.conv_dgrad(dy, w, x.shape, s), brute_dgrad_scatter(dy, w, x.shape, s), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(oracle.conv_wgrad(x, dy, k, s), brute_wgrad_scatter(x, dy, k, s), rtol=1e-12, atol=1e-12)


def test_out_extent_values():
    assert oracle.out_extent(640, 3, 2) == 320
    assert oracle.out_extent(5, 3, 2) == 3
    assert oracle.out_extent(6, 3, 2) == 3
    assert oracle.out_extent(7, 1, 2) == 4
    assert oracle.out_extent(160, 3, 1) == 160
    assert oracle.out_extent(40, 1, 1) == 40


# --------------------------------------------------------------------------- conv special cases
def test_conv_1x1_is_matmul():
    x = RNG.normal(size=(2, 5, 4, 7))
    w = RNG.normal(size=(6, 1, 1, 7))
    y = oracle.conv_fwd(x, w, 1)
    ref = x.reshape(-1, 7) @ w.reshape(6, 7).T
    np.testing.assert_allclose(y.reshape(-1, 6), ref, rtol=1e-12, atol=1e-13)
    dy = RNG.normal(size=y.shape)
    np.testing.assert_allclose(oracle.conv_dgrad(dy, w, x.shape, 1).reshape(-1, 7), dy.reshape(-1, 6) @ w.reshape(6, 7), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(oracle.conv_wgrad(x, dy, 1, 1).reshape(6, 7), dy.reshape(-1, 6).T @ x.reshape(-1, 7), rtol=1e-12, atol=1e-12)


def test_conv_identity_and_shift_kernels():
    C = 3
    x = RNG.normal(size=(2, 6, 5, C))
    for r in range(3):
        for t in range(3):
            w = np.zeros((C, 3, 3, C))
            for c in range(C):
                w[c, r, t, c] = 1.0
            y = oracle.conv_fwd(x, w, 1)
            # y[p,q] = x[p-1+r, q-1+t] with zero fill: cross-correlation, no flip
            ref = np.zeros_like(x)
            for p in range(6):
                for q in range(5):
                    h, ww = p - 1 + r, q - 1 + t
                    if 0 <= h < 6 and 0 <= ww < 5:
                        ref[:, p, q, :] = x[:, h, ww, :]
            np.testing.assert_array_equal(y, ref)
    # a non-symmetric tap pattern distinguishes correlation from convolution
    w = np.zeros((1, 3, 3, 1))
    w[0, 0, 2, 0] = 1.0
    xx = np.arange(16.0).reshape(1, 4, 4, 1)
    y = oracle.conv_fwd(xx, w, 1)
    assert y[0, 1, 1, 0] == xx[0, 0, 2, 0]


@pytest.mark.parametrize("s", [1, 2])
def test_conv_all_ones_closed_form(s):
    H, W, C, K = 8, 6, 5, 2
    y = oracle.conv_fwd(np.ones((1, H, W, C)), np.ones((K, 3, 3, C)), s)
    Ho, Wo = y.shape[1:3]
    for p in range(Ho):
        for q in range(Wo):
            nh = sum(1 for r in range(3) if 0 <= p * s - 1 + r < H)
            nw = sum(1 for t in range(3) if 0 <= q * s - 1 + t < W)
            assert y[0, p, q, 0] == nh * nw * C
    if s == 1:
        assert y[0, 0, 0, 0] == 4 * C and y[0, 0, 2, 1] == 6 * C and y[0, 3, 3, 0] == 9 * C


@pytest.mark.parametrize("N,H,W,C,K,k,s", SHAPES + [(2, 9, 8, 6, 5, 3, 2), (3, 8, 8, 4, 4, 3, 1)])
def test_adjoint_identities(N, H, W, C, K, k, s):
    x = RNG.normal(size=(N, H, W, C))
    w = RNG.normal(size=(K, k, k, C))
    y = oracle.conv_fwd(x, w, s)
    g = RNG.normal(size=y.shape)
    lhs = float((y * g).sum())
    a1 = float((x * oracle.conv_dgrad(g, w, x.shape, s)).sum())
    a2 = float((w * oracle.conv_wgrad(x, g, k, s)).sum())
    scale = abs(lhs) + 1.0
    assert abs(lhs - a1) / scale < 1e-12
    assert abs(lhs - a2) / scale < 1e-12


# --------------------------------------------------------------------------- batch-norm statistics
def test_bn_stats_against_numpy_and_invariants():
    y = RNG.normal(size=(3, 5, 4, 6)) * RNG.uniform(0.5, 3.0, size=6) + RNG.normal(size=6) * 4
    eps = 1e-3
    mean, var, invstd = oracle.bn_stats(y, eps)
    flat = y.reshape(-1, 6)
    np.testing.assert_allclose(mean, flat.mean(0), rtol=1e-13)
    np.testing.assert_allclose(var, flat.var(0), rtol=1e-12)  # ddof=0: biased
    np.testing.assert_allclose(invstd, 1 / np.sqrt(flat.var(0) + eps), rtol=1e-12)
    xhat = (flat - mean) * invstd
    assert np.abs(xhat.sum(0)).max() < 1e-11
    # not exactly unit variance: mean(xhat^2) = var/(var+eps) = 1 - eps*invstd^2
    np.testing.assert_allclose((xhat ** 2).mean(0), 1 - eps * invstd ** 2, rtol=1e-12)


def test_bn_constant_channel_and_affine_equivariance():
    y = RNG.normal(size=(2, 3, 3, 2))
    y[..., 1] = 2.5
    eps = 1e-3
    mean, var, invstd = oracle.bn_stats(y, eps)
    assert var[1] == 0.0 and mean[1] == 2.5
    assert math.isclose(invstd[1], eps ** -0.5, rel_tol=1e-15)
    a = oracle.bn_silu_fwd(y, mean, invstd, np.array([1.0, 1.3]), np.array([0.0, 0.4]))
    np.testing.assert_allclose(a[..., 1], 0.4 / (1 + math.exp(-0.4)), rtol=1e-14)
    # y -> alpha*y + delta with eps -> alpha^2 eps leaves xhat unchanged
    alpha, delta = 3.0, -7.0
    m2, v2, i2 = oracle.bn_stats(alpha * y + delta, alpha * alpha * eps)
    np.testing.assert_allclose(((alpha * y + delta) - m2) * i2, (y - mean) * invstd, rtol=1e-10, atol=1e-12)


def test_bn_running_stats_hand_recurrence():
    # M = 4 values of one channel: 1, 2, 3, 6 -> mean 3, biased var 3.5, unbiased var 14/3
    y = np.array([1.0, 2.0, 3.0, 6.0]).reshape(4, 1, 1, 1)
    rm, rv = np.array([10.0]), np.array([2.0])
    mean, var, _ = oracle.bn_stats(y, 1e-3, rm, rv, momentum=0.1)
    assert mean[0] == 3.0 and var[0] == 3.5
    assert math.isclose(rm[0], 0.9 * 10.0 + 0.1 * 3.0, rel_tol=1e-15)
    assert math.isclose(rv[0], 0.9 * 2.0 + 0.1 * (14.0 / 3.0), rel_tol=1e-15)


# --------------------------------------------------------------------------- SiLU
def _silu_via_oracle(z):
    z = np.asarray(z, dtype=np.float64).reshape(-1, 1)
    # mean 0, invstd 1, gamma 1, beta 0 turn the normalise step into the identity
    return oracle.bn_silu_fwd(z, np.zeros(1), np.ones(1), np.ones(1), np.zeros(1)).ravel()


def test_silu_closed_form_values():
    a = _silu_via_oracle([0.0, 1.0, -1.0, 40.0, -40.0, -800.0])
    assert a[0] == 0.0
    assert math.isclose(a[1], 0.7310585786300049, rel_tol=1e-15)
    assert math.isclose(a[2], -0.2689414213699951, rel_tol=1e-15)
    assert math.isclose(a[3], 40.0, rel_tol=1e-15)
    assert -1e-15 < a[4] <= 0.0
    assert a[5] == 0.0 or (a[5] <= 0.0 and a[5] > -1e-300)
    z = np.linspace(-6, 6, 101)
    np.testing.assert_allclose(_silu_via_oracle(z) - _silu_via_oracle(-z), z, atol=1e-14)
    zz = np.linspace(-3, 0, 300001)
    az = _silu_via_oracle(zz)
    i = int(np.argmin(az))
    assert abs(zz[i] + 1.2784645) < 2e-5 and abs(az[i] + 0.2784645) < 1e-7


def test_silu_derivative_through_backward():
    # with mean 0, invstd 1, gamma 1 and M large the BN correction terms vanish for a single perturbed element;
    # use the dz the oracle forms by choosing g = e_i and reading dbeta = sum dz = silu'(z_i)
    for z0, want in [(0.0, 0.5), (40.0, 1.0), (-40.0, 0.0)]:
        y = np.array([z0, 0.0]).reshape(2, 1)
        g = np.array([1.0, 0.0]).reshape(2, 1)
        _, _, dbeta = oracle.bn_silu_bwd(g, y, np.zeros(1), np.ones(1), np.ones(1), np.zeros(1))
        assert abs(dbeta[0] - want) < 1e-12
    s = 1 / (1 + math.exp(-1.0))
    y = np.array([1.0, 0.0]).reshape(2, 1)
    g = np.array([1.0, 0.0]).reshape(2, 1)
    _, _, dbeta = oracle.bn_silu_bwd(g, y, np.zeros(1), np.ones(1), np.ones(1), np.zeros(1))
    assert math.isclose(dbeta[0], s * (1 + 1.0 * (1 - s)), rel_tol=1e-14)


# --------------------------------------------------------------------------- whole block: finite differences and invariants
def _loss(x, w, gamma, beta, g, s, eps):
    return float((oracle.cbs_fwd(x, w, gamma, beta, s, eps).a * g).sum())


@pytest.mark.parametrize("k,s", [(3, 1), (3, 2), (1, 1)])
def test_block_backward_finite_differences(k, s):
    N, H, W, C, K = 2, 6, 5, 3, 4
    eps = 1e-3
    x = RNG.normal(size=(N, H, W, C)) + 0.5
    w = RNG.normal(size=(K, k, k, C)) * 0.4
    gamma = RNG.uniform(0.5, 1.5, size=K)
    beta = RNG.normal(size=K) * 0.3
    Ho, Wo = oracle.out_extent(H, k, s), oracle.out_extent(W, k, s)
    g = RNG.normal(size=(N, Ho, Wo, K))
    res = oracle.cbs_fwd_bwd(x, w, gamma, beta, g, s, eps)
    h = 1e-6
    for arr, grad in ((x, res.dx), (w, res.dw), (gamma, res.dgamma), (beta, res.dbeta)):
        for _ in range(6):
            idx = tuple(int(RNG.integers(0, d)) for d in arr.shape)
            old = arr[idx]
            arr[idx] = old + h
            lp = _loss(x, w, gamma, beta, g, s, eps)
            arr[idx] = old - h
            lm = _loss(x, w, gamma, beta, g, s, eps)
            arr[idx] = old
            fd = (lp - lm) / (2 * h)
            assert abs(fd - grad[idx]) < 2e-7 * (1 + abs(fd)), (idx, fd, grad[idx])


def test_block_backward_invariants():
    N, H, W, C, K, k, s = 2, 7, 6, 3, 4, 3, 2
    eps = 1e-3
    x = RNG.normal(size=(N, H, W, C)) + 0.7
    w = RNG.normal(size=(K, k, k, C)) * 0.3
    gamma = RNG.normal(size=K) + 1
    beta = RNG.normal(size=K)
    g = RNG.normal(size=(N, oracle.out_extent(H, k, s), oracle.out_extent(W, k, s), K))
    r = oracle.cbs_fwd_bwd(x, w, gamma, beta, g, s, eps)
    xhat = (r.y - r.mean) * r.invstd
    assert np.abs(r.dy.sum((0, 1, 2))).max() < 1e-12
    np.testing.assert_allclose((r.dy * xhat).sum((0, 1, 2)), gamma * r.dgamma * eps * r.invstd ** 3, rtol=1e-9, atol=1e-13)
    # scaling w[c'] leaves the block output unchanged except through eps: <dw[c'], w[c']> = gamma*dgamma*eps*invstd^2
    np.testing.assert_allclose((r.dw * w).sum((1, 2, 3)), gamma * r.dgamma * eps * r.invstd ** 2, rtol=1e-9, atol=1e-13)


# --------------------------------------------------------------------------- second opinion from a library (special case reduces to library routines)
def test_block_matches_torch_fp64_autograd():
    torch = pytest.importorskip("torch")
    import torch.nn.functional as F

    for (N, H, W, C, K, k, s) in [(2, 8, 7, 5, 6, 3, 1), (2, 9, 8, 4, 3, 3, 2), (3, 5, 5, 6, 4, 1, 1)]:
        x = RNG.normal(size=(N, H, W, C))
        w = RNG.normal(size=(K, k, k, C)) * 0.3
        gamma = RNG.uniform(0.5, 1.5, size=K)
        beta = RNG.normal(size=K) * 0.2
        res0 = oracle.cbs_fwd(x, w, gamma, beta, s, 1e-3)
        g = RNG.normal(size=res0.a.shape)
        rm, rv = np.zeros(K), np.ones(K)
        r = oracle.cbs_fwd(x, w, gamma, beta, s, 1e-3, rm, rv, 0.03)
        r = oracle.cbs_fwd_bwd(x, w, gamma, beta, g, s, 1e-3)
        tx = torch.tensor(x).permute(0, 3, 1, 2).contiguous().requires_grad_(True)
        tw = torch.tensor(w).permute(0, 3, 1, 2).contiguous().requires_grad_(True)
        tg, tb = torch.tensor(gamma, requires_grad=True), torch.tensor(beta, requires_grad=True)
        trm, trv = torch.zeros(K, dtype=torch.float64), torch.ones(K, dtype=torch.float64)
        ty = F.conv2d(tx, tw, stride=s, padding=k // 2)
        ta = F.silu(F.batch_norm(ty, trm, trv, tg, tb, training=True, momentum=0.03, eps=1e-3))
        (ta * torch.tensor(g).permute(0, 3, 1, 2)).sum().backward()
        np.testing.assert_allclose(r.a, ta.detach().permute(0, 2, 3, 1).numpy(), rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(r.dx, tx.grad.permute(0, 2, 3, 1).numpy(), rtol=1e-9, atol=1e-11)
        np.testing.assert_allclose(r.dw, tw.grad.permute(0, 2, 3, 1).numpy(), rtol=1e-9, atol=1e-11)
        np.testing.assert_allclose(r.dgamma, tg.grad.numpy(), rtol=1e-9, atol=1e-11)
        np.testing.assert_allclose(r.dbeta, tb.grad.numpy(), rtol=1e-9, atol=1e-11)
        np.testing.assert_allclose(rm, trm.numpy(), rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(rv, trv.numpy(), rtol=1e-12, atol=1e-14)
