"""Pins of the oracle's evaluation-mode and plain variants (CPU only): evaluation-mode BN with running statistics
(Table 2 row 9), convolution + bias without normalisation (the head of Table 2 row 3), BN folded into the filter.

Each pin is a value or an identity fixed outside the function under test, chosen so that a plausible slip (eps inside
or outside the root, variance used as a standard deviation, mean not subtracted, bias indexed by pixel, fold scaling the
wrong filter axis, sign of the folded bias) fails at least one of them.  Nothing here uses the CUDA library.
"""
import math

import numpy as np
import pytest
from scipy.signal import correlate2d

import oracle

RNG = np.random.default_rng(20261125)


def test_eval_bn_hand_worked_value():
    # y = 2, running mean 1, running variance 3, eps 1: xhat = (2-1)/sqrt(4) = 1/2; gamma 4, beta -1: z = 1; SiLU(1) = 1/(1+e^-1)
    y = np.full((1, 1, 1, 1), 2.0)
    one = lambda v: np.array([v], dtype=np.float64)
    a = oracle.bn_eval_act(y, one(4.0), one(-1.0), one(1.0), one(3.0), eps=1.0, act=True)
    assert a.item() == pytest.approx(1.0 / (1.0 + math.exp(-1.0)), rel=1e-15)
    z = oracle.bn_eval_act(y, one(4.0), one(-1.0), one(1.0), one(3.0), eps=1.0, act=False)
    assert z.item() == pytest.approx(1.0, rel=1e-15)
    # eps inside the root and added to the variance (not to the standard deviation): variance 0, eps 1/4 -> divide by 1/2
    z = oracle.bn_eval_act(y, one(1.0), one(0.0), one(0.0), one(0.0), eps=0.25, act=False)
    assert z.item() == pytest.approx(4.0, rel=1e-15)


def test_eval_bn_per_channel_values_against_numpy_broadcast():
    y = RNG.normal(size=(2, 3, 4, 5))
    gamma, beta = RNG.uniform(0.5, 1.5, 5), RNG.normal(size=5)
    rm, rv = RNG.normal(size=5), RNG.uniform(0.2, 3.0, 5)
    z = oracle.bn_eval_act(y, gamma, beta, rm, rv, eps=1e-3, act=False)
    want = (y - rm[None, None, None, :]) / np.sqrt(rv + 1e-3)[None, None, None, :] * gamma + beta
    np.testing.assert_allclose(z, want, rtol=1e-14, atol=1e-14)
    a = oracle.bn_eval_act(y, gamma, beta, rm, rv, eps=1e-3, act=True)
    np.testing.assert_allclose(a, want / (1.0 + np.exp(-want)), rtol=1e-14, atol=1e-14)


def test_eval_bn_with_batch_statistics_reproduces_the_training_forward():
    # the training-mode forward (pinned elsewhere) normalises with the batch mean and the biased batch variance:
    # handing exactly those to the evaluation-mode function must give the same activations
    x = RNG.normal(size=(2, 6, 5, 4))
    w = RNG.normal(size=(8, 3, 3, 4)) * 0.3
    gamma, beta = RNG.uniform(0.5, 1.5, 8), RNG.normal(size=8) * 0.1
    tr = oracle.cbs_fwd(x, w, gamma, beta, stride=1, eps=1e-3)
    ev = oracle.cbs_infer(x, w, gamma, beta, tr.mean, tr.var, stride=1, eps=1e-3)
    np.testing.assert_allclose(ev, tr.a, rtol=1e-12, atol=1e-13)
    # and it must NOT depend on the batch: a second batch with the same statistics handed in gives per-pixel the same map
    x2 = np.concatenate([x, RNG.normal(size=(1, 6, 5, 4))], axis=0)
    ev2 = oracle.cbs_infer(x2, w, gamma, beta, tr.mean, tr.var, stride=1, eps=1e-3)
    np.testing.assert_array_equal(ev2[:2], ev)


def test_eval_bn_limits():
    y = RNG.normal(size=(1, 4, 4, 3)) * 5
    beta = np.array([0.3, -2.0, 1.5])
    silu = lambda z: z / (1.0 + np.exp(-z))
    # gamma = 0: every output is SiLU(beta_c)
    a = oracle.bn_eval_act(y, np.zeros(3), beta, RNG.normal(size=3), np.ones(3), eps=1e-3, act=True)
    np.testing.assert_allclose(a, np.broadcast_to(silu(beta), a.shape), rtol=1e-15)
    # a huge running variance flattens the input the same way
    a = oracle.bn_eval_act(y, np.ones(3), beta, np.zeros(3), np.full(3, 1e300), eps=1e-3, act=True)
    np.testing.assert_allclose(a, np.broadcast_to(silu(beta), a.shape), rtol=1e-12)


@pytest.mark.parametrize("k,stride", [(1, 1), (3, 1), (3, 2)])
def test_conv_bias_against_library_correlation(k, stride):
    N, H, W, Cin, Cout = 2, 7, 6, 3, 4
    x = RNG.normal(size=(N, H, W, Cin))
    w = RNG.normal(size=(Cout, k, k, Cin))
    bias = np.array([0.5, -1.25, 2.0, 0.0])  # distinct per channel: an index slip shows
    got = oracle.conv_bias_act(x, w, bias, stride, act=False)
    P = k // 2
    for n in range(N):
        for co in range(Cout):
            full = sum(correlate2d(np.pad(x[n, :, :, c], P), w[co, :, :, c], mode="valid") for c in range(Cin))
            np.testing.assert_allclose(got[n, :, :, co], full[::stride, ::stride] + bias[co], rtol=1e-12, atol=1e-12)
    # no bias == zero bias; with the activation it is SiLU of the same numbers
    np.testing.assert_array_equal(oracle.conv_bias_act(x, w, None, stride), oracle.conv_bias_act(x, w, np.zeros(Cout), stride))
    np.testing.assert_allclose(oracle.conv_bias_act(x, w, bias, stride, act=True), got / (1.0 + np.exp(-got)), rtol=1e-14, atol=1e-15)


def test_fold_hand_worked_values():
    # one output channel, two taps: gamma 3, variance 8, eps 1 -> s = 3/sqrt(9) = 1; mean 2, beta 5 -> bias' = 5 - 2*1 = 3
    w = np.array([[[[0.5, -4.0]]]])
    wf, bf = oracle.bn_fold(w, [3.0], [5.0], [2.0], [8.0], eps=1.0)
    np.testing.assert_allclose(wf, w, rtol=1e-15)
    assert bf[0] == pytest.approx(3.0, rel=1e-15)
    # s = 6/sqrt(4) = 3: every tap of that output channel triples, the others keep their own scale
    w = RNG.normal(size=(2, 3, 3, 2))
    wf, bf = oracle.bn_fold(w, [6.0, 1.0], [0.0, 0.5], [1.0, -1.0], [3.0, 0.0], eps=1.0)
    np.testing.assert_allclose(wf[0], 3.0 * w[0], rtol=1e-15)
    np.testing.assert_allclose(wf[1], w[1], rtol=1e-15)
    np.testing.assert_allclose(bf, [-3.0, 1.5], rtol=1e-15)


@pytest.mark.parametrize("k,stride", [(1, 1), (3, 1), (3, 2)])
def test_folded_convolution_equals_the_evaluation_mode_block(k, stride):
    x = RNG.normal(size=(2, 9, 8, 5))
    w = RNG.normal(size=(6, k, k, 5)) * 0.4
    gamma, beta = RNG.uniform(0.5, 1.5, 6), RNG.normal(size=6) * 0.2
    rm, rv = RNG.normal(size=6) * 0.5, RNG.uniform(0.3, 2.0, 6)
    want = oracle.cbs_infer(x, w, gamma, beta, rm, rv, stride, eps=1e-3, act=True)
    wf, bf = oracle.bn_fold(w, gamma, beta, rm, rv, eps=1e-3)
    got = oracle.conv_bias_act(x, wf, bf, stride, act=True)
    np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-12)


def test_conv_bias_backward_is_the_adjoint_of_the_forward():
    x = RNG.normal(size=(2, 6, 5, 3))
    w = RNG.normal(size=(4, 3, 3, 3))
    bias = RNG.normal(size=4)
    g = RNG.normal(size=(2, 3, 3, 4))
    dx, dw, db = oracle.conv_bias_bwd(x, w, g, 2)
    loss = lambda xx, ww, bb: float((oracle.conv_bias_act(xx, ww, bb, 2) * g).sum())
    h = 1e-6
    for arr, grad in ((x, dx), (w, dw), (bias, db)):
        idx = tuple(int(RNG.integers(0, d)) for d in arr.shape)
        saved = arr[idx]
        arr[idx] = saved + h
        lp = loss(x, w, bias)
        arr[idx] = saved - h
        lm = loss(x, w, bias)
        arr[idx] = saved
        assert grad[idx] == pytest.approx((lp - lm) / (2 * h), rel=1e-7, abs=1e-9)
    np.testing.assert_allclose(db, g.sum(axis=(0, 1, 2)), rtol=1e-14)
