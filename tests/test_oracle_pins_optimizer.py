"""Pins of the optimiser oracle (CPU only): global-norm clipping + SGD with Nesterov momentum (Sec. 3.2, Table 1).

Chosen so that a plausible slip fails one of them: clipping per tensor instead of globally, a missing 1e-6, scaling up
when the norm is small, weight decay applied after the momentum, the classical instead of the Nesterov look-ahead,
momentum buffer initialised to zero instead of to the first gradient, groups mixed up.
"""
import numpy as np
import pytest

from oracle import optimizer as opt

RNG = np.random.default_rng(20261126)


def test_clip_hand_worked():
    g = [np.array([3.0, 0.0]), np.array([[4.0]])]  # global norm 5 (per-tensor norms 3 and 4)
    out, total = opt.clip_global_norm(g, max_norm=1.0)
    assert total == pytest.approx(5.0, rel=1e-15)
    c = 1.0 / (5.0 + 1e-6)
    np.testing.assert_allclose(out[0], [3.0 * c, 0.0], rtol=1e-15)
    np.testing.assert_allclose(out[1], [[4.0 * c]], rtol=1e-15)
    # below the threshold nothing changes (never scaled up)
    out, total = opt.clip_global_norm(g, max_norm=10.0)
    np.testing.assert_array_equal(out[0], g[0])
    np.testing.assert_array_equal(out[1], g[1])
    # the norm after clipping is max_norm * total / (total + 1e-6)
    out, total = opt.clip_global_norm(g, max_norm=2.0)
    assert opt.global_norm(out) == pytest.approx(2.0 * 5.0 / (5.0 + 1e-6), rel=1e-14)


def test_nesterov_hand_worked_two_steps():
    # p = 1, g = 0.5, wd = 0.1, lr = 0.1, momentum 0.9
    # step 1: d = 0.5 + 0.1*1 = 0.6; buf = 0.6; step = 0.6 + 0.9*0.6 = 1.14; p = 1 - 0.114 = 0.886
    p, b = opt.sgd_nesterov_update(np.array([1.0]), np.array([0.5]), None, lr=0.1, momentum=0.9, weight_decay=0.1, first_step=True)
    assert p[0] == pytest.approx(0.886, rel=1e-15) and b[0] == pytest.approx(0.6, rel=1e-15)
    # step 2 with g = -0.2: d = -0.2 + 0.0886 = -0.1114; buf = 0.54 - 0.1114 = 0.4286; step = -0.1114 + 0.38574 = 0.27434
    p, b = opt.sgd_nesterov_update(p, np.array([-0.2]), b, lr=0.1, momentum=0.9, weight_decay=0.1, first_step=False)
    assert b[0] == pytest.approx(0.4286, rel=1e-13)
    assert p[0] == pytest.approx(0.886 - 0.027434, rel=1e-13)


def test_momentum_zero_is_plain_gradient_descent():
    p, g = RNG.normal(size=7), RNG.normal(size=7)
    q, _ = opt.sgd_nesterov_update(p, g, RNG.normal(size=7), lr=0.05, momentum=0.0, weight_decay=0.01, first_step=False)
    np.testing.assert_allclose(q, p - 0.05 * (g + 0.01 * p), rtol=1e-15)


def test_against_the_frameworks_cpu_optimiser_in_float64():
    torch = pytest.importorskip("torch")
    shapes = [(8, 3, 3, 4), (8,), (8,), (5, 1, 1, 8), (5,)]
    groups = [0, 1, 2, 0, 2]
    lr, wd, mom, max_norm = [0.01, 0.02, 0.1], [5e-4, 0.0, 0.0], 0.937, 0.5
    params = [RNG.normal(size=s) for s in shapes]
    tparams = [torch.tensor(p, dtype=torch.float64, requires_grad=True) for p in params]
    sgd = torch.optim.SGD(
        [{"params": [tp for tp, g in zip(tparams, groups) if g == k], "lr": lr[k], "weight_decay": wd[k]} for k in range(3)],
        lr=0.01, momentum=mom, nesterov=True)
    bufs = [None] * len(params)
    for step in range(4):
        scale = [3.0, 0.01, 1.0, 0.2][step]  # the first and third steps clip, the others do not
        grads = [RNG.normal(size=s) * scale for s in shapes]
        for tp, g in zip(tparams, grads):
            tp.grad = torch.tensor(g, dtype=torch.float64)
        tn = float(torch.nn.utils.clip_grad_norm_(tparams, max_norm))
        sgd.step()
        params, bufs, total = opt.clip_sgd_step(params, grads, bufs, groups, lr, wd, mom, max_norm, first_step=(step == 0))
        assert total == pytest.approx(tn, rel=1e-12)
        for p, tp in zip(params, tparams):
            np.testing.assert_allclose(p, tp.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_loss_scaler_against_the_frameworks_cpu_scaler():
    torch = pytest.importorskip("torch")
    shapes, groups = [(6, 4), (6,)], [0, 2]
    lr, wd, mom, max_norm = [0.05, 0.1, 0.1], [1e-3, 0.0, 0.0], 0.9, 1.0
    params = [RNG.normal(size=s) for s in shapes]
    tparams = [torch.tensor(p, dtype=torch.float64, requires_grad=True) for p in params]
    sgd = torch.optim.SGD([{"params": [tparams[0]], "lr": lr[0], "weight_decay": wd[0]}, {"params": [tparams[1]], "lr": lr[2], "weight_decay": wd[2]}],
                          lr=0.1, momentum=mom, nesterov=True)
    scaler = torch.amp.GradScaler("cpu", init_scale=1024.0, growth_factor=2.0, backoff_factor=0.5, growth_interval=2)
    scale, tracker, bufs, first = 1024.0, 0, [None, None], True
    for step in range(7):
        grads = [RNG.normal(size=s) * scale for s in shapes]  # what the backward pass of a scaled loss delivers
        if step in (1, 4):
            grads[0][2, 1] = np.inf if step == 1 else np.nan
        scaler.scale(torch.tensor(1.0))
        for tp, g in zip(tparams, grads):
            tp.grad = torch.tensor(g, dtype=torch.float64)
        scaler.unscale_(sgd)
        torch.nn.utils.clip_grad_norm_(tparams, max_norm)
        scaler.step(sgd)
        scaler.update()
        params, bufs, total, scale, tracker, skipped = opt.scaled_clip_sgd_step(params, grads, bufs, groups, lr, wd, mom, max_norm, first, scale, tracker,
                                                                                 2.0, 0.5, 2, floor=0.0)
        if not skipped:
            first = False
        assert skipped == (step in (1, 4))
        assert scale == scaler.get_scale() and tracker == int(scaler._growth_tracker)
        for p, tp in zip(params, tparams):
            np.testing.assert_allclose(p, tp.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_loss_scaler_floor_and_hand_sequence():
    p, g = [np.array([1.0])], [np.array([np.inf])]
    scale, tracker = 4.0, 1
    for want in (2.0, 1.5, 1.5):  # halves until the floor 1.5 holds it
        p2, _, total, scale, tracker, skipped = opt.scaled_clip_sgd_step(p, g, [None], [0], [0.1] * 3, [0.0] * 3, 0.9, 10.0, True, scale, tracker, floor=1.5)
        assert skipped and scale == want and tracker == 0 and p2[0][0] == 1.0 and not np.isfinite(total)
    # a good step with scale 8: gradient 16 means 2; lr 0.1, no momentum history: p = 1 - 0.1*(2 + 0.9*2) = 0.62
    p2, b2, total, scale, tracker, skipped = opt.scaled_clip_sgd_step([np.array([1.0])], [np.array([16.0])], [None], [0], [0.1] * 3, [0.0] * 3, 0.9, 10.0, True,
                                                                      8.0, 0, growth_interval=1)
    assert not skipped and total == pytest.approx(2.0) and p2[0][0] == pytest.approx(0.62) and scale == 16.0 and tracker == 0
