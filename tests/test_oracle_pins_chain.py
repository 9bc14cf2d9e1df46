"""Pins of the chained-block oracle (CPU only): the C2f unit's forward and backward, composed from the single-block
oracle (pinned elsewhere) with numpy slicing.  What can go wrong here is the wiring: which part feeds which block, the
shortcut, and the accumulation of gradients where a tensor has several consumers -- central finite differences of the
whole unit catch all of it."""
import numpy as np
import pytest

import oracle
from oracle import chain

RNG = np.random.default_rng(20261127)
EPS = 1e-3


def _params(c1, c2, n):
    c = c2 // 2
    shapes = [(2 * c, 1, 1, c1)] + [(c, 3, 3, c)] * (2 * n) + [(c2, 1, 1, (2 + n) * c)]
    return [chain.BlockParams(RNG.normal(size=s) * 0.5, RNG.uniform(0.5, 1.5, s[0]), RNG.normal(size=s[0]) * 0.1) for s in shapes]


@pytest.mark.parametrize("n,shortcut", [(1, True), (2, True), (2, False)])
def test_whole_unit_finite_differences(n, shortcut):
    x = RNG.normal(size=(2, 4, 3, 4))
    prm = _params(4, 4, n)
    G = RNG.normal(size=(2, 4, 3, 4))
    res = chain.c2f_fwd_bwd(x, prm, n, shortcut, EPS, G)
    loss = lambda xx, pp: float((chain.c2f_fwd_bwd(xx, pp, n, shortcut, EPS).out * G).sum())
    h = 1e-5
    for idx in [(0, 0, 0, 0), (1, 3, 2, 3), (0, 2, 1, 1)]:
        xp, xm = x.copy(), x.copy()
        xp[idx] += h
        xm[idx] -= h
        fd = (loss(xp, prm) - loss(xm, prm)) / (2 * h)
        assert res.dx[idx] == pytest.approx(fd, rel=2e-5, abs=1e-7)
    # one filter tap, one gain and one shift of every block
    for b in range(len(prm)):
        for name, slot in (("w", 0), ("gamma", 1), ("beta", 2)):
            arr = getattr(prm[b], name)
            idx = tuple(int(RNG.integers(0, d)) for d in arr.shape)
            saved = arr[idx]
            arr[idx] = saved + h
            lp = loss(x, prm)
            arr[idx] = saved - h
            lm = loss(x, prm)
            arr[idx] = saved
            assert res.grads[b][slot][idx] == pytest.approx((lp - lm) / (2 * h), rel=2e-5, abs=1e-7), (b, name)


def test_no_bottlenecks_is_two_blocks_in_sequence():
    x = RNG.normal(size=(2, 5, 4, 6))
    prm = _params(6, 8, 0)
    G = RNG.normal(size=(2, 5, 4, 8))
    res = chain.c2f_fwd_bwd(x, prm, 0, True, EPS, G)
    first = oracle.cbs_fwd(x, prm[0].w, prm[0].gamma, prm[0].beta, 1, EPS)
    second = oracle.cbs_fwd_bwd(first.a, prm[1].w, prm[1].gamma, prm[1].beta, G, 1, EPS)
    np.testing.assert_allclose(res.out, second.a, rtol=1e-13)
    np.testing.assert_allclose(res.grads[1][0], second.dw, rtol=1e-12, atol=1e-14)
    back = oracle.bn_silu_bwd(second.dx, first.y, first.mean, first.invstd, prm[0].gamma, prm[0].beta)
    np.testing.assert_allclose(res.dx, oracle.conv_dgrad(back[0], prm[0].w, x.shape, 1), rtol=1e-11, atol=1e-13)


def test_shortcut_adds_the_bottleneck_input():
    x = RNG.normal(size=(1, 4, 4, 4))
    prm = _params(4, 4, 1)
    with_sc = chain.c2f_fwd_bwd(x, prm, 1, True, EPS)
    without = chain.c2f_fwd_bwd(x, prm, 1, False, EPS)
    np.testing.assert_allclose(with_sc.parts[2] - without.parts[2], with_sc.parts[1], rtol=1e-13, atol=1e-15)
    assert len(with_sc.parts) == 3 and with_sc.parts[0].shape[-1] == 2


def test_maxpool5_against_brute_force_and_library_filter():
    from scipy.ndimage import maximum_filter

    x = RNG.normal(size=(2, 7, 6, 3))
    y, idx = chain.maxpool5(x)
    # library routine: a 5x5 maximum filter over H and W with -inf outside
    want = maximum_filter(x, size=(1, 5, 5, 1), mode="constant", cval=-np.inf)
    np.testing.assert_array_equal(y, want)
    # brute force incl. the index convention
    for n, p, q, c in [(0, 0, 0, 0), (1, 6, 5, 2), (0, 3, 2, 1), (1, 0, 5, 0)]:
        best, bi = -np.inf, -1
        for r in range(5):
            for t in range(5):
                h, w = p - 2 + r, q - 2 + t
                if 0 <= h < 7 and 0 <= w < 6 and x[n, h, w, c] > best:
                    best, bi = x[n, h, w, c], r * 5 + t
        assert y[n, p, q, c] == best and idx[n, p, q, c] == bi


def test_maxpool5_ties_go_to_the_first_element_and_gradient_is_the_adjoint():
    x = np.zeros((1, 5, 5, 1))  # all equal: every window's first in-bounds element wins
    y, idx = chain.maxpool5(x)
    assert idx[0, 2, 2, 0] == 0 and idx[0, 0, 0, 0] == 2 * 5 + 2
    g = RNG.normal(size=(2, 6, 5, 4))
    x = RNG.normal(size=(2, 6, 5, 4))
    y, idx = chain.maxpool5(x)
    dx = chain.maxpool5_bwd(g, idx)
    assert dx.sum() == pytest.approx(g.sum(), rel=1e-12)
    # directional derivative: moving x by a small v changes sum(y*g) by <dx, v> (no ties in random data)
    v = RNG.normal(size=x.shape)
    h = 1e-7
    fd = ((chain.maxpool5(x + h * v)[0] - chain.maxpool5(x - h * v)[0]) * g).sum() / (2 * h)
    assert (dx * v).sum() == pytest.approx(fd, rel=1e-6)


def test_upsample2_and_its_adjoint():
    x = RNG.normal(size=(2, 3, 4, 5))
    y = chain.upsample2(x)
    assert y.shape == (2, 6, 8, 5)
    for a in (0, 1):
        for b in (0, 1):
            np.testing.assert_array_equal(y[:, a::2, b::2, :], x)
    g = RNG.normal(size=y.shape)
    assert (chain.upsample2_bwd(g) * x).sum() == pytest.approx((g * y).sum(), rel=1e-12)


def test_sppf_unit_finite_differences():
    x = RNG.normal(size=(1, 6, 6, 4))
    prm = [chain.BlockParams(RNG.normal(size=(2, 1, 1, 4)) * 0.7, RNG.uniform(0.5, 1.5, 2), RNG.normal(size=2) * 0.1),
           chain.BlockParams(RNG.normal(size=(4, 1, 1, 8)) * 0.5, RNG.uniform(0.5, 1.5, 4), RNG.normal(size=4) * 0.1)]
    G = RNG.normal(size=(1, 6, 6, 4))
    out, parts, dx, grads = chain.sppf_fwd_bwd(x, prm, EPS, G)
    assert len(parts) == 4 and out.shape == G.shape
    loss = lambda xx: float((chain.sppf_fwd_bwd(xx, prm, EPS)[0] * G).sum())
    h = 1e-6
    for idx in [(0, 0, 0, 0), (0, 3, 2, 1), (0, 5, 5, 3)]:
        xp, xm = x.copy(), x.copy()
        xp[idx] += h
        xm[idx] -= h
        assert dx[idx] == pytest.approx((loss(xp) - loss(xm)) / (2 * h), rel=1e-4, abs=1e-7)
    w = prm[0].w
    saved = w[1, 0, 0, 2]
    w[1, 0, 0, 2] = saved + h
    lp = loss(x)
    w[1, 0, 0, 2] = saved - h
    lm = loss(x)
    w[1, 0, 0, 2] = saved
    assert grads[0][0][1, 0, 0, 2] == pytest.approx((lp - lm) / (2 * h), rel=1e-4, abs=1e-7)


def test_round_bf16_is_nearest_even_on_known_values():
    # 1 + 2^-8 lies halfway between 1 and 1 + 2^-7: ties go to the even mantissa (1.0); 1 + 3*2^-8 goes up to 1 + 2^-6
    vals = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -2.5, 0.0, 3.0e-5])
    got = chain.round_bf16(vals)
    assert got[0] == 1.0 and got[1] == 1.0 and got[2] == 1.0 + 2.0 ** -6 and got[3] == 1.0 + 2.0 ** -7 and got[4] == -2.5 and got[5] == 0.0
    assert abs(got[6] - 3.0e-5) <= 3.0e-5 * 2.0 ** -8
    assert np.array_equal(chain.round_bf16(got), got)


def _detector_params(layers):
    return [chain.BlockParams(RNG.uniform(-1, 1, (s.c_out, s.k, s.k, s.c_in)) / np.sqrt(s.c_in * s.k * s.k) * 1.7,
                              RNG.uniform(0.5, 1.5, s.c_out), RNG.normal(size=s.c_out) * 0.1) for s in layers]


def test_graph_interpreter_reproduces_the_c2f_unit():
    # the same unit written twice: once by hand (c2f_fwd_bwd, pinned by finite differences above), once as a graph
    from paper_2609_10632_b200 import workloads as wl

    c, n = 2, 2
    layers = [wl.ConvShape("cv1", 2, 4, 3, 4, 2 * c, 1, 1)] + [wl.ConvShape(f"m{i}", 2, 4, 3, c, c, 3, 1) for i in range(2 * n)]
    layers.append(wl.ConvShape("cv2", 2, 4, 3, (2 + n) * c, 4, 1, 1))
    ops = [{"out": "a0", "op": "cbs", "ins": ["img"], "layer": 0},
           {"out": "p0", "op": "slice", "ins": ["a0"], "c0": 0, "c1": c}, {"out": "p1", "op": "slice", "ins": ["a0"], "c0": c, "c1": 2 * c}]
    parts = ["p0", "p1"]
    for i in range(n):
        ops += [{"out": f"u{i}", "op": "cbs", "ins": [parts[-1]], "layer": 1 + 2 * i}, {"out": f"v{i}", "op": "cbs", "ins": [f"u{i}"], "layer": 2 + 2 * i},
                {"out": f"p{2 + i}", "op": "add", "ins": [parts[-1], f"v{i}"]}]
        parts.append(f"p{2 + i}")
    ops += [{"out": "cat", "op": "concat", "ins": parts}, {"out": "out", "op": "cbs", "ins": ["cat"], "layer": 1 + 2 * n}]
    prm = _params(4, 4, n)
    x, G = RNG.normal(size=(2, 4, 3, 4)), RNG.normal(size=(2, 4, 3, 4))
    want = chain.c2f_fwd_bwd(x, prm, n, True, EPS, G)
    T, grads, bg = chain.graph_fwd_bwd(ops, layers, prm, x, EPS, {"out": G})
    np.testing.assert_allclose(T["out"], want.out, rtol=1e-13)
    np.testing.assert_allclose(grads["img"], want.dx, rtol=1e-11, atol=1e-13)
    for k in range(len(prm)):
        for a, b in zip(bg[k], want.grads[k]):
            np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-13)


def test_detector_graph_finite_differences_at_a_tiny_size():
    """The whole detector dataflow (77 blocks, splits, adds, concats, three pools, two upsamplings) at batch 2, 64 x 64
    (the coarsest level is then 2 x 2: batch statistics over 8 values; over the 2 values of a 32 x 32 image BN degenerates
    to a sign function and finite differences stop being meaningful):
    directional derivative with respect to the image and single-entry derivatives of a few filters in different places
    (backbone behind the pools, neck, head) against central differences of sum(outputs * G)."""
    from paper_2609_10632_b200 import workloads as wl

    ops, layers, outs, plain = wl.detector_graph(2, 64, plain_head=True)  # up to the raw head outputs
    prm = _detector_params(layers)
    pprm = [(RNG.uniform(-1, 1, (s.c_out, 1, 1, s.c_in)) / np.sqrt(s.c_in), RNG.normal(size=s.c_out) * 0.5) for s in plain]
    kw = dict(plain_layers=plain, plain_params=pprm)
    x = RNG.uniform(0, 1, (2, 64, 64, 3))
    T = chain.graph_fwd_bwd(ops, layers, prm, x, EPS, **kw)[0]
    Gs = {name: RNG.normal(size=T[name].shape) for name in outs}
    T, grads, bg, pg = chain.graph_fwd_bwd(ops, layers, prm, x, EPS, Gs, **kw)
    assert all(g is not None for g in bg) and all(g is not None for g in pg)

    def loss(xx):
        TT = chain.graph_fwd_bwd(ops, layers, prm, xx, EPS, **kw)[0]
        return float(sum((TT[n] * Gs[n]).sum() for n in outs))

    v = RNG.normal(size=x.shape)
    h = 1e-6
    fd = (loss(x + h * v) - loss(x - h * v)) / (2 * h)
    assert float((grads["img"] * v).sum()) == pytest.approx(fd, rel=2e-4)
    names = [s.name for s in layers]
    for lname in ("b2.c2f.m1.cv1", "b8.c2f.cv2", "b9.sppf.cv1", "n12.c2f.m0.cv2", "n18.c2f.cv1", "h22.cls1.0"):
        k = names.index(lname)
        w = prm[k].w
        idx = tuple(int(RNG.integers(0, d)) for d in w.shape)
        saved = w[idx]
        hh = 1e-5
        w[idx] = saved + hh
        lp = loss(x)
        w[idx] = saved - hh
        lm = loss(x)
        w[idx] = saved
        assert bg[k][0][idx] == pytest.approx((lp - lm) / (2 * hh), rel=5e-4, abs=1e-6), lname

    # a plain head convolution: one filter entry and one bias entry
    w, b = pprm[3]
    for arr, grad, idx in ((w, pg[3][0], (5, 0, 0, 7)), (b, pg[3][1], (11,))):
        saved = arr[idx]
        arr[idx] = saved + 1e-5
        lp = loss(x)
        arr[idx] = saved - 1e-5
        lm = loss(x)
        arr[idx] = saved
        assert grad[idx] == pytest.approx((lp - lm) / 2e-5, rel=5e-4, abs=1e-6)


def test_storage_rounding_mode_stays_close_to_the_exact_graph_on_a_shallow_unit():
    # the 16-bit storage mode only rounds stored tensors: on one C2f unit it must agree with the exact graph to bf16 accuracy,
    # every stored activation must be exactly representable in bf16, and the exact mode must be untouched by the flag's code
    from paper_2609_10632_b200 import workloads as wl

    c, n = 4, 1
    layers = [wl.ConvShape("cv1", 2, 6, 5, 8, 2 * c, 1, 1), wl.ConvShape("m0", 2, 6, 5, c, c, 3, 1), wl.ConvShape("m1", 2, 6, 5, c, c, 3, 1),
              wl.ConvShape("cv2", 2, 6, 5, 3 * c, 8, 1, 1)]
    ops = [{"out": "a0", "op": "cbs", "ins": ["img"], "layer": 0},
           {"out": "p0", "op": "slice", "ins": ["a0"], "c0": 0, "c1": c}, {"out": "p1", "op": "slice", "ins": ["a0"], "c0": c, "c1": 2 * c},
           {"out": "u", "op": "cbs", "ins": ["p1"], "layer": 1}, {"out": "v", "op": "cbs", "ins": ["u"], "layer": 2},
           {"out": "p2", "op": "add", "ins": ["p1", "v"]}, {"out": "cat", "op": "concat", "ins": ["p0", "p1", "p2"]},
           {"out": "out", "op": "cbs", "ins": ["cat"], "layer": 3}]
    prm = _params(8, 8, n)
    x = chain.round_bf16(RNG.normal(size=(2, 6, 5, 8)))
    G = chain.round_bf16(RNG.normal(size=(2, 6, 5, 8)))
    T0, G0, b0 = chain.graph_fwd_bwd(ops, layers, prm, x, EPS, {"out": G})
    T1, G1, b1 = chain.graph_fwd_bwd(ops, layers, prm, x, EPS, {"out": G}, storage_16bit=True)
    for name in ("a0", "v", "p2", "out"):
        assert np.array_equal(chain.round_bf16(T1[name]), T1[name]), name
        assert np.linalg.norm(T1[name] - T0[name]) <= 1e-2 * np.linalg.norm(T0[name]), name
    assert np.array_equal(chain.round_bf16(G1["img"]), G1["img"])
    assert np.linalg.norm(G1["img"] - G0["img"]) <= 3e-2 * np.linalg.norm(G0["img"])
    for k in range(4):
        assert np.linalg.norm(b1[k][0] - b0[k][0]) <= 3e-2 * np.linalg.norm(b0[k][0])
