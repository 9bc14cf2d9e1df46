"""Seeded random layer shapes through every call of the block against the fp64 oracle, and through the options of a
chained network against the dense run.

The hand-picked shapes of test_gpu_parity.py aim at the tile boundaries known to the author; this file draws shapes
without knowing them: 96 layers with 1-3 images of 2..69 x 2..69 pixels, 8..384 channels on either side, 1x1 and 3x3,
stride 1 and 2, at least 32 output pixels.  Each goes through the training step (forward, data gradient, weight
gradient), the inference call and the bias-head calls (forward and backward), in bf16 and in fp16 operand mode, at the
bars of the hand-picked shapes.

One reading, for the data gradient of a 1x1 stride-2 layer only: three of four input pixels receive no gradient.  They
must be exactly zero, and the per-element bar is taken relative to the rms of the pixels that do receive one (the zeros
would halve the rms and with it the bar, which is defined for a dense tensor)."""
import numpy as np
import pytest

import oracle
from paper_2609_10632_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

EPS = 1e-3
CHANNELS_IN = [8, 16, 24, 32, 40, 48, 64, 80, 96, 112, 128, 144, 160, 192, 224, 256, 288, 320, 384]
CHANNELS_OUT = [8, 16, 24, 32, 48, 64, 80, 96, 128, 144, 160, 192, 256, 288, 320, 384]


def _draw(rs):
    while True:
        n, h, w = int(rs.randint(1, 4)), int(rs.randint(2, 70)), int(rs.randint(2, 70))
        k, s = int(rs.choice([1, 3])), int(rs.choice([1, 2]))
        ci, co = int(rs.choice(CHANNELS_IN)), int(rs.choice(CHANNELS_OUT))
        m = n * oracle.out_extent(h, k, s) * oracle.out_extent(w, k, s)
        if m < 32 or m * k * k * ci * co > 1.5e9:
            continue
        return wl.ConvShape(f"r{n}x{h}x{w}x{ci}->{co}k{k}s{s}", n, h, w, ci, co, k, s, False)


def _shapes(seed, count):
    rs = np.random.RandomState(seed)
    return [_draw(rs) for _ in range(count)]


def _check_dx(name, got, ref, shape):
    if shape.k == 1 and shape.stride == 2:
        hit = np.zeros(ref.shape, dtype=bool)
        hit[:, ::2, ::2, :] = True
        assert not got[~hit].any() and not ref[~hit].any(), f"{name}: a pixel outside the stride-2 grid received a gradient"
        sel = lambda t: t[:, ::2, ::2, :]
        parity.check(name, sel(got), sel(ref), "bf16")
    else:
        parity.check(name, got, ref, "bf16")


@pytest.mark.parametrize("mode_name,seed", [("bf16", 101), ("fp16", 202)])
def test_random_shapes_match_oracle(mode_name, seed):
    import torch

    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200.block import CbsBlock

    mode = nb.NB_MODE_BF16_TC if mode_name == "bf16" else nb.NB_MODE_F16_TC
    paths = set()
    for i, shape in enumerate(_shapes(seed, 48)):
        inp = wl.make_inputs(shape, 31, i, bf16=True, affine="random")
        blk = CbsBlock(shape, mode=mode, eps=EPS)
        blk.upload(inp)
        blk.step()
        blk.poll()
        out = blk.download()
        ref = oracle.cbs_fwd_bwd(inp.x, inp.w, inp.gamma, inp.beta, inp.g, shape.stride, EPS)
        try:
            parity.check_stats(out["mean"], out["invstd"], ref.y, EPS, "bf16")
            for name in ("a", "dgamma", "dbeta", "dw", "y", "dy"):
                parity.check(name, out[name], getattr(ref, name), "bf16")
            _check_dx("dx", out["dx"], ref.dx, shape)

            rm, rv, bias = wl.make_eval_stats(shape, 31, i)
            up = lambda a: torch.from_numpy(a).to(blk.dev)
            o = torch.empty_like(blk.a)
            ws = torch.empty(max(blk.plan.infer_bytes, blk.plan.bwd_bytes, 256), dtype=torch.uint8, device=blk.dev)
            nb.nb_conv_bn_silu_infer(blk.plan, blk.x, blk.w, blk.gamma, blk.beta, up(rm), up(rv), o, ws)
            torch.cuda.synchronize()
            want = oracle.cbs_infer(inp.x, inp.w, inp.gamma, inp.beta, rm, rv, shape.stride, EPS)
            parity.check("a_eval", o.double().cpu().numpy(), want, "bf16")

            nb.nb_conv_bias_act(blk.plan, blk.x, blk.w, up(bias), 0, o, ws)
            dx, dw = torch.empty_like(blk.x), torch.empty_like(blk.dw)
            db = torch.empty(shape.c_out, dtype=torch.float32, device=blk.dev)
            nb.nb_conv_bias_bwd(blk.plan, blk.x, blk.w, blk.g, dx, dw, db, ws)
            torch.cuda.synchronize()
            blk.poll()
            parity.check("head out", o.double().cpu().numpy(), oracle.conv_bias_act(inp.x, inp.w, bias, shape.stride), "bf16")
            rdx, rdw, rdb = oracle.conv_bias_bwd(inp.x, inp.w, inp.g, shape.stride)
            _check_dx("head dx", dx.double().cpu().numpy(), rdx, shape)
            parity.check("head dw", dw.double().cpu().numpy(), rdw, "bf16")
            parity.check("head dbias", db.double().cpu().numpy(), rdb, "bf16")
        except AssertionError as e:
            raise AssertionError(f"{shape.name} (shape {i} of seed {seed}, paths {blk.plan.paths}): {e}") from None
        paths.add((blk.plan.paths["fprop"], blk.plan.paths["dgrad"], blk.plan.paths["wgrad"]))
    # the draw reaches the tensor-core kernels, the CUDA-core fallback and the mixed case (tensor-core forward and weight
    # gradient beside a CUDA-core data gradient)
    assert {(1, 1, 1), (0, 0, 0), (1, 0, 1)} <= paths, paths


def test_random_shapes_with_every_chain_option_give_the_dense_bits():
    """The options a chained network uses (x, a_out and g as channel slices of wider tensors; a residual added in the
    forward pass; the incoming gradient handed to the shortcut; the data gradient written or added into a slice of a
    wider buffer) switched on in random combinations with random pitches and offsets on 64 random shapes.  None of them
    changes the arithmetic, so everything the calls write equals the dense run's bits; the sums are the fp32 sum of two
    16-bit values rounded once (checked exactly); the block output with a residual is held to the oracle's bars; and
    nothing beside a slice may change.  A plan that cannot take an option says NB_ERR_UNSUPPORTED and runs without it."""
    import torch

    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200.block import CbsBlock

    rs = np.random.RandomState(303)
    used = dict(x_pitch=0, res=0, gres=0, dx_target=0, dx_add=0)
    for i in range(64):
        s = _draw(rs)
        inp = wl.make_inputs(s, 33, i, bf16=True, affine="random")
        dense = CbsBlock(s, eps=EPS)
        dense.upload(inp)
        dense.step()
        dense.poll()
        blk = CbsBlock(s, eps=EPS)
        blk.upload(inp)
        dev = blk.dev
        gen = torch.Generator(device=dev)
        gen.manual_seed(303000 + i)
        pad = lambda: 8 * int(rs.randint(0, 6))
        off = {k: pad() for k in "xagrqd"}
        ld = {k: (s.c_in if k in "xd" else s.c_out) + off[k] + pad() for k in "xagrqd"}
        try:
            blk.plan.set_pitches(ld_x=ld["x"], ld_a=ld["a"], ld_g=ld["g"])
            used["x_pitch"] += 1
        except nb.NbError as e:  # the CUDA-core forward reads a dense x
            assert e.status == nb.NB_ERR_UNSUPPORTED
            off["x"], ld["x"] = 0, s.c_in
            blk.plan.set_pitches(ld_x=0, ld_a=ld["a"], ld_g=ld["g"])
        mk = lambda h, w, c: torch.randn(s.n, h, w, c, generator=gen, device=dev).to(torch.bfloat16)
        X, D = mk(s.h, s.w, ld["x"]), mk(s.h, s.w, ld["d"])
        A, G, R, Q = (mk(s.ho, s.wo, ld[k]) for k in "agrq")
        cut = lambda t, k: t[..., off[k]:off[k] + (s.c_in if k in "xd" else s.c_out)]
        cut(X, "x").copy_(blk.x)
        cut(G, "g").copy_(blk.g)
        A0, Q0, D0 = A.clone(), Q.clone(), D.clone()
        with_res, with_gres, gres_add = rs.rand() < 0.6, rs.rand() < 0.6, bool(rs.rand() < 0.5)
        dx_target, dx_add = rs.rand() < 0.7, bool(rs.rand() < 0.5)
        if with_res:
            blk.plan.set_fwd_residual(cut(R, "r"), ld["r"])
            used["res"] += 1
        if with_gres:
            blk.plan.set_bwd_residual(cut(Q, "q"), ld["q"], accumulate=gres_add)
            used["gres"] += 1
        if dx_target:
            try:
                blk.plan.set_dx_target(ld_dx=ld["d"], accumulate=dx_add)
                used["dx_target"] += 1
                used["dx_add"] += dx_add
            except nb.NbError as e:  # only the bulk-store epilogue of the stride-1 tensor-core data gradient can
                assert e.status == nb.NB_ERR_UNSUPPORTED
                dx_target = False
        first = lambda t, k: t.data_ptr() + off[k] * t.element_size()
        nb.nb_conv_bn_silu_fwd(blk.plan, first(X, "x"), blk.w, blk.gamma, blk.beta, None, None, blk.y, blk.mean, blk.invstd, first(A, "a"), blk.ws)
        nb.nb_conv_bn_silu_bwd_data(blk.plan, first(G, "g"), blk.y, blk.mean, blk.invstd, blk.gamma, blk.beta, blk.w,
                                    first(D, "d") if dx_target else blk.dx, blk.dgamma, blk.dbeta, blk.dy, blk.ws)
        nb.nb_conv_bn_silu_bwd_weight(blk.plan, first(X, "x"), blk.dy, blk.dw, blk.ws)
        torch.cuda.synchronize()
        blk.poll()

        def beside_untouched(t, t0, k):
            c = s.c_in if k in "xd" else s.c_out
            return torch.equal(t[..., :off[k]], t0[..., :off[k]]) and torch.equal(t[..., off[k] + c:], t0[..., off[k] + c:])

        add16 = lambda old, new: (old.float() + new.float()).to(torch.bfloat16)
        what = f"{s.name} (shape {i}; paths {blk.plan.paths}; res {with_res}, gres {with_gres}/{gres_add}, dx target {dx_target}/{dx_add}; ld {ld}, off {off})"
        assert beside_untouched(A, A0, "a"), what
        if with_res:
            ref = oracle.cbs_fwd_bwd(inp.x, inp.w, inp.gamma, inp.beta, inp.g, s.stride, EPS, need_dx=False)
            parity.check(what + ": a + res", cut(A, "a").double().cpu().numpy(), ref.a + cut(R, "r").double().cpu().numpy(), "bf16")
        else:
            assert torch.equal(cut(A, "a"), dense.a), what
        for name in ("y", "dy", "dw", "dgamma", "dbeta", "mean", "invstd"):
            assert torch.equal(getattr(blk, name), getattr(dense, name)), (what, name)
        if dx_target:
            assert beside_untouched(D, D0, "d"), what
            assert torch.equal(cut(D, "d"), add16(cut(D0, "d"), dense.dx) if dx_add else dense.dx), what
        else:
            assert torch.equal(blk.dx, dense.dx) and torch.equal(D, D0), what
        if with_gres:
            assert beside_untouched(Q, Q0, "q"), what
            assert torch.equal(cut(Q, "q"), add16(cut(Q0, "q"), blk.g) if gres_add else blk.g), what
        else:
            assert torch.equal(Q, Q0), what
    assert min(used.values()) >= 4, used


def test_random_shapes_through_the_glue_calls_and_the_plan_free_statistics():
    """The wiring calls of a chained network (5x5 max-pool, 2x upsampling, slice add) forward and backward on 80 random
    extents (1-3 images of 1..39 x 1..39 pixels, 8..392 channels), both 16-bit types, every operand a randomly placed
    channel slice of a wider tensor or dense, against the chain oracle's definitions; and the plan-free statistics call on
    random matrices against the fp64 moments of the tensor it read."""
    import torch

    from oracle import chain as och
    from paper_2609_10632_b200 import binding as nb

    rs = np.random.RandomState(404)
    dev = torch.device("cuda:0")
    gen = torch.Generator(device=dev)
    gen.manual_seed(404)

    def wide(n, h, w, c, dt):
        off = 8 * int(rs.randint(0, 5))
        ld = c + off + 8 * int(rs.randint(0, 5))
        if rs.rand() < 0.3:
            off, ld = 0, c
        return torch.randn(n, h, w, ld, generator=gen, device=dev).to(dt), off, ld

    first = lambda t, off: t.data_ptr() + off * t.element_size()
    f64 = lambda t: t.double().cpu().numpy()

    def beside_untouched(t, t0, off, c):
        return torch.equal(t[..., :off], t0[..., :off]) and torch.equal(t[..., off + c:], t0[..., off + c:])

    for i in range(80):
        n, h, w, c = int(rs.randint(1, 4)), int(rs.randint(1, 40)), int(rs.randint(1, 40)), 8 * int(rs.randint(1, 50))
        dtn = int(rs.choice([nb.NB_DTYPE_BF16, nb.NB_DTYPE_F16]))
        dt, ulp = (torch.bfloat16, 2.0**-8) if dtn == nb.NB_DTYPE_BF16 else (torch.float16, 2.0**-10)
        what = f"draw {i}: {n} x {h} x {w} x {c}, dtype {dtn}"

        X, ox, lx = wide(n, h, w, c, dt)
        Y, oy, ly = wide(n, h, w, c, dt)
        Y0 = Y.clone()
        idx = torch.empty(n, h, w, c, dtype=torch.uint8, device=dev)
        nb.nb_maxpool5_fwd(dtn, n, h, w, c, first(X, ox), first(Y, oy), idx, ld_x=lx, ld_y=ly)
        ref_y, _ = och.maxpool5(f64(X[..., ox:ox + c]))
        assert np.array_equal(f64(Y[..., oy:oy + c]), ref_y) and beside_untouched(Y, Y0, oy, c), what + ": max-pool"
        G, og, lg = wide(n, h, w, c, dt)
        DX, od, ldd = wide(n, h, w, c, dt)
        DX0, add = DX.clone(), bool(rs.rand() < 0.5)
        nb.nb_maxpool5_bwd(dtn, n, h, w, c, first(G, og), idx, first(DX, od), accumulate=add, ld_g=lg, ld_dx=ldd)
        torch.cuda.synchronize()
        # equal maxima may be routed to either position: the gradient is checked from the positions the kernel recorded
        want = och.maxpool5_bwd(f64(G[..., og:og + c]), idx.cpu().numpy()) + (f64(DX0[..., od:od + c]) if add else 0.0)
        assert np.abs(f64(DX[..., od:od + c]) - want).max() <= ulp * max(1.0, np.abs(want).max()), what + ": max-pool gradient"
        assert beside_untouched(DX, DX0, od, c), what + ": max-pool gradient"

        S, os_, ls = wide(n, h, w, c, dt)
        L, ol, ll = wide(n, 2 * h, 2 * w, c, dt)
        L0 = L.clone()
        nb.nb_upsample2(dtn, n, h, w, c, first(S, os_), first(L, ol), ld_small=ls, ld_large=ll)
        torch.cuda.synchronize()
        assert np.array_equal(f64(L[..., ol:ol + c]), och.upsample2(f64(S[..., os_:os_ + c]))) and beside_untouched(L, L0, ol, c), what + ": upsampling"
        S0, add = S.clone(), bool(rs.rand() < 0.5)
        nb.nb_upsample2(dtn, n, h, w, c, first(L, ol), first(S, os_), backward=True, accumulate=add, ld_small=ls, ld_large=ll)
        torch.cuda.synchronize()
        want = och.upsample2_bwd(f64(L[..., ol:ol + c])) + (f64(S0[..., os_:os_ + c]) if add else 0.0)
        assert np.abs(f64(S[..., os_:os_ + c]) - want).max() <= ulp * max(1.0, np.abs(want).max()), what + ": upsampling gradient"
        assert beside_untouched(S, S0, os_, c), what + ": upsampling gradient"

        A, oa, la = wide(n, h, w, c, dt)
        B, ob, lb = wide(n, h, w, c, dt)
        O, oo, lo = wide(n, h, w, c, dt)
        O0, with_b, add = O.clone(), bool(rs.rand() < 0.6), bool(rs.rand() < 0.5)
        nb.nb_slice_add(dtn, n * h * w, c, first(O, oo), lo, first(A, oa), la, first(B, ob) if with_b else None, lb if with_b else 0, accumulate=add)
        torch.cuda.synchronize()
        want = A[..., oa:oa + c].float() + (B[..., ob:ob + c].float() if with_b else 0.0) + (O0[..., oo:oo + c].float() if add else 0.0)
        assert torch.equal(O[..., oo:oo + c], want.to(dt)) and beside_untouched(O, O0, oo, c), what + ": slice add"

        m, cc = int(rs.randint(2, 5000)), 8 * int(rs.randint(1, 73))
        sdt = int(rs.choice([nb.NB_DTYPE_F16, nb.NB_DTYPE_F32]))
        y = torch.randn(m, cc, generator=gen, device=dev) * float(rs.uniform(0.5, 3)) + float(rs.uniform(-2, 2))
        y = y.to(torch.float16 if sdt == nb.NB_DTYPE_F16 else torch.float32)
        mean, invstd = torch.empty(cc, device=dev), torch.empty(cc, device=dev)
        nb.nb_bn_stats_static(y, sdt, m, cc, EPS, mean, invstd)
        torch.cuda.synchronize()
        ref_mean, ref_var = f64(y).mean(0), f64(y).var(0)
        ref_invstd = 1.0 / np.sqrt(ref_var + EPS)
        assert (np.abs(f64(mean) - ref_mean) <= 2e-6 * np.sqrt(ref_mean**2 + ref_var) + 1e-7).all(), f"{what}: mean of {m} x {cc}"
        assert (np.abs(f64(invstd) - ref_invstd) / ref_invstd <= 1e-6 * (1 + ref_mean**2 / (ref_var + EPS)) + 2e-6).all(), f"{what}: invstd of {m} x {cc}"


@pytest.mark.parametrize("strips", ["by_width", "wide", "narrow"])
def test_random_first_layer_shapes_match_oracle(strips, monkeypatch):
    """The network's first layer (3 -> 48 channels, 3x3, stride 2) has kernels of its own, which cut every output row into
    strips: 320 pixels (forward) and 128 pixels (weight gradient) on rows of at least 160 output pixels, 64 otherwise.  30
    random images per form (1-2 images, 2..78 x 2..838 pixels, even; bf16 and fp16 operands) through the training step
    and the inference call, with the form chosen by the width as in production and with either form forced on every
    width (NB_STEM_WIDE), so that ragged last strips, rows narrower than a strip and rows of several strips all occur."""
    import torch

    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200.block import CbsBlock

    if strips != "by_width":
        monkeypatch.setenv("NB_STEM_WIDE", "1" if strips == "wide" else "0")
    rs = np.random.RandomState({"by_width": 505, "wide": 606, "narrow": 707}[strips])
    for i in range(30):
        n, h = int(rs.randint(1, 3)), 2 * int(rs.randint(1, 40))
        w = 2 * int(rs.randint(150, 340)) if rs.rand() < 0.3 else 2 * int(rs.randint(1, 420))
        mode = int(rs.choice([nb.NB_MODE_BF16_TC, nb.NB_MODE_F16_TC]))
        shape = wl.ConvShape(f"first{n}x{h}x{w}", n, h, w, 3, 48, 3, 2, True)
        inp = wl.make_inputs(shape, 35, i, bf16=True, affine="random")
        blk = CbsBlock(shape, mode=mode, eps=EPS)
        blk.upload(inp)
        blk.step()
        blk.poll()
        out = blk.download()
        ref = oracle.cbs_fwd_bwd(inp.x, inp.w, inp.gamma, inp.beta, inp.g, 2, EPS)
        try:
            parity.check_stats(out["mean"], out["invstd"], ref.y, EPS, "bf16")
            for name in ("a", "dgamma", "dbeta", "dw", "dx", "y", "dy"):
                parity.check(name, out[name], getattr(ref, name), "bf16")
            rm, rv, _ = wl.make_eval_stats(shape, 35, i)
            up = lambda a: torch.from_numpy(a).to(blk.dev)
            o = torch.empty_like(blk.a)
            ws = torch.empty(max(blk.plan.infer_bytes, blk.plan.bwd_bytes, 256), dtype=torch.uint8, device=blk.dev)
            nb.nb_conv_bn_silu_infer(blk.plan, blk.x, blk.w, blk.gamma, blk.beta, up(rm), up(rv), o, ws)
            torch.cuda.synchronize()
            parity.check("a_eval", o.double().cpu().numpy(), oracle.cbs_infer(inp.x, inp.w, inp.gamma, inp.beta, rm, rv, 2, EPS), "bf16")
        except AssertionError as e:
            raise AssertionError(f"{shape.name} (draw {i}, mode {mode}, strips {strips}): {e}") from None


def test_random_shapes_on_the_other_paths_match_oracle():
    """The paths beside the default one on 60 random shapes, one of the three per shape: the fp32 reference mode (CUDA-core
    kernels, fp32 tensors; bar 1e-5), the CUDA-core kernels forced in bf16 mode, and the fixed-order statistics kernels
    (NB_CBS_FLAG_SEPARATE_FINALIZE) under the tensor-core convolutions."""
    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200.block import CbsBlock

    rs = np.random.RandomState(808)
    seen = set()
    for i in range(60):
        s = _draw(rs)
        which = int(rs.randint(0, 3))
        if which == 0 and s.c_out % 4:
            continue  # (fp32 mode reads the channels as 16-byte vectors)
        mode, flags = [(nb.NB_MODE_F32_REF, 0), (nb.NB_MODE_BF16_TC, nb.NB_CBS_FLAG_FORCE_SIMT), (nb.NB_MODE_BF16_TC, nb.NB_CBS_FLAG_SEPARATE_FINALIZE)][which]
        inp = wl.make_inputs(s, 37, i, bf16=(which != 0), affine="random")
        blk = CbsBlock(s, mode=mode, eps=EPS, flags=flags)
        blk.upload(inp)
        blk.step()
        blk.poll()
        out = blk.download()
        ref = oracle.cbs_fwd_bwd(inp.x, inp.w, inp.gamma, inp.beta, inp.g, s.stride, EPS)
        tag = "f32" if which == 0 else "bf16"
        try:
            parity.check_stats(out["mean"], out["invstd"], ref.y, EPS, tag)
            for name in ("a", "dgamma", "dbeta", "dw", "y", "dy"):
                parity.check(name, out[name], getattr(ref, name), tag)
            if s.k == 1 and s.stride == 2:  # (see _check_dx; fp32 mode has only the relative L2 bar)
                assert not out["dx"][:, 1::2].any() and not out["dx"][:, :, 1::2].any()
                parity.check("dx", out["dx"][:, ::2, ::2, :], ref.dx[:, ::2, ::2, :], tag)
            else:
                parity.check("dx", out["dx"], ref.dx, tag)
        except AssertionError as e:
            raise AssertionError(f"{s.name} (draw {i}, path {which}, {blk.plan.paths}): {e}") from None
        if which == 1:
            assert blk.plan.paths == {"fprop": 0, "dgrad": 0, "wgrad": 0}
        seen.add(which)
    assert seen == {0, 1, 2}


def test_random_shapes_of_the_row_tile_weight_gradient_match_oracle():
    """3x3 stride-1 layers whose width is a multiple of 16 take their weight gradient from a kernel of its own (a stage is
    one output row; the three taps of a filter row read one staged input row at three start addresses).  40 random
    shapes of that kind (1-3 images, 1..39 rows, widths 16..80, 16..384 channels on either side, bf16 and fp16 operands),
    with the form chosen by the plan and with it forced on (NB_WG_ROWS=1: also where the plan prefers the other kernel),
    against the oracle; and on a pitched x, which must give the dense run's bits."""
    import os

    import torch

    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200.block import CbsBlock

    channels = [16, 32, 48, 64, 80, 96, 128, 160, 192, 256, 288, 384]
    rs = np.random.RandomState(909)
    old = os.environ.get("NB_WG_ROWS")
    try:
        for i in range(40):
            n, h, w = int(rs.randint(1, 4)), int(rs.randint(1, 40)), 16 * int(rs.randint(1, 6))
            ci, co = int(rs.choice(channels)), int(rs.choice(channels))
            if n * h * w * 9 * ci * co > 2e9:
                continue
            if i % 2:
                os.environ["NB_WG_ROWS"] = "1"
            else:
                os.environ.pop("NB_WG_ROWS", None)
            mode = int(rs.choice([nb.NB_MODE_BF16_TC, nb.NB_MODE_F16_TC]))
            s = wl.ConvShape(f"rows{n}x{h}x{w}x{ci}->{co}", n, h, w, ci, co, 3, 1, False)
            inp = wl.make_inputs(s, 39, i, bf16=True, affine="random")
            blk = CbsBlock(s, mode=mode, eps=EPS)
            blk.upload(inp)
            blk.step()
            blk.poll()
            ref = oracle.cbs_fwd_bwd(inp.x, inp.w, inp.gamma, inp.beta, inp.g, 1, EPS, need_dx=False)
            what = f"{s.name} (draw {i}, mode {mode}, forced {i % 2})"
            parity.check(what + ": dw", blk.dw.double().cpu().numpy(), ref.dw, "bf16")
            # x as a channel slice of a wider tensor: the same bits
            ld, off = ci + 24, 8
            wide = torch.randn(n, h, w, ld, device=blk.dev).to(blk.x.dtype)
            wide[..., off:off + ci] = blk.x
            pitched = CbsBlock(s, mode=mode, eps=EPS)
            pitched.upload(inp)
            pitched.plan.set_pitches(ld_x=ld)
            dw2 = torch.empty_like(blk.dw)
            nb.nb_conv_bn_silu_bwd_weight(pitched.plan, wide.data_ptr() + off * wide.element_size(), blk.dy, dw2, pitched.ws)
            torch.cuda.synchronize()
            pitched.poll()
            assert torch.equal(dw2, blk.dw), what + ": pitched x"
    finally:
        if old is None:
            os.environ.pop("NB_WG_ROWS", None)
        else:
            os.environ["NB_WG_ROWS"] = old
