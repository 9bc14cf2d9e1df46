"""GPU results of the C-ABI calls against the fp64 CPU oracle, element by element, on seeded inputs.

bf16 mode: relative L2 <= 5e-3 and per-element |err| <= 5e-2 * rms(ref) for a, dx, dw, dgamma, dbeta;
fp32 reference mode: relative L2 <= 1e-5.  The oracle always computes end to end from (x, w, gamma, beta, g).
"""
import numpy as np
import pytest

import oracle
from paper_2609_10632_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

EPS = 1e-3


def _run_block(shape, mode, cfg_id, layer_id=0, affine="init", flags=0, need_dx=True, running=False, momentum=0.03):
    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200.block import CbsBlock

    bf16 = mode != nb.NB_MODE_F32_REF  # the seeded 16-bit inputs are bf16-representable, hence also exact in fp16
    inp = wl.make_inputs(shape, cfg_id, layer_id, bf16=bf16, affine=affine)
    blk = CbsBlock(shape, mode=mode, eps=EPS, momentum=momentum, flags=flags, need_dx=need_dx, running_stats=running)
    blk.upload(inp)
    blk.step()
    blk.poll()
    return inp, blk, blk.download()


def _oracle(inp, need_dx=True):
    s = inp.shape
    return oracle.cbs_fwd_bwd(inp.x, inp.w, inp.gamma, inp.beta, inp.g, s.stride, EPS, need_dx=need_dx)


def _compare(out, ref, mode, need_dx=True, report=None):
    tag = "bf16" if mode == 0 else "f32"
    rep = {} if report is None else report
    parity.check_stats(out["mean"], out["invstd"], ref.y, EPS, tag)
    parity.check("a", out["a"], ref.a, tag, rep)
    parity.check("dgamma", out["dgamma"], ref.dgamma, tag, rep)
    parity.check("dbeta", out["dbeta"], ref.dbeta, tag, rep)
    parity.check("dw", out["dw"], ref.dw, tag, rep)
    if need_dx:
        parity.check("dx", out["dx"], ref.dx, tag, rep)
    # diagnostics (internal tensors): same bars
    parity.check("y", out["y"], ref.y, tag, rep)
    parity.check("dy", out["dy"], ref.dy, tag, rep)
    return rep


def S(n, h, w, ci, co, k, s, img=False):
    return wl.ConvShape(f"t{n}x{h}x{w}x{ci}->{co}k{k}s{s}", n, h, w, ci, co, k, s, img)


SMALL_SHAPES = [
    S(2, 32, 32, 16, 32, 3, 1),     # benchmark configuration 1
    S(2, 7, 6, 3, 8, 3, 2),         # odd extents, stride 2, 3 input channels
    S(1, 5, 5, 5, 8, 3, 2),
    S(3, 9, 11, 24, 16, 3, 1),
    S(2, 12, 10, 40, 24, 1, 1),
    S(2, 13, 9, 16, 16, 1, 2),
    S(1, 1, 3, 8, 8, 3, 1),         # fewer rows than any tile
    S(2, 40, 40, 64, 64, 3, 1),     # several tiles and a ragged tail (3200 rows = 25 x 128)
    S(2, 38, 42, 48, 96, 3, 1),     # 3192 rows: ragged last tile
    S(2, 36, 36, 96, 192, 3, 2),
    S(1, 64, 64, 3, 48, 3, 2, True),  # stem-like
    S(2, 20, 20, 576, 64, 3, 1),
    S(2, 20, 20, 288, 288, 1, 1),
    S(2, 36, 36, 48, 96, 3, 2),     # data gradient: four parity classes over 96 channels (64 + a 32-channel k-block per tap)
    S(2, 24, 24, 80, 160, 3, 1),    # 80 = 64 + 16: the 32-channel k-block is half zero fill; 160 = 2 x 64 + 32
]


@pytest.mark.parametrize("shape", SMALL_SHAPES, ids=lambda s: s.name)
@pytest.mark.parametrize("mode", [0, 1], ids=["bf16", "f32"])
def test_block_matches_oracle(shape, mode):
    if mode == 1 and shape.c_out % 4:
        pytest.skip("fp32 mode needs c_out % 4 == 0")
    inp, blk, out = _run_block(shape, mode, cfg_id=11, layer_id=SMALL_SHAPES.index(shape), affine="random")
    ref = _oracle(inp)
    _compare(out, ref, mode)


@pytest.mark.parametrize("shape", SMALL_SHAPES, ids=lambda s: s.name)
def test_block_matches_oracle_in_fp16_mode(shape):
    """NB_MODE_F16_TC (the paper's own 16-bit format, Sec. 3.2): the same kernels with fp16 operands and outputs.  fp16 keeps
    three more significant bits than bf16, so the bf16 bars hold with room; and the results must really be fp16-accurate:
    a good deal closer to the oracle than the bf16 mode can be."""
    from paper_2609_10632_b200 import binding as nb

    inp, blk, out = _run_block(shape, nb.NB_MODE_F16_TC, cfg_id=11, layer_id=SMALL_SHAPES.index(shape), affine="random")
    rep = _compare(out, _oracle(inp), 0)
    assert rep["a"][0] < 1.2e-3  # bf16 rounding alone is about 1.7e-3 relative L2
    if shape.c_in % 16 == 0 and shape.c_out % 16 == 0:
        assert blk.plan.paths["fprop"] == 1 and blk.plan.paths["wgrad"] == 1  # (a 1x1 stride-2 data gradient stays on the CUDA cores)


def test_fp16_mode_inference_calls_match_oracle():
    import torch

    from paper_2609_10632_b200 import binding as nb

    shape = SMALL_SHAPES[8]
    inp = wl.make_inputs(shape, 18, 0, bf16=True, affine="random")
    rm, rv, bias = wl.make_eval_stats(shape, 18, 0)
    blk = CbsBlock_f16(shape)
    blk.upload(inp)
    dev = blk.dev
    up = lambda a: torch.from_numpy(a).to(dev)
    out = torch.empty_like(blk.a)
    ws = torch.empty(max(blk.plan.infer_bytes, blk.plan.bwd_bytes, 256), dtype=torch.uint8, device=dev)
    assert blk.plan.infer_fused
    nb.nb_conv_bn_silu_infer(blk.plan, blk.x, blk.w, blk.gamma, blk.beta, up(rm), up(rv), out, ws)
    torch.cuda.synchronize()
    parity.check("a_eval", out.double().cpu().numpy(), oracle.cbs_infer(inp.x, inp.w, inp.gamma, inp.beta, rm, rv, shape.stride, EPS), "bf16")
    nb.nb_conv_bias_act(blk.plan, blk.x, blk.w, up(bias), 0, out, ws)
    dx, dw, db = torch.empty_like(blk.x), torch.empty_like(blk.dw), torch.empty(shape.c_out, dtype=torch.float32, device=dev)
    nb.nb_conv_bias_bwd(blk.plan, blk.x, blk.w, blk.g, dx, dw, db, ws)
    torch.cuda.synchronize()
    blk.poll()
    parity.check("out", out.double().cpu().numpy(), oracle.conv_bias_act(inp.x, inp.w, bias, shape.stride), "bf16")
    rdx, rdw, rdb = oracle.conv_bias_bwd(inp.x, inp.w, inp.g, shape.stride)
    parity.check("dx", dx.double().cpu().numpy(), rdx, "bf16")
    parity.check("dw", dw.double().cpu().numpy(), rdw, "bf16")
    parity.check("dbias", db.double().cpu().numpy(), rdb, "bf16")


def CbsBlock_f16(shape):
    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200.block import CbsBlock

    return CbsBlock(shape, mode=nb.NB_MODE_F16_TC, eps=EPS)


@pytest.mark.parametrize("shape", [SMALL_SHAPES[0], SMALL_SHAPES[7], SMALL_SHAPES[9]], ids=lambda s: s.name)
def test_forced_cuda_core_path_matches_oracle(shape):
    from paper_2609_10632_b200 import binding as nb

    inp, blk, out = _run_block(shape, 0, cfg_id=12, flags=nb.NB_CBS_FLAG_FORCE_SIMT)
    assert blk.plan.paths == {"fprop": 0, "dgrad": 0, "wgrad": 0}
    _compare(out, _oracle(inp), 0)


@pytest.mark.parametrize("shape", [SMALL_SHAPES[7], SMALL_SHAPES[9], SMALL_SHAPES[12]], ids=lambda s: s.name)
def test_separate_finalize_kernels_match_oracle(shape):
    """NB_CBS_FLAG_SEPARATE_FINALIZE: the statistics are finished by separate kernels that add per-block partial sums in a
    fixed order (instead of fp64 atomics and a finalize inside the consuming pass): same bars, and bit-identical statistics
    from run to run."""
    import torch

    from paper_2609_10632_b200 import binding as nb

    inp, blk, out = _run_block(shape, 0, cfg_id=14, affine="random", flags=nb.NB_CBS_FLAG_SEPARATE_FINALIZE, running=True)
    _compare(out, _oracle(inp), 0)
    first = {k: getattr(blk, k).clone() for k in ("mean", "invstd", "dgamma", "dbeta")}
    for _ in range(3):
        blk.step()
        torch.cuda.synchronize()
        for k, v in first.items():
            assert torch.equal(getattr(blk, k), v), k
    blk.poll()


def test_two_plans_on_two_streams():
    """Calls of different plans may overlap on the GPU: no kernel waits for another block or kernel, so two plans that
    each hold part of the GPU cannot block each other."""
    import torch

    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200.block import CbsBlock

    shapes = [SMALL_SHAPES[7], SMALL_SHAPES[9]]
    inps = [wl.make_inputs(s, 16, i, bf16=True, affine="random") for i, s in enumerate(shapes)]
    blks = [CbsBlock(s, eps=EPS) for s in shapes]
    for b, inp in zip(blks, inps):
        b.upload(inp)
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in blks]
    for _ in range(3):  # interleave the launches of the two plans
        for b, st in zip(blks, streams):
            b.step(stream=st)
    torch.cuda.synchronize()
    for b, inp in zip(blks, inps):
        b.poll()
        _compare(b.download(), _oracle(inp), 0)


def test_weight_gradient_on_a_second_stream_overlaps_the_next_layers():
    """The step bench.py times: each layer's weight gradient runs on a second stream with a workspace of its own while
    the main stream goes on with the next layer."""
    import torch

    from paper_2609_10632_b200.block import CbsBlock

    shapes = [SMALL_SHAPES[7], SMALL_SHAPES[9], SMALL_SHAPES[11], SMALL_SHAPES[0]]
    inps = [wl.make_inputs(s, 17, i, bf16=True, affine="random") for i, s in enumerate(shapes)]
    need = 0
    blks = []
    for s in shapes:
        blks.append(CbsBlock(s, eps=EPS))
        need = max(need, blks[-1].plan.bwd_bytes)
    for b, inp in zip(blks, inps):
        b.upload(inp)
    side_ws = torch.empty(need, dtype=torch.uint8, device=blks[0].dev)
    side = torch.cuda.Stream()
    main = torch.cuda.current_stream()
    torch.cuda.synchronize()
    for _ in range(3):
        side.wait_stream(main)
        for b in blks:
            b.step(wgrad_stream=side, wgrad_workspace=side_ws)
        main.wait_stream(side)
    torch.cuda.synchronize()
    for b, inp in zip(blks, inps):
        b.poll()
        _compare(b.download(), _oracle(inp), 0)


@pytest.mark.parametrize("shape", [SMALL_SHAPES[7], SMALL_SHAPES[8], SMALL_SHAPES[9], SMALL_SHAPES[12], SMALL_SHAPES[3]], ids=lambda s: s.name)
def test_channel_slice_operands_give_bitwise_the_dense_results(shape):
    """nb_cbs_plan_set_pitches: x, a_out and g as channel slices of wider tensors (what a chained network's split and
    concat buffers are).  Results must equal the dense run bit for bit (the kernels do the same arithmetic on the same
    values, only addresses change), match the oracle, and nothing outside the output slice may be written."""
    import torch

    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200.block import CbsBlock

    inp, dense, want = _run_block(shape, 0, cfg_id=20, affine="random")
    tc_x = dense.plan.paths["fprop"] == 1 and dense.plan.paths["wgrad"] == 1
    blk = CbsBlock(shape, eps=EPS)
    blk.upload(inp)
    dev, s = blk.dev, shape
    ldx, lda, ldg = (s.c_in + 24 if tc_x else s.c_in), s.c_out + 40, s.c_out + 8
    offx, offa, offg = (16 if tc_x else 0), 24, 8
    if not tc_x:
        with pytest.raises(nb.NbError) as e:
            blk.plan.set_pitches(ld_x=s.c_in + 8)
        assert e.value.status == nb.NB_ERR_UNSUPPORTED
    blk.plan.set_pitches(ld_x=ldx, ld_a=lda, ld_g=ldg)
    gen = torch.Generator(device=dev)
    gen.manual_seed(5)
    X = torch.randn(s.n, s.h, s.w, ldx, generator=gen, device=dev).to(torch.bfloat16)
    A = torch.randn(s.n, s.ho, s.wo, lda, generator=gen, device=dev).to(torch.bfloat16)
    G = torch.randn(s.n, s.ho, s.wo, ldg, generator=gen, device=dev).to(torch.bfloat16)
    X[..., offx:offx + s.c_in] = blk.x
    G[..., offg:offg + s.c_out] = blk.g
    A0 = A.clone()
    at = lambda t, c: t.data_ptr() + c * t.element_size()
    nb.nb_conv_bn_silu_fwd(blk.plan, at(X, offx), blk.w, blk.gamma, blk.beta, None, None, blk.y, blk.mean, blk.invstd, at(A, offa), blk.ws)
    nb.nb_conv_bn_silu_bwd_data(blk.plan, at(G, offg), blk.y, blk.mean, blk.invstd, blk.gamma, blk.beta, blk.w, blk.dx, blk.dgamma, blk.dbeta, blk.dy, blk.ws)
    nb.nb_conv_bn_silu_bwd_weight(blk.plan, at(X, offx), blk.dy, blk.dw, blk.ws)
    torch.cuda.synchronize()
    blk.poll()
    blk.a.copy_(A[..., offa:offa + s.c_out])
    got = blk.download()
    for name in ("a", "y", "dy", "dx", "dw", "dgamma", "dbeta", "mean", "invstd"):
        np.testing.assert_array_equal(got[name], want[name], err_msg=name)
    _compare(got, _oracle(inp), 0)
    assert torch.equal(A[..., :offa], A0[..., :offa]) and torch.equal(A[..., offa + s.c_out:], A0[..., offa + s.c_out:])
    # the other calls refuse a pitched plan; clearing the pitches brings them back
    ws = torch.empty(max(blk.plan.infer_bytes, 256), dtype=torch.uint8, device=dev)
    with pytest.raises(nb.NbError) as e:
        nb.nb_conv_bias_act(blk.plan, blk.x, blk.w, None, 0, blk.a, ws)
    assert e.value.status == nb.NB_ERR_UNSUPPORTED
    blk.plan.set_pitches()
    nb.nb_conv_bias_act(blk.plan, blk.x, blk.w, None, 0, blk.a, ws)
    torch.cuda.synchronize()


@pytest.mark.parametrize("shape", [SMALL_SHAPES[7], SMALL_SHAPES[8], SMALL_SHAPES[12], SMALL_SHAPES[11]], ids=lambda s: s.name)
def test_data_gradient_into_a_pitched_and_accumulating_target(shape):
    """nb_cbs_plan_set_dx_target: the data gradient written straight into a channel slice of a wider gradient buffer, and
    ADDED to what the slice holds (TMA reductions in the epilogue), as a tensor with several consumers needs.  Overwriting
    must give the dense run's bits; accumulating must give round(old + dx) -- one rounding to bf16 per element, what a
    separate accumulation pass gives -- and nothing outside the slice may change.  Layers without the TMA epilogue refuse."""
    import torch

    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200.block import CbsBlock

    inp, dense, want = _run_block(shape, 0, cfg_id=21, affine="random")
    assert dense.plan.paths["dgrad"] == 1
    blk = CbsBlock(shape, eps=EPS)
    blk.upload(inp)
    blk.step()
    s, dev = shape, blk.dev
    ld, off = s.c_in + 24, 16
    gen = torch.Generator(device=dev)
    gen.manual_seed(9)
    wide = torch.randn(s.n, s.h, s.w, ld, generator=gen, device=dev).to(torch.bfloat16)
    before = wide.clone()
    view = wide[..., off:off + s.c_in]

    def bwd(dx):
        nb.nb_conv_bn_silu_bwd_data(blk.plan, blk.g, blk.y, blk.mean, blk.invstd, blk.gamma, blk.beta, blk.w, dx, blk.dgamma, blk.dbeta, blk.dy, blk.ws)
        torch.cuda.synchronize()
        blk.poll()

    blk.plan.set_dx_target(ld_dx=ld, accumulate=False)
    bwd(view.data_ptr())
    assert torch.equal(view, dense.dx)
    assert torch.equal(wide[..., :off], before[..., :off]) and torch.equal(wide[..., off + s.c_in:], before[..., off + s.c_in:])
    wide.copy_(before)
    blk.plan.set_dx_target(ld_dx=ld, accumulate=True)
    bwd(view.data_ptr())
    expect = (before[..., off:off + s.c_in].float() + dense.dx.float()).to(torch.bfloat16)
    assert torch.equal(view, expect)
    assert torch.equal(wide[..., :off], before[..., :off]) and torch.equal(wide[..., off + s.c_in:], before[..., off + s.c_in:])
    blk.plan.set_dx_target()  # back to a dense, overwritten dx
    bwd(blk.dx)
    assert torch.equal(blk.dx, dense.dx)
    strided = CbsBlock(SMALL_SHAPES[9], eps=EPS)  # stride 2: its epilogue does not go through TMA
    with pytest.raises(nb.NbError) as e:
        strided.plan.set_dx_target(accumulate=True)
    assert e.value.status == nb.NB_ERR_UNSUPPORTED


@pytest.mark.parametrize("shape", [SMALL_SHAPES[7], SMALL_SHAPES[12], SMALL_SHAPES[3]], ids=lambda s: s.name)
@pytest.mark.parametrize("mode", [0, 1], ids=["bf16", "f32"])
def test_forward_with_a_residual_adds_it_once(shape, mode):
    """nb_cbs_plan_set_fwd_residual: a_out = SiLU(z) + res in the normalise + SiLU pass (res dense or a channel slice), the
    sum rounded once; against the oracle's block output plus the same residual, at the block's own bars; the saved
    tensors are those of the plain block, bit for bit."""
    import torch

    from paper_2609_10632_b200 import binding as nb

    inp, blk, plain = _run_block(shape, mode, cfg_id=22, affine="random")
    ref = _oracle(inp)
    s, dev = shape, blk.dev
    dt = blk.a.dtype
    gen = torch.Generator(device=dev)
    gen.manual_seed(3)
    for ld, off in ((0, 0), (s.c_out + 16, 8)):
        wide = torch.randn(s.n, s.ho, s.wo, ld or s.c_out, generator=gen, device=dev).to(dt)
        res = wide[..., off:off + s.c_out]
        blk.plan.set_fwd_residual(res, res.stride(-2))
        blk.forward()
        torch.cuda.synchronize()
        blk.poll()
        got = blk.a.double().cpu().numpy()
        parity.check("a + res", got, ref.a + res.double().cpu().numpy(), "bf16" if mode == 0 else "f32")
        np.testing.assert_array_equal(blk.y.double().cpu().numpy(), plain["y"])
        np.testing.assert_array_equal(blk.mean.double().cpu().numpy(), plain["mean"])
    ws = torch.empty(max(blk.plan.infer_bytes, 256), dtype=torch.uint8, device=dev)
    with pytest.raises(nb.NbError) as e:
        nb.nb_conv_bias_act(blk.plan, blk.x, blk.w, None, 0, blk.a, ws)
    assert e.value.status == nb.NB_ERR_UNSUPPORTED
    blk.plan.set_fwd_residual(None)
    blk.forward()
    torch.cuda.synchronize()
    np.testing.assert_array_equal(blk.a.double().cpu().numpy(), plain["a"])


@pytest.mark.parametrize("shape", [SMALL_SHAPES[7], SMALL_SHAPES[12]], ids=lambda s: s.name)
def test_saturated_fp16_stores_of_the_convolution_output_are_reported(shape):
    """The saved convolution output is fp16 (Sec. 3.2): a value beyond +-65504 is stored as +-65504 and the call says so
    through nb_cbs_poll_status (still NB_OK).  One input pixel made huge saturates the outputs around it and nothing else
    is reported when the inputs are ordinary."""
    import torch

    inp, blk, out = _run_block(shape, 0, cfg_id=24, affine="random")
    assert "saturated" not in blk.poll()
    blk.x[0, shape.h // 2, shape.w // 2, :] = 3.0e4
    blk.w.fill_(1.0)
    blk.forward()
    msg = blk.poll()
    assert "saturated" in msg, msg
    assert float(blk.y.abs().max()) == 65504.0 and bool(torch.isfinite(blk.y.float()).all())


@pytest.mark.parametrize("shape", [SMALL_SHAPES[7], SMALL_SHAPES[9], SMALL_SHAPES[5]], ids=lambda s: s.name)
def test_backward_hands_the_gradient_to_the_shortcut(shape):
    """nb_cbs_plan_set_bwd_residual: the data-gradient call also adds (or copies) its incoming gradient g into the
    shortcut's gradient tensor (dense or a channel slice), inside its dy pass.  The sum is the fp32 sum of the two 16-bit
    values rounded once -- checked exactly --, everything else the call writes is what the plain call writes, bit for
    bit, and the plans that cannot do it say so."""
    import torch

    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200.block import CbsBlock

    inp, blk, plain = _run_block(shape, 0, cfg_id=23, affine="random")
    s, dev = shape, blk.dev
    gen = torch.Generator(device=dev)
    gen.manual_seed(5)
    for ld, off, accumulate in ((0, 0, True), (s.c_out + 24, 16, True), (s.c_out + 8, 8, False)):
        wide = torch.randn(s.n, s.ho, s.wo, ld or s.c_out, generator=gen, device=dev).to(torch.bfloat16)
        before = wide.clone()
        gres = wide[..., off:off + s.c_out]
        blk.plan.set_bwd_residual(gres, gres.stride(-2), accumulate=accumulate)
        blk.backward_data()
        torch.cuda.synchronize()
        blk.poll()
        old = before[..., off:off + s.c_out]
        want = (old.float() + blk.g.float()).to(torch.bfloat16) if accumulate else blk.g
        assert torch.equal(gres, want)
        untouched = torch.ones(wide.shape[-1], dtype=torch.bool, device=dev)
        untouched[off:off + s.c_out] = False
        assert torch.equal(wide[..., untouched], before[..., untouched])  # the channels beside the slice
        for k in ("dx", "dy", "dgamma", "dbeta"):
            np.testing.assert_array_equal(getattr(blk, k).double().cpu().numpy(), plain[k], err_msg=k)
    blk.plan.set_bwd_residual(None)
    blk.backward_data()
    torch.cuda.synchronize()
    np.testing.assert_array_equal(blk.dy.double().cpu().numpy(), plain["dy"])
    fixed = CbsBlock(shape, eps=EPS, flags=nb.NB_CBS_FLAG_SEPARATE_FINALIZE)
    with pytest.raises(nb.NbError) as e:
        fixed.plan.set_bwd_residual(blk.g, 0)
    assert e.value.status == nb.NB_ERR_UNSUPPORTED


@pytest.mark.parametrize("shape", [SMALL_SHAPES[7], SMALL_SHAPES[9], SMALL_SHAPES[12], SMALL_SHAPES[13]], ids=lambda s: s.name)
def test_channel_accumulators_are_clean_between_calls(shape):
    """The default plans sum the BatchNorm statistics with fp64 atomics into accumulators that the plan owns, and the last
    block of the pass that reads them zeroes them again.  Whatever the sequence of calls -- whole steps, forward calls
    alone, data-gradient calls alone -- every call must start from zeros: the statistics of later calls equal those of
    the first one (the order of the atomic additions can move a total by one fp64 unit in the last place at most, hence an
    fp32 result by one unit in the last place at the very most), and the outputs still meet the bars."""
    import torch

    inp, blk, out = _run_block(shape, 0, cfg_id=15, affine="random", running=False)
    ref = _oracle(inp)
    _compare(out, ref, 0)
    first = {k: getattr(blk, k).clone() for k in ("mean", "invstd", "dgamma", "dbeta")}

    def same(k):
        a, b = getattr(blk, k), first[k]
        assert torch.all((a - b).abs() <= 1.2e-7 * b.abs()), k

    for _ in range(3):
        blk.forward()
    torch.cuda.synchronize()
    same("mean"); same("invstd")
    for _ in range(3):
        blk.backward_data()
    torch.cuda.synchronize()
    same("dgamma"); same("dbeta")
    for _ in range(2):
        blk.step()
    blk.poll()
    for k in first:
        same(k)
    _compare(blk.download(), ref, 0)


def test_config1_fresh_bn_both_modes():
    shape, = wl.config_shapes(1)
    for mode in (1, 0):
        inp, blk, out = _run_block(shape, mode, cfg_id=1)
        _compare(out, _oracle(inp), mode)


def test_results_are_not_suspiciously_exact():
    # bf16 outputs cannot be closer to the fp64 oracle than bf16 rounding allows; a much smaller error would mean
    # the comparison is not comparing two implementations.
    shape = SMALL_SHAPES[7]
    inp, blk, out = _run_block(shape, 0, cfg_id=13)
    ref = _oracle(inp)
    assert parity.rel_l2(out["a"], ref.a) > 3e-4
    assert parity.rel_l2(out["dx"], ref.dx) > 3e-4


def test_first_layer_without_dx():
    shape = SMALL_SHAPES[10]
    inp, blk, out = _run_block(shape, 0, cfg_id=14, need_dx=False)
    assert "dx" not in out
    _compare(out, _oracle(inp, need_dx=False), 0, need_dx=False)


def test_running_statistics_update():
    shape = SMALL_SHAPES[3]
    for mode in (0, 1):
        inp, blk, out = _run_block(shape, mode, cfg_id=15, running=True, momentum=0.1)
        rm, rv = np.zeros(shape.c_out), np.ones(shape.c_out)
        oracle.cbs_fwd(inp.x, inp.w, inp.gamma, inp.beta, shape.stride, EPS, rm, rv, 0.1)
        np.testing.assert_allclose(out["running_mean"], rm, rtol=0, atol=2e-3 if mode == 0 else 1e-6)
        np.testing.assert_allclose(out["running_var"], rv, rtol=3e-3 if mode == 0 else 1e-5)


def test_constant_channel_has_zero_variance():
    # a filter of zeros makes one output channel constant: invstd = eps^-1/2, a = SiLU(beta)
    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200.block import CbsBlock

    shape = SMALL_SHAPES[3]
    inp = wl.make_inputs(shape, 16, 0, affine="random")
    inp.w[3] = 0.0
    blk = CbsBlock(shape, mode=nb.NB_MODE_BF16_TC, eps=EPS)
    blk.upload(inp)
    blk.step()
    blk.poll()
    out = blk.download()
    ref = _oracle(inp)
    assert abs(out["invstd"][3] - EPS ** -0.5) < 1e-3 * EPS ** -0.5
    _compare(out, ref, 0)


def test_bn_stats_entry_point():
    import torch

    from paper_2609_10632_b200 import binding as nb

    for mode, dt, tag in ((nb.NB_MODE_BF16_TC, torch.float16, nb.NB_DTYPE_F16), (nb.NB_MODE_F32_REF, torch.float32, nb.NB_DTYPE_F32)):
        shape = S(2, 30, 34, 8, 48, 3, 1)
        plan = nb.Plan.for_shape(shape, mode=mode)
        rng = np.random.default_rng(5)
        y = (rng.normal(size=(shape.m, shape.c_out)) * rng.uniform(0.5, 2, shape.c_out) + rng.normal(size=shape.c_out) * 3).astype(np.float32)
        ty = torch.from_numpy(y).to(dt).cuda()
        yq = ty.to(torch.float64).cpu().numpy()
        mean, invstd, sm, sq = (torch.empty(shape.c_out, dtype=torch.float32, device="cuda") for _ in range(4))
        ws = torch.empty(plan.fwd_bytes, dtype=torch.uint8, device="cuda")
        nb.nb_bn_stats(plan, ty, tag, mean, invstd, sm, sq, ws)
        torch.cuda.synchronize()
        rmean, rvar, rinv = oracle.bn_stats(yq, EPS)
        np.testing.assert_allclose(mean.cpu().numpy(), rmean, rtol=1e-5, atol=1e-6)
        np.testing.assert_allclose(invstd.cpu().numpy(), rinv, rtol=1e-5)
        np.testing.assert_allclose(sm.cpu().numpy(), yq.sum(0), rtol=1e-5, atol=1e-3)
        np.testing.assert_allclose(sq.cpu().numpy(), (yq * yq).sum(0), rtol=1e-5)
        with pytest.raises(nb.NbError) as ei:
            nb.nb_bn_stats(plan, ty, nb.NB_DTYPE_BF16, mean, invstd, None, None, ws)
        assert ei.value.status == nb.NB_ERR_UNSUPPORTED


def test_bitwise_reproducible():
    import torch

    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200.block import CbsBlock

    for shape in (SMALL_SHAPES[7], SMALL_SHAPES[9]):
        inp = wl.make_inputs(shape, 17, 0, affine="random")
        blk = CbsBlock(shape, mode=nb.NB_MODE_BF16_TC)
        blk.upload(inp)
        blk.step()
        torch.cuda.synchronize()
        first = {k: getattr(blk, k).clone() for k in ("a", "y", "dx", "dw", "dgamma", "dbeta", "mean", "invstd", "dy")}
        for k in first:
            getattr(blk, k).zero_()
        blk.step()
        torch.cuda.synchronize()
        for k, v in first.items():
            assert torch.equal(v.view(torch.uint8), getattr(blk, k).view(torch.uint8)), k


def test_invalid_runtime_arguments_launch_nothing():
    import torch

    from paper_2609_10632_b200 import binding as nb
    from paper_2609_10632_b200.block import CbsBlock

    shape = SMALL_SHAPES[0]
    blk = CbsBlock(shape)
    blk.a.fill_(7.0)
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(nb.NbError) as ei:
        nb.nb_conv_bn_silu_fwd(blk.plan, blk.x, blk.w, blk.gamma, blk.beta, None, None, blk.y, blk.mean, blk.invstd, blk.a, small)
    assert ei.value.status == nb.NB_ERR_WORKSPACE
    with pytest.raises(nb.NbError) as ei:
        nb.nb_conv_bn_silu_fwd(blk.plan, blk.x.data_ptr() + 2, blk.w, blk.gamma, blk.beta, None, None, blk.y, blk.mean, blk.invstd, blk.a, blk.ws)
    assert ei.value.status == nb.NB_ERR_ALIGNMENT
    with pytest.raises(nb.NbError) as ei:
        nb.nb_conv_bn_silu_fwd(blk.plan, blk.x, blk.w, blk.gamma, blk.beta, blk.mean, None, blk.y, blk.mean, blk.invstd, blk.a, blk.ws)
    assert ei.value.status == nb.NB_ERR_INVALID_ARG
    with pytest.raises(nb.NbError) as ei:
        nb.nb_conv_bn_silu_bwd_weight(blk.plan, blk.x, None, blk.dw, blk.ws)
    assert ei.value.status == nb.NB_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert bool((blk.a == 7.0).all())


def test_step_from_host_buffers():
    import torch

    from paper_2609_10632_b200 import binding as nb

    shape = SMALL_SHAPES[8]
    inp = wl.make_inputs(shape, 18, 0, affine="random")
    plan = nb.Plan.for_shape(shape)
    pin = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).pin_memory()
    hx, hw, hg = pin(inp.x, torch.bfloat16), pin(inp.w, torch.bfloat16), pin(inp.g, torch.bfloat16)
    hgam, hbet = pin(inp.gamma, torch.float32), pin(inp.beta, torch.float32)
    ha = torch.empty(hg.shape, dtype=torch.bfloat16).pin_memory()
    hdx = torch.empty(hx.shape, dtype=torch.bfloat16).pin_memory()
    hdw = torch.empty(hw.shape, dtype=torch.float32).pin_memory()
    hdg, hdb = torch.empty(shape.c_out).pin_memory(), torch.empty(shape.c_out).pin_memory()
    scratch = torch.empty(plan.step_host_scratch_bytes(), dtype=torch.uint8, device="cuda")
    nb.nb_conv_bn_silu_step_host(plan, hx, hw, hgam, hbet, hg, ha, hdx, hdw, hdg, hdb, scratch)
    nb.nb_cbs_poll_status(plan)
    ref = _oracle(inp)
    parity.check("a", ha.double().numpy(), ref.a)
    parity.check("dx", hdx.double().numpy(), ref.dx)
    parity.check("dw", hdw.double().numpy(), ref.dw)
    parity.check("dgamma", hdg.double().numpy(), ref.dgamma)
    parity.check("dbeta", hdb.double().numpy(), ref.dbeta)
