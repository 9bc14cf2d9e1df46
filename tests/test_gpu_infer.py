"""Evaluation-mode and plain variants on the GPU against the fp64 oracle (same tolerances as the training path):
nb_conv_bn_silu_infer (running statistics, Table 2 row 9), nb_conv_bias_act (bias, no normalisation: the head of
Table 2 row 3) and nb_bn_fold.  The oracle always computes from (x, w, gamma, beta, running statistics / bias)."""
import numpy as np
import pytest

import oracle
from paper_2609_10632_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

EPS = 1e-3


def S(n, h, w, ci, co, k, s, img=False):
    return wl.ConvShape(f"t{n}x{h}x{w}x{ci}->{co}k{k}s{s}", n, h, w, ci, co, k, s, img)


SHAPES = [
    S(2, 32, 32, 16, 32, 3, 1),       # one tile pair, fused
    S(2, 40, 40, 64, 64, 3, 1),       # 25 tiles
    S(2, 38, 42, 48, 96, 3, 1),       # ragged last tile, two epilogue teams of 48 columns
    S(2, 36, 36, 96, 192, 3, 2),      # stride 2, CTA pairs
    S(2, 20, 20, 288, 288, 1, 1),     # 1x1: tiled A map, two n-tiles
    S(2, 20, 20, 576, 64, 3, 1),
    S(3, 24, 24, 128, 80, 1, 1),      # head-like: 80 output channels
    S(2, 7, 6, 3, 8, 3, 2),           # not on the tensor-core path: convolution, coefficient kernel, elementwise pass
    S(2, 12, 10, 40, 24, 1, 1),
    S(1, 64, 64, 3, 48, 3, 2, True),  # stem-like
]


class Dev:
    """Device tensors of one layer for the inference calls (torch only allocates and copies)."""

    def __init__(self, shape, mode, cfg_id, layer_id, flags=0):
        import torch

        from paper_2609_10632_b200 import binding as nb

        self.nb, self.torch = nb, torch
        self.s = s = shape
        self.mode = mode
        self.f32 = mode == nb.NB_MODE_F32_REF
        self.inp = wl.make_inputs(s, cfg_id, layer_id, bf16=not self.f32, affine="random")
        self.rm, self.rv, self.bias = wl.make_eval_stats(s, cfg_id, layer_id)
        self.plan = nb.Plan.for_shape(s, eps=EPS, mode=mode, flags=flags)
        act = torch.float32 if self.f32 else torch.bfloat16
        dev = torch.device("cuda", 0)
        up = lambda a, dt=torch.float32: torch.from_numpy(np.ascontiguousarray(a)).to(dt).to(dev)
        self.x, self.w = up(self.inp.x, act), up(self.inp.w, act)
        self.gamma, self.beta = up(self.inp.gamma), up(self.inp.beta)
        self.d_rm, self.d_rv, self.d_bias = up(self.rm), up(self.rv), up(self.bias)
        self.out = torch.empty(s.n, s.ho, s.wo, s.c_out, dtype=act, device=dev)
        self.ws = torch.empty(max(self.plan.infer_bytes, 256), dtype=torch.uint8, device=dev)

    def result(self):
        self.torch.cuda.synchronize()
        self.nb.nb_cbs_poll_status(self.plan)
        return self.out.detach().to(self.torch.float64).cpu().numpy()


def _tag(mode):
    return "bf16" if mode == 0 else "f32"


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: s.name)
@pytest.mark.parametrize("mode", [0, 1], ids=["bf16", "f32"])
def test_eval_mode_forward_matches_oracle(shape, mode):
    if mode == 1 and shape.c_out % 4:
        pytest.skip("fp32 mode needs c_out % 4 == 0")
    d = Dev(shape, mode, cfg_id=21, layer_id=SHAPES.index(shape))
    tc_ok = mode == 0 and shape.c_in % 16 == 0 and shape.c_out % 16 == 0
    first_layer = mode == 0 and (shape.c_in, shape.c_out, shape.k, shape.stride) == (3, 48, 3, 2) and shape.h % 2 == 0 and shape.w % 2 == 0
    assert d.plan.infer_fused == (tc_ok or first_layer)
    d.nb.nb_conv_bn_silu_infer(d.plan, d.x, d.w, d.gamma, d.beta, d.d_rm, d.d_rv, d.out, d.ws)
    ref = oracle.cbs_infer(d.inp.x, d.inp.w, d.inp.gamma, d.inp.beta, d.rm, d.rv, shape.stride, EPS)
    parity.check("a", d.result(), ref, _tag(mode))


@pytest.mark.parametrize("shape", [SHAPES[0], SHAPES[2], SHAPES[3], SHAPES[6], SHAPES[8]], ids=lambda s: s.name)
@pytest.mark.parametrize("act", [0, 1], ids=["linear", "silu"])
@pytest.mark.parametrize("with_bias", [True, False], ids=["bias", "nobias"])
def test_conv_bias_matches_oracle(shape, act, with_bias):
    d = Dev(shape, 0, cfg_id=22, layer_id=SHAPES.index(shape))
    d.nb.nb_conv_bias_act(d.plan, d.x, d.w, d.d_bias if with_bias else None, act, d.out, d.ws)
    ref = oracle.conv_bias_act(d.inp.x, d.inp.w, d.bias if with_bias else None, shape.stride, act=bool(act))
    parity.check("out", d.result(), ref, "bf16")


def test_conv_bias_fp32_mode_matches_oracle():
    shape = SHAPES[1]
    d = Dev(shape, 1, cfg_id=22, layer_id=1)
    d.nb.nb_conv_bias_act(d.plan, d.x, d.w, d.d_bias, 0, d.out, d.ws)
    parity.check("out", d.result(), oracle.conv_bias_act(d.inp.x, d.inp.w, d.bias, shape.stride), "f32")


@pytest.mark.parametrize("shape", [SHAPES[1], SHAPES[3], SHAPES[4], SHAPES[8]], ids=lambda s: s.name)
@pytest.mark.parametrize("mode", [0, 1], ids=["bf16", "f32"])
def test_folded_block_matches_oracle(shape, mode):
    """nb_bn_fold then nb_conv_bias_act(act = 1) against the oracle's UNFOLDED evaluation-mode block, and the folded
    filter and bias themselves against the oracle's fold (the filter within one rounding of the activation dtype)."""
    d = Dev(shape, mode, cfg_id=23, layer_id=SHAPES.index(shape))
    torch = d.torch
    wf = torch.empty_like(d.w)
    bf = torch.empty(shape.c_out, dtype=torch.float32, device=d.w.device)
    d.nb.nb_bn_fold(d.plan, d.w, d.gamma, d.beta, d.d_rm, d.d_rv, wf, bf)
    d.nb.nb_conv_bias_act(d.plan, d.x, wf, bf, 1, d.out, d.ws)
    got = d.result()
    ref_w, ref_b = oracle.bn_fold(d.inp.w, d.inp.gamma, d.inp.beta, d.rm, d.rv, EPS)
    rel = 2.0 ** -8 if mode == 0 else 1e-6  # bf16 keeps 8 significant bits: half an ulp is 2^-9 relative
    np.testing.assert_allclose(wf.to(torch.float64).cpu().numpy(), ref_w, rtol=rel, atol=1e-30)
    np.testing.assert_allclose(bf.to(torch.float64).cpu().numpy(), ref_b, rtol=1e-5, atol=1e-6)
    ref = oracle.cbs_infer(d.inp.x, d.inp.w, d.inp.gamma, d.inp.beta, d.rm, d.rv, shape.stride, EPS)
    parity.check("a", got, ref, _tag(mode))


def test_eval_mode_on_the_cuda_core_path_matches_oracle():
    shape = SHAPES[1]
    from paper_2609_10632_b200 import binding as nb

    d = Dev(shape, 0, cfg_id=24, layer_id=0, flags=nb.NB_CBS_FLAG_FORCE_SIMT)
    assert not d.plan.infer_fused
    d.nb.nb_conv_bn_silu_infer(d.plan, d.x, d.w, d.gamma, d.beta, d.d_rm, d.d_rv, d.out, d.ws)
    ref = oracle.cbs_infer(d.inp.x, d.inp.w, d.inp.gamma, d.inp.beta, d.rm, d.rv, shape.stride, EPS)
    parity.check("a", d.result(), ref, "bf16")


def test_eval_mode_equals_training_forward_when_given_the_batch_statistics():
    """Cross-check inside the library: the training forward's saved mean and 1/invstd^2 - eps as running statistics
    must reproduce the training activations (both round the same fp32 value to bf16; y goes through fp16 in training)."""
    import torch

    from paper_2609_10632_b200.block import CbsBlock

    shape = SHAPES[2]
    inp = wl.make_inputs(shape, 25, 0, bf16=True, affine="random")
    blk = CbsBlock(shape, eps=EPS)
    blk.upload(inp)
    blk.forward()
    torch.cuda.synchronize()
    var = (1.0 / blk.invstd.double() ** 2 - EPS).float()
    out = torch.empty_like(blk.a)
    ws = torch.empty(max(blk.plan.infer_bytes, 256), dtype=torch.uint8, device=blk.dev)
    from paper_2609_10632_b200 import binding as nb

    nb.nb_conv_bn_silu_infer(blk.plan, blk.x, blk.w, blk.gamma, blk.beta, blk.mean, var, out, ws)
    torch.cuda.synchronize()
    blk.poll()
    a_train = blk.a.double().cpu().numpy()
    parity.check("a", out.double().cpu().numpy(), a_train, "bf16")


def test_infer_argument_checks():
    from paper_2609_10632_b200 import binding as nb

    d = Dev(SHAPES[0], 0, cfg_id=26, layer_id=0)
    with pytest.raises(nb.NbError) as e:
        nb.nb_conv_bias_act(d.plan, d.x, d.w, None, 2, d.out, d.ws)
    assert e.value.status == nb.NB_ERR_INVALID_ARG
    with pytest.raises(nb.NbError) as e:
        nb.nb_conv_bn_silu_infer(d.plan, d.x, d.w, d.gamma, d.beta, None, d.d_rv, d.out, d.ws)
    assert e.value.status == nb.NB_ERR_INVALID_ARG
    small = S(1, 8, 8, 3, 8, 3, 1)
    d2 = Dev(small, 0, cfg_id=26, layer_id=1)
    assert d2.plan.infer_bytes > 256  # not fused: the workspace holds the convolution output
    with pytest.raises(nb.NbError) as e:
        nb.nb_conv_bn_silu_infer(d2.plan, d2.x, d2.w, d2.gamma, d2.beta, d2.d_rm, d2.d_rv, d2.out, d2.ws[:256])
    assert e.value.status == nb.NB_ERR_WORKSPACE


@pytest.mark.parametrize("shape", [SHAPES[6], SHAPES[1], SHAPES[3], SHAPES[8]], ids=lambda s: s.name)
@pytest.mark.parametrize("mode", [0, 1], ids=["bf16", "f32"])
def test_conv_bias_backward_matches_oracle(shape, mode):
    d = Dev(shape, mode, cfg_id=27, layer_id=SHAPES.index(shape))
    torch = d.torch
    act = torch.float32 if d.f32 else torch.bfloat16
    g = d.inp.g  # seeded upstream gradient of the output's shape (bf16-representable in bf16 mode)
    dev = d.x.device
    dout = torch.from_numpy(np.ascontiguousarray(g)).to(act).to(dev)
    dx = torch.empty_like(d.x)
    dw = torch.empty(d.w.shape, dtype=torch.float32, device=dev)
    db = torch.empty(shape.c_out, dtype=torch.float32, device=dev)
    ws = torch.empty(d.plan.bwd_bytes, dtype=torch.uint8, device=dev)
    d.nb.nb_conv_bias_bwd(d.plan, d.x, d.w, dout, dx, dw, db, ws)
    torch.cuda.synchronize()
    d.nb.nb_cbs_poll_status(d.plan)
    rdx, rdw, rdb = oracle.conv_bias_bwd(d.inp.x, d.inp.w, g, shape.stride)
    tag = _tag(mode)
    parity.check("dx", dx.double().cpu().numpy(), rdx, tag)
    parity.check("dw", dw.double().cpu().numpy(), rdw, tag)
    parity.check("dbias", db.double().cpu().numpy(), rdb, tag)
    # dx and dbias are optional
    dw2 = torch.empty_like(dw)
    d.nb.nb_conv_bias_bwd(d.plan, d.x, d.w, dout, None, dw2, None, ws)
    torch.cuda.synchronize()
    assert torch.equal(dw, dw2)
