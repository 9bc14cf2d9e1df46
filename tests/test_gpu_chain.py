"""A chained C2f unit on the GPU (block calls + nb_slice_add) against the chained fp64 oracle, and nb_slice_add alone.

Tolerance of the chain: every block adds its own bf16 rounding (the single-block bar is 5e-3 relative L2 from exact
inputs); through the 2 + 2n blocks of a unit and back the errors add roughly in quadrature, so the chained results are
held to 2e-2 relative L2 and 0.2 * rms per element (observed values are printed by the test)."""
import numpy as np
import pytest

import oracle
from oracle import chain
from paper_2609_10632_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu
EPS = 1e-3
CHAIN_REL_L2, CHAIN_MAX_OVER_RMS = 2e-2, 0.2


@pytest.mark.parametrize("dtype_name,rows,channels,ld_out,ld_a,ld_b,off", [
    ("bfloat16", 300, 32, 96, 32, 64, 32),   # vector path: concat into a slice
    ("bfloat16", 77, 24, 56, 24, 40, 8),     # vector path with 8-element granularity
    ("bfloat16", 50, 5, 13, 7, 9, 3),        # scalar path: nothing aligned
    ("float32", 64, 12, 20, 12, 16, 4),
    ("float16", 33, 16, 48, 16, 16, 16),
])
@pytest.mark.parametrize("with_b,accumulate", [(False, False), (True, False), (False, True), (True, True)])
def test_slice_add_matches_numpy_definition(dtype_name, rows, channels, ld_out, ld_a, ld_b, off, with_b, accumulate):
    import torch

    from paper_2609_10632_b200 import binding as nb

    dt = getattr(torch, dtype_name)
    code = {"float32": nb.NB_DTYPE_F32, "bfloat16": nb.NB_DTYPE_BF16, "float16": nb.NB_DTYPE_F16}[dtype_name]
    rng = np.random.Generator(np.random.Philox(key=[41, rows * 1000 + channels]))
    dev = torch.device("cuda", 0)
    mk = lambda ld: torch.from_numpy(rng.standard_normal((rows, ld)).astype(np.float32)).to(dt).to(dev)
    out, a, b = mk(ld_out), mk(ld_a), mk(ld_b)
    before = out.clone()
    es = out.element_size()
    nb.nb_slice_add(code, rows, channels, out.data_ptr() + off * es, ld_out, a, ld_a, b if with_b else None, ld_b, accumulate)
    torch.cuda.synchronize()
    # the definition, summed in fp32 in the documented order a + b + out and rounded once to the element type (for the 16-bit
    # types every partial sum is exact in fp32, so this is also the correctly rounded exact sum)
    want = a[:, :channels].float()
    if with_b:
        want = want + b[:, :channels].float()
    if accumulate:
        want = want + before[:, off:off + channels].float()
    want = want.to(dt)
    assert torch.equal(out[:, off:off + channels], want)
    # nothing outside the slice was touched
    assert torch.equal(out[:, :off], before[:, :off]) and torch.equal(out[:, off + channels:], before[:, off + channels:])


def _run_chain(batch, h, w, c1, c2, n, shortcut, cfg_id):
    import torch

    from paper_2609_10632_b200.c2f import C2fChain

    ch = C2fChain(batch, h, w, c1, c2, n, shortcut, eps=EPS)
    params, inputs = [], []
    for i, blk in enumerate(ch.blocks):
        inp = wl.make_inputs(blk.shape, cfg_id, i, bf16=True, affine="random")
        inputs.append(inp)
        params.append(chain.BlockParams(inp.w, inp.gamma, inp.beta))
        for name in ("w", "gamma", "beta"):
            dst = getattr(blk, name)
            dst.copy_(torch.from_numpy(np.ascontiguousarray(getattr(inp, name))).to(dst.dtype))
    x = inputs[0].x
    g_out = inputs[-1].g
    ch.cv1.x.copy_(torch.from_numpy(x).to(torch.bfloat16))
    ch.cv2.g.copy_(torch.from_numpy(g_out).to(torch.bfloat16))
    ch.forward()
    ch.backward()
    torch.cuda.synchronize()
    ch.poll()
    ref = chain.c2f_fwd_bwd(x, params, n, shortcut, EPS, g_out)
    return ch, ref


def _check(name, got, ref, report):
    r, m = parity.rel_l2(got, ref), parity.max_over_rms(got, ref)
    report.append(f"{name}: rel_l2={r:.2e} max/rms={m:.2e}")
    assert np.isfinite(got).all(), name
    assert r <= CHAIN_REL_L2, f"{name}: rel L2 {r:.3e}"
    assert m <= CHAIN_MAX_OVER_RMS, f"{name}: max/rms {m:.3e}"


@pytest.mark.parametrize("n,shortcut,c1,c2", [(2, True, 64, 64), (1, False, 96, 64), (2, True, 48, 32)], ids=["n2-shortcut", "n1-plain", "n2-cuda-core"])
def test_c2f_unit_matches_chained_oracle(n, shortcut, c1, c2):
    ch, ref = _run_chain(2, 24, 20, c1, c2, n, shortcut, cfg_id=51)
    f64 = lambda t: t.detach().double().cpu().numpy()
    report = []
    _check("out", f64(ch.cv2.a), ref.out, report)
    cat = f64(ch.cat)
    for j, part in enumerate(ref.parts):
        _check(f"part{j}", cat[..., j * ch.c:(j + 1) * ch.c], part, report)
    _check("dx", f64(ch.cv1.dx), ref.dx, report)
    for i, blk in enumerate(ch.blocks):
        dw, dgamma, dbeta = ref.grads[i]
        _check(f"block{i}.dw", f64(blk.dw), dw, report)
        _check(f"block{i}.dgamma", f64(blk.dgamma), dgamma, report)
        _check(f"block{i}.dbeta", f64(blk.dbeta), dbeta, report)
    print("\n".join(report))


@pytest.mark.parametrize("dtype_name,n,h,w,c", [("bfloat16", 2, 9, 7, 16), ("bfloat16", 1, 5, 6, 3), ("float32", 2, 6, 6, 5), ("float16", 1, 20, 20, 8)])
def test_maxpool5_forward_backward(dtype_name, n, h, w, c):
    """Values and recorded positions bit-exact (bf16 data has many ties: the first maximum must win on both sides);
    gradient within one rounding of the exact scatter-sum."""
    import torch

    from paper_2609_10632_b200 import binding as nb

    dt = getattr(torch, dtype_name)
    code = {"float32": nb.NB_DTYPE_F32, "bfloat16": nb.NB_DTYPE_BF16, "float16": nb.NB_DTYPE_F16}[dtype_name]
    rng = np.random.Generator(np.random.Philox(key=[42, n * 100 + c]))
    dev = torch.device("cuda", 0)
    x = torch.from_numpy(rng.standard_normal((n, h, w, c)).astype(np.float32)).to(dt)
    if dtype_name == "bfloat16":
        x = (x.float() * 4).round().div(4).to(dt)  # quarter steps: plenty of exact ties
    g = torch.from_numpy(rng.standard_normal((n, h, w, c)).astype(np.float32)).to(dt)
    xd, gd = x.to(dev), g.to(dev)
    y, idx, dx = torch.empty_like(xd), torch.empty(n, h, w, c, dtype=torch.uint8, device=dev), torch.empty_like(xd)
    nb.nb_maxpool5_fwd(code, n, h, w, c, xd, y, idx)
    nb.nb_maxpool5_bwd(code, n, h, w, c, gd, idx, dx)
    torch.cuda.synchronize()
    ref_y, ref_idx = chain.maxpool5(x.double().numpy())
    np.testing.assert_array_equal(y.double().cpu().numpy(), ref_y)
    np.testing.assert_array_equal(idx.cpu().numpy().astype(np.int64), ref_idx)
    ref_dx = chain.maxpool5_bwd(g.double().numpy(), ref_idx)
    ulp = {"float32": 2.0 ** -23, "bfloat16": 2.0 ** -8, "float16": 2.0 ** -10}[dtype_name]
    # up to 25 terms: in fp32 the running sum rounds after every term (error <= 25 ulp of the largest partial sum);
    # 16-bit terms add exactly in fp32, so those results are one rounding away from the exact sum
    atol = 25 * ulp * float(np.abs(g.double().numpy()).max()) * 5 if dtype_name == "float32" else ulp * 1e-3
    np.testing.assert_allclose(dx.double().cpu().numpy(), ref_dx, rtol=ulp, atol=atol)
    dx1 = dx.clone()
    # accumulate: dx += the same gradient again
    nb.nb_maxpool5_bwd(code, n, h, w, c, gd, idx, dx, accumulate=True)
    torch.cuda.synchronize()
    np.testing.assert_allclose(dx.double().cpu().numpy(), 2 * ref_dx, rtol=4 * ulp, atol=2 * atol)
    # every tensor a channel slice of a wider one (pixel pitches): the same bits, nothing beside the slices touched
    pad = 8 if c % 8 == 0 else 3
    wx, wy = torch.full((n, h, w, c + pad), 3.0, dtype=dt, device=dev), torch.full((n, h, w, c + 2 * pad), 5.0, dtype=dt, device=dev)
    xs, ys = wx[..., pad:], wy[..., pad:pad + c]
    xs.copy_(xd)
    idx2 = torch.empty_like(idx)
    nb.nb_maxpool5_fwd(code, n, h, w, c, xs, ys, idx2, ld_x=xs.stride(-2), ld_y=ys.stride(-2))
    torch.cuda.synchronize()
    assert torch.equal(ys, y) and torch.equal(idx2, idx) and bool((wy[..., :pad] == 5).all()) and bool((wy[..., pad + c:] == 5).all())
    ys.copy_(gd)
    nb.nb_maxpool5_bwd(code, n, h, w, c, ys, idx, xs, ld_g=ys.stride(-2), ld_dx=xs.stride(-2))
    torch.cuda.synchronize()
    assert torch.equal(xs, dx1) and bool((wx[..., :pad] == 3).all())


@pytest.mark.parametrize("dtype_name", ["bfloat16", "float32"])
def test_upsample2_forward_and_adjoint(dtype_name):
    import torch

    from paper_2609_10632_b200 import binding as nb

    dt = getattr(torch, dtype_name)
    code = {"float32": nb.NB_DTYPE_F32, "bfloat16": nb.NB_DTYPE_BF16}[dtype_name]
    n, h, w, c = 2, 5, 7, 12
    rng = np.random.Generator(np.random.Philox(key=[43, 1]))
    dev = torch.device("cuda", 0)
    x = torch.from_numpy(rng.standard_normal((n, h, w, c)).astype(np.float32)).to(dt).to(dev)
    g = torch.from_numpy(rng.standard_normal((n, 2 * h, 2 * w, c)).astype(np.float32)).to(dt).to(dev)
    y, dx = torch.empty(n, 2 * h, 2 * w, c, dtype=dt, device=dev), torch.empty_like(x)
    nb.nb_upsample2(code, n, h, w, c, x, y)
    nb.nb_upsample2(code, n, h, w, c, g, dx, backward=True)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(y.double().cpu().numpy(), chain.upsample2(x.double().cpu().numpy()))
    ref = chain.upsample2_bwd(g.double().cpu().numpy())
    if dtype_name == "bfloat16":  # four 16-bit values sum exactly in fp32: the result is the correctly rounded exact sum
        assert torch.equal(dx, torch.from_numpy(ref).to(dt).to(dev))
    else:
        np.testing.assert_allclose(dx.double().cpu().numpy(), ref, rtol=1e-6, atol=2e-6)  # three fp32 additions with cancellation
    # channel slices of wider tensors on both sides (pixel pitches): the same values, nothing beside the slices touched
    ws = torch.full((n, h, w, c + 8), 7.0, dtype=dt, device=dev)
    wl_ = torch.full((n, 2 * h, 2 * w, c + 16), 9.0, dtype=dt, device=dev)
    xs, yl = ws[..., 4:4 + c], wl_[..., 8:8 + c]
    xs.copy_(x)
    nb.nb_upsample2(code, n, h, w, c, xs, yl, ld_small=xs.stride(-2), ld_large=yl.stride(-2))
    torch.cuda.synchronize()
    assert torch.equal(yl, y) and bool((wl_[..., :8] == 9).all()) and bool((wl_[..., 8 + c:] == 9).all())
    yl.copy_(g)
    nb.nb_upsample2(code, n, h, w, c, yl, xs, backward=True, ld_small=xs.stride(-2), ld_large=yl.stride(-2))
    torch.cuda.synchronize()
    assert torch.equal(xs, dx) and bool((ws[..., :4] == 7).all()) and bool((ws[..., 4 + c:] == 7).all())


def test_sppf_unit_matches_chained_oracle():
    import torch

    from paper_2609_10632_b200.c2f import SppfChain

    ch = SppfChain(2, 20, 20, 64, 64, eps=EPS)
    params, inputs = [], []
    for i, blk in enumerate(ch.blocks):
        inp = wl.make_inputs(blk.shape, 52, i, bf16=True, affine="random")
        inputs.append(inp)
        params.append(chain.BlockParams(inp.w, inp.gamma, inp.beta))
        for name in ("w", "gamma", "beta"):
            dst = getattr(blk, name)
            dst.copy_(torch.from_numpy(np.ascontiguousarray(getattr(inp, name))).to(dst.dtype))
    x, g_out = inputs[0].x, inputs[1].g
    ch.cv1.x.copy_(torch.from_numpy(x).to(torch.bfloat16))
    ch.cv2.g.copy_(torch.from_numpy(g_out).to(torch.bfloat16))
    ch.forward()
    ch.backward()
    torch.cuda.synchronize()
    ch.poll()
    # which window element is the maximum is decided on bf16 activations on the GPU: the oracle decides in the same precision
    out, parts, dx, grads = chain.sppf_fwd_bwd(x, params, EPS, g_out, pool_in_bf16=True)
    f64 = lambda t: t.detach().double().cpu().numpy()
    report = []
    # unique results: the forward and everything of the backward that does not pass through a pool
    _check("out", f64(ch.cv2.a), out, report)
    cat = f64(ch.cat)
    for j, part in enumerate(parts):
        _check(f"part{j}", cat[..., j * ch.c:(j + 1) * ch.c], part, report)
    _check("cv2.dw", f64(ch.cv2.dw), grads[1][0], report)
    _check("cv2.dgamma", f64(ch.cv2.dgamma), grads[1][1], report)
    _check("cv2.dbeta", f64(ch.cv2.dbeta), grads[1][2], report)
    # The gradient behind the pools is NOT unique: the GPU's activations differ from the oracle's by a bf16 ulp in many
    # elements (they pass through the fp16 convolution output), so a few per cent of the windows have a different, equally
    # valid maximum position and their gradient lands on a neighbouring pixel.  Checked instead: (1) every recorded
    # position IS the first maximum of the GPU's own window (the decision is valid), (2) the pools' gradient routing
    # conserves the gradient mass per channel, (3) the results stay close to the oracle's (loose bar).
    src = f64(ch.cv1.a)
    for j in range(3):
        want_y, want_idx = chain.maxpool5(src)
        np.testing.assert_array_equal(f64(ch.pool[j]), want_y)
        np.testing.assert_array_equal(ch.idx[j].cpu().numpy().astype(np.int64), want_idx)
        src = want_y
    dcat = f64(ch.dcat)
    mass = sum(dcat[..., j * ch.c:(j + 1) * ch.c].sum(axis=(0, 1, 2)) for j in range(4))
    l1 = sum(np.abs(dcat[..., j * ch.c:(j + 1) * ch.c]).sum(axis=(0, 1, 2)) for j in range(4))
    # every stored gradient value carries a bf16 rounding (2^-9 relative), three accumulations deep
    np.testing.assert_allclose(f64(ch.dpart[0]).sum(axis=(0, 1, 2)), mass, rtol=0, atol=float((4 * 2.0 ** -9 * l1).max()))
    for name, got, ref in (("dx", ch.cv1.dx, dx), ("cv1.dw", ch.cv1.dw, grads[0][0]), ("cv1.dgamma", ch.cv1.dgamma, grads[0][1]), ("cv1.dbeta", ch.cv1.dbeta, grads[0][2])):
        r = parity.rel_l2(f64(got), ref)
        report.append(f"{name} (behind the pools): rel_l2={r:.2e}")
        assert r <= 0.1, name
    print("\n".join(report))


def test_detector_dataflow_matches_graph_oracle():
    """All 77 blocks chained as the detector's dataflow (batch 2, 256 x 256 image: the coarsest level is 8 x 8) against the
    oracle's interpretation of the same description.

    A deep randomly initialised BN network amplifies perturbations from block to block: in the oracle alone, rounding the
    stored tensors to 16 bits (its storage mode) moves the results away from the exact fp64 graph by 2e-3 after the first
    block, 2e-2 after the third C2f unit and 0.2 at the heads, and two 16-bit runs that round slightly differently drift
    apart just as much.  No fixed small tolerance is meaningful at that depth, so the oracle's own drift is the
    yardstick: for every tensor of the forward pass and every block's dw, dgamma, dbeta the GPU's distance from the exact
    graph must stay within TWICE the distance of the oracle's 16-bit storage run from the exact graph (+ 5e-3).  A wiring
    mistake (a missing shortcut, a wrong slice, a dropped gradient contribution) is an O(1) error from the first
    affected tensor on, where the yardstick is still a few 1e-3.  The yardstick also absorbs the non-uniqueness of the
    gradients behind the max-pools (see the SPPF test), because the storage run's pools flip in the same way."""
    import torch

    from paper_2609_10632_b200.detector import GraphRunner

    ops, layers, outs, plain = wl.detector_graph(2, 256, plain_head=True)  # up to the six raw head outputs
    run = GraphRunner(ops, layers, outs, eps=EPS, plain_layers=plain)  # channel-slice views: split / concat without copies
    pparams = []
    for j, pl in enumerate(run.plain):
        w = wl.make_inputs(plain[j], 54, j, bf16=True).w
        bias = wl.make_eval_stats(plain[j], 54, j)[2]
        pparams.append((w, bias))
        pl["w"].copy_(torch.from_numpy(w).to(torch.bfloat16))
        pl["bias"].copy_(torch.from_numpy(bias))
    kw = dict(plain_layers=plain, plain_params=pparams)
    params = []
    for k, blk in enumerate(run.blocks):
        inp = wl.make_inputs(layers[k], 53, k, bf16=True, affine="random")
        params.append(chain.BlockParams(inp.w, inp.gamma, inp.beta))
        for name in ("w", "gamma", "beta"):
            dst = getattr(blk, name)
            dst.copy_(torch.from_numpy(np.ascontiguousarray(getattr(inp, name))).to(dst.dtype))
    x = wl.make_inputs(layers[0], 53, 0, bf16=True).x
    run.buf["img"].copy_(torch.from_numpy(x).to(torch.bfloat16))
    gouts = {}
    for j, name in enumerate(outs):
        rng = np.random.Generator(np.random.Philox(key=[53, 5000 + j]))
        g = wl.round_to_bf16(rng.standard_normal(run.shape[name], dtype=np.float32))
        gouts[name] = g
        run.grad[name].copy_(torch.from_numpy(g).to(torch.bfloat16))
    run.forward()
    run.backward()
    torch.cuda.synchronize()
    run.poll()
    f64 = lambda t: t.detach().double().cpu().numpy()
    T0, G0, b0, q0 = chain.graph_fwd_bwd(ops, layers, params, x, EPS, gouts, **kw)                      # exact
    T1, G1, b1, q1 = chain.graph_fwd_bwd(ops, layers, params, x, EPS, gouts, storage_16bit=True, **kw)  # the yardstick
    worst = {"ratio": 0.0, "gpu": 0.0, "yardstick": 0.0}

    def held(name, got, exact, stored):
        e, y = parity.rel_l2(got, exact), parity.rel_l2(stored, exact)
        assert np.isfinite(got).all(), name
        worst["ratio"], worst["gpu"], worst["yardstick"] = max(worst["ratio"], e / (y + 2.5e-3)), max(worst["gpu"], e), max(worst["yardstick"], y)
        assert e <= 2 * y + 5e-3, (name, e, y)

    for name in T0:
        if name != "img" and name not in run.fused_v:  # (the output of a block that adds its shortcut itself exists only as the sum)
            held(name, f64(run.buf[name]), T0[name], T1[name])
    held("d img", f64(run.grad["img"]), G0["img"], G1["img"])
    for k, blk in enumerate(run.blocks):
        for slot, t in enumerate((blk.dw, blk.dgamma, blk.dbeta)):
            held(f"{layers[k].name}.{('dw', 'dgamma', 'dbeta')[slot]}", f64(t), b0[k][slot], b1[k][slot])
    for j, pl in enumerate(run.plain):
        held(f"{plain[j].name}.dw", f64(pl["dw"]), q0[j][0], q1[j][0])
        held(f"{plain[j].name}.dbias", f64(pl["dbias"]), q0[j][1], q1[j][1])
    print("worst:", {k: f"{v:.2e}" for k, v in worst.items()}, "glue launches fwd/bwd:", run.glue_launches())


@pytest.mark.parametrize("batch,image", [(2, 128), (4, 320)], ids=["b2-128", "b4-320"])
def test_detector_stage_by_stage_against_the_oracle_on_the_gpus_own_inputs(batch, image):
    """The localising check: every operation of the 77-block dataflow is verified on its own.  The oracle's operation is
    applied to the tensors the GPU itself fed into that operation, and the GPU's output is held to the SINGLE-BLOCK
    bars (relative L2 <= 5e-3, |err| <= 5e-2 * rms; copies, adds, pools and upsampling bit-exactly).  Nothing drifts, so a
    wiring or arithmetic fault at any depth shows at the operation that has it, at full tolerance.  Forward: a block's
    a, y, mean, invstd from its input; backward: dy, dgamma, dbeta from (g, y, mean, invstd), dx from dy, dw from
    (x, dy); the gradient of every tensor is the sum of its consumers' contributions.  The larger case (batch 4,
    320 x 320) reaches multi-tile launches with channel-slice (pitched) operands on every level."""
    import torch

    from paper_2609_10632_b200.detector import GraphRunner

    ops, layers, outs, plain = wl.detector_graph(batch, image, plain_head=True)
    run = GraphRunner(ops, layers, outs, eps=EPS, plain_layers=plain)
    params, pparams = [], []
    for j, pl in enumerate(run.plain):
        w = wl.make_inputs(plain[j], 56, j, bf16=True).w
        bias = wl.make_eval_stats(plain[j], 56, j)[2]
        pparams.append((w, bias))
        pl["w"].copy_(torch.from_numpy(w).to(torch.bfloat16))
        pl["bias"].copy_(torch.from_numpy(bias))
    for k, blk in enumerate(run.blocks):
        inp = wl.make_inputs(layers[k], 55, k, bf16=True, affine="random")
        params.append(chain.BlockParams(inp.w, inp.gamma, inp.beta))
        for name in ("w", "gamma", "beta"):
            dst = getattr(blk, name)
            dst.copy_(torch.from_numpy(np.ascontiguousarray(getattr(inp, name))).to(dst.dtype))
    run.buf["img"].copy_(torch.from_numpy(wl.make_inputs(layers[0], 55, 0, bf16=True).x).to(torch.bfloat16))
    for j, name in enumerate(outs):
        rng = np.random.Generator(np.random.Philox(key=[55, 5000 + j]))
        run.grad[name].copy_(torch.from_numpy(wl.round_to_bf16(rng.standard_normal(run.shape[name], dtype=np.float32))).to(torch.bfloat16))
    # With channel-slice views the gradient of a tensor placed inside a concatenation buffer lives in the consuming block's
    # dx buffer, where later contributions are added in place: keep each block's own dx as it was right after its call.
    # A block that adds its data gradient straight into a shared gradient buffer (nb_cbs_plan_set_dx_target): keep the
    # buffer as it was before the call too.
    adds = {o["layer"] for oi, o in enumerate(ops) if o["op"] == "cbs" and oi in run.direct_dx and run.acc[(oi, 0)]}
    for k, blk in enumerate(run.blocks):
        def keep_dx(stream=None, _call=blk.backward_data, _blk=blk, _adds=k in adds):
            _blk.dx_before = _blk.dx.clone() if _adds else None
            _call(stream)
            _blk.dx_own = _blk.dx.clone()
        blk.backward_data = keep_dx
    run.forward()
    run.backward()
    torch.cuda.synchronize()
    run.poll()
    f64 = lambda t: t.detach().double().cpu().numpy()
    B, G = run.buf, run.grad
    worst = {}
    dx_of_consumer = {o["ins"][0]: run.blocks[o["layer"]] for o in ops if o["op"] == "cbs"}  # tensor -> the block that reads it

    def bar(stage, name, got, ref):
        # The tensors inside a deep network are heavy-tailed (single elements at 30 x rms and more), and a stored bf16
        # value is off by up to 2^-9 of its own magnitude whatever the arithmetic did: the per-element bar allows that one
        # rounding on top of 5e-2 * rms.  The relative-L2 bar is unchanged.
        assert got.shape == ref.shape and np.isfinite(got).all(), (name, stage)
        r = parity.rel_l2(got, ref)
        rms = float(np.sqrt((ref * ref).mean()))
        m = float((np.abs(got - ref) - 2.0**-9 * np.abs(ref)).max()) / rms if rms > 0 else 0.0
        assert r <= parity.BF16_REL_L2, f"{name}.{stage}: rel L2 {r:.3e}"
        assert m <= parity.BF16_MAX_OVER_RMS, f"{name}.{stage}: (max|err| - one bf16 rounding)/rms {m:.3e}"
        w = worst.setdefault(stage, [0.0, 0.0])
        w[0], w[1] = max(w[0], r), max(w[1], m)

    def same(name, got, ref):
        np.testing.assert_array_equal(got, ref, err_msg=name)

    contrib = {}  # tensor -> list of gradient contributions of its consumers (fp64, full shape of the tensor)

    def give(name, g, c0=None):
        if c0 is None:
            contrib.setdefault(name, []).append(g)
        else:
            full = np.zeros(run.shape[name])
            full[..., c0:c0 + g.shape[-1]] = g
            contrib.setdefault(name, []).append(full)

    for o in ops:
        kind, out, ins = o["op"], o["out"], o["ins"]
        x = f64(B[ins[0]])
        if kind == "cbs":
            k = o["layer"]
            blk, prm, st = run.blocks[k], params[k], layers[k].stride
            f = oracle.cbs_fwd(x, prm.w, prm.gamma, prm.beta, st, EPS)
            if out in run.fused_v:  # the block adds the bottleneck's shortcut itself: its output tensor is the sum
                bar("a + shortcut", out, f64(B[out]), f.a + f64(B[run.fused_v[out]["ins"][0]]))
            else:
                bar("a", out, f64(B[out]), f.a)
            bar("y", out, f64(blk.y), f.y)
            parity.check_stats(f64(blk.mean), f64(blk.invstd), f.y, EPS, "bf16")
            # backward stages, each from the GPU's own inputs of that stage
            y_gpu, dy_gpu = f64(blk.y), f64(blk.dy)
            dy, dgamma, dbeta = oracle.bn_silu_bwd(f64(G[out]), y_gpu, f64(blk.mean), f64(blk.invstd), prm.gamma, prm.beta)
            bar("dy", out, dy_gpu, dy)
            bar("dgamma", out, f64(blk.dgamma), dgamma)
            bar("dbeta", out, f64(blk.dbeta), dbeta)
            bar("dw", out, f64(blk.dw), oracle.conv_wgrad(x, dy_gpu, layers[k].k, st))
            want_dx = oracle.conv_dgrad(dy_gpu, prm.w, x.shape, st)
            if blk.dx_before is None:
                bar("dx", out, f64(blk.dx_own), want_dx)
                give(ins[0], f64(blk.dx_own))
            else:  # the buffer after the call = what it held before + this block's data gradient (one rounding)
                bar("dx (added)", out, f64(blk.dx_own), f64(blk.dx_before) + want_dx)
                give(ins[0], f64(blk.dx_own) - f64(blk.dx_before))
        elif kind == "plain":
            k = o["layer"]
            pl, (w, bias) = run.plain[k], pparams[k]
            bar("out", out, f64(B[out]), oracle.conv_bias_act(x, w, bias, plain[k].stride))
            dx, dw, db = oracle.conv_bias_bwd(x, w, f64(G[out]), plain[k].stride)
            bar("dx", out, f64(pl["dx"]), dx)
            bar("dw", out, f64(pl["dw"]), dw)
            bar("dbias", out, f64(pl["dbias"]), db)
            give(ins[0], f64(pl["dx"]))
        elif kind == "slice":
            same(out, f64(B[out]), x[..., o["c0"]:o["c1"]])
            give(ins[0], f64(G[out]), o["c0"])
        elif kind == "add":
            give(ins[0], f64(G[out]))
            if ins[1] not in run.fused_v:  # (a fused add was checked with the block that performs it)
                same(out, f64(B[out]), chain.round_bf16(x + f64(B[ins[1]])))
                give(ins[1], f64(G[out]))
        elif kind == "concat":
            same(out, f64(B[out]), np.concatenate([f64(B[i]) for i in ins], axis=-1))
            # (the concatenation's own gradient is the consuming block's dx before anything was added into it)
            c0, g = 0, f64(dx_of_consumer[out].dx_own if out in dx_of_consumer else G[out])
            for name in ins:
                c = run.shape[name][3]
                give(name, g[..., c0:c0 + c])
                c0 += c
        elif kind == "maxpool":
            want, idx = chain.maxpool5(x)
            same(out, f64(B[out]), want)
            same(out + ".idx", run.idx[out].cpu().numpy().astype(np.int64), idx)
            give(ins[0], chain.maxpool5_bwd(f64(G[out]), idx))
        elif kind == "upsample":
            same(out, f64(B[out]), chain.upsample2(x))
            give(ins[0], chain.upsample2_bwd(f64(G[out])))
    # gradient accumulation at fan-out: the stored gradient of a tensor is the sum of its consumers' contributions
    # (bf16-rounded after each addition on the GPU: the same bars)
    for name, parts in contrib.items():
        if name in outs:
            continue
        if len(parts) == 1:
            # one consumer: a block's dx IS the stored gradient (checked above, and tensors placed inside it add to it
            # later); any other single contribution must have been stored unchanged
            if name not in dx_of_consumer:
                same("d " + name, f64(G[name]), parts[0])
        else:
            bar("fan-out", name, f64(G[name]), np.sum(parts, axis=0))
    print("worst per stage (rel L2, max/rms):", {k: (f"{v[0]:.2e}", f"{v[1]:.2e}") for k, v in worst.items()})


def test_chained_detector_in_the_benchmarks_launch_configuration_is_bitwise_the_plain_run():
    """bench.py replays the chained detector as a CUDA graph with the weight gradients on a second stream: that launch
    configuration must give bit for bit what the plain single-stream eager run (checked against the oracle above) gives."""
    import torch

    from paper_2609_10632_b200.detector import GraphRunner

    ops, layers, outs = wl.detector_graph(2, 128)
    run = GraphRunner(ops, layers, outs, eps=EPS)
    gen = torch.Generator(device=run.dev)
    gen.manual_seed(7)
    run.fill_parameters(seed=100)
    img = torch.rand(run.shape["img"], generator=gen, device=run.dev).to(torch.bfloat16)
    gout = {n: torch.randn(run.shape[n], generator=gen, device=run.dev).to(torch.bfloat16) for n in outs}

    def load():
        run.buf["img"].copy_(img)
        for n in outs:
            run.grad[n].copy_(gout[n])

    load()
    run.forward()
    run.backward()
    torch.cuda.synchronize()
    want = [(b.dw.clone(), b.dgamma.clone(), b.dbeta.clone()) for b in run.blocks]
    want_dimg = run.grad["img"].clone()
    side = torch.cuda.Stream()
    side_ws = torch.empty(max(b.plan.bwd_bytes for b in run.blocks), dtype=torch.uint8, device=run.dev)

    def step():
        main = torch.cuda.current_stream()
        run.forward()
        side.wait_stream(main)
        run.backward(wgrad_stream=side, wgrad_workspace=side_ws)
        main.wait_stream(side)

    load()
    step()  # eager, two streams
    torch.cuda.synchronize()
    for b in run.blocks:
        b.dw.zero_()
    cap = torch.cuda.Stream()
    cap.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(cap):
        with torch.cuda.graph(graph, stream=cap):
            step()
    torch.cuda.current_stream().wait_stream(cap)
    load()
    graph.replay()
    torch.cuda.synchronize()
    run.poll()
    for b, (dw, dgamma, dbeta) in zip(run.blocks, want):
        assert torch.equal(b.dw, dw) and torch.equal(b.dgamma, dgamma) and torch.equal(b.dbeta, dbeta), b.shape.name
    assert torch.equal(run.grad["img"], want_dimg)


def test_views_and_copies_give_the_same_bits():
    """GraphRunner(views=True) places tensors inside concatenation buffers and hands channel slices to the calls;
    views=False copies.  Same arithmetic on the same values: every forward tensor and every gradient must agree bit for
    bit, and the views must save most of the glue launches."""
    import torch

    from paper_2609_10632_b200.detector import GraphRunner

    ops, layers, outs, plain = wl.detector_graph(2, 128, plain_head=True)
    runs = [GraphRunner(ops, layers, outs, eps=EPS, plain_layers=plain, views=v) for v in (True, False)]
    gen = torch.Generator(device=runs[0].dev)
    gen.manual_seed(11)
    img = torch.rand(runs[0].shape["img"], generator=gen, device=runs[0].dev).to(torch.bfloat16)
    gout = {n: torch.randn(runs[0].shape[n], generator=gen, device=runs[0].dev).to(torch.bfloat16) for n in outs}
    for r in runs:
        r.fill_parameters(seed=200)
        for j, pl in enumerate(r.plain):
            g2 = torch.Generator(device=r.dev)
            g2.manual_seed(300 + j)
            pl["w"].copy_(torch.randn(pl["w"].shape, generator=g2, device=r.dev) * 0.05)
            pl["bias"].copy_(torch.randn(pl["bias"].shape, generator=g2, device=r.dev) * 0.5)
        r.buf["img"].copy_(img)
        for n in outs:
            r.grad[n].copy_(gout[n])
        r.forward()
        r.backward()
    torch.cuda.synchronize()
    a, b = runs
    a.poll()
    b.poll()
    for name in a.buf:
        assert torch.equal(a.buf[name], b.buf[name]), name
    assert torch.equal(a.grad["img"], b.grad["img"])
    for x, y in zip(a.blocks, b.blocks):
        assert torch.equal(x.dw, y.dw) and torch.equal(x.dgamma, y.dgamma) and torch.equal(x.dbeta, y.dbeta), x.shape.name
    for x, y in zip(a.plain, b.plain):
        assert torch.equal(x["dw"], y["dw"]) and torch.equal(x["dbias"], y["dbias"])
    va, vb = sum(a.glue_launches()), sum(b.glue_launches())
    print("glue launches with views", a.glue_launches(), "with copies", b.glue_launches(), "placed", len(a.placed), "slice views", len(a.slice_view))
    assert va < 0.6 * vb


def test_the_shortcut_gradient_inside_the_dy_pass_gives_the_same_bits():
    """GraphRunner(fuse_shortcut_grad=True) lets the block that performs a residual add also hand the sum's gradient to the
    shortcut (nb_cbs_plan_set_bwd_residual) instead of a glue launch per bottleneck: same additions in the same order, so
    every gradient agrees bit for bit, with twelve launches fewer."""
    import torch

    from paper_2609_10632_b200.detector import GraphRunner

    ops, layers, outs, plain = wl.detector_graph(2, 128, plain_head=True)
    runs = [GraphRunner(ops, layers, outs, eps=EPS, plain_layers=plain, fuse_shortcut_grad=f) for f in (True, False)]
    gen = torch.Generator(device=runs[0].dev)
    gen.manual_seed(13)
    img = torch.rand(runs[0].shape["img"], generator=gen, device=runs[0].dev).to(torch.bfloat16)
    gout = {n: torch.randn(runs[0].shape[n], generator=gen, device=runs[0].dev).to(torch.bfloat16) for n in outs}
    for r in runs:
        r.fill_parameters(seed=210)
        for j, pl in enumerate(r.plain):
            g2 = torch.Generator(device=r.dev)
            g2.manual_seed(310 + j)
            pl["w"].copy_(torch.randn(pl["w"].shape, generator=g2, device=r.dev) * 0.05)
            pl["bias"].copy_(torch.randn(pl["bias"].shape, generator=g2, device=r.dev) * 0.5)
        r.buf["img"].copy_(img)
        for n in outs:
            r.grad[n].copy_(gout[n])
        r.forward()
        r.backward()
    torch.cuda.synchronize()
    a, b = runs
    a.poll()
    b.poll()
    assert len(a.shortcut_by_block) == 12 and not b.shortcut_by_block
    assert torch.equal(a.grad["img"], b.grad["img"])
    for x, y in zip(a.blocks, b.blocks):
        assert torch.equal(x.dw, y.dw) and torch.equal(x.dgamma, y.dgamma) and torch.equal(x.dbeta, y.dbeta), x.shape.name
    assert sum(a.glue_launches()) == sum(b.glue_launches()) - 12

