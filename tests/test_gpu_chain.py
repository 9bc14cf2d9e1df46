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
