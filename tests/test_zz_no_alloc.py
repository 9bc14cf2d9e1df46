"""nb_bn_stats_static: the batch-statistics entry point for callers that cannot allocate device memory.

Hosts that run under an allocator they do not control (or under a fixed memory budget) can neither create a plan
nor hand over a workspace; this entry point keeps its partial sums in an array built into the library instead.
The test calls it through the C ABI twice in a row -- the second time on a different, smaller tensor, so that stale
contents of the shared array from the first call would show -- and checks each result against the CPU oracle's
statistics of the same tensor and against nb_bn_stats (the plan + workspace entry point) within the tolerance the
other statistics tests use.  It also covers the documented limits and checks that sizes beyond the built-in array
are refused.  This file is collected last on purpose.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

EPS = 1e-3


def _reference_stats(nb, torch, ty, shape_m, c, mode, tag):
    # any block shape with N*Ho*Wo == m and c_out == c gives the plan nb_bn_stats needs
    plan = nb.Plan(1, 1, shape_m, 8, c, 1, 1, eps=EPS, mode=mode)
    assert plan.m == shape_m
    outs = [torch.empty(c, dtype=torch.float32, device="cuda") for _ in range(4)]
    ws = torch.empty(plan.fwd_bytes, dtype=torch.uint8, device="cuda")
    nb.nb_bn_stats(plan, ty, tag, *outs, ws)
    torch.cuda.synchronize()
    return [o.cpu().numpy() for o in outs]


def _check_against_oracle_and_workspace_call(nb, torch, dt, tag, mode, m, c, rng, with_sums=True):
    import oracle

    y = (rng.normal(size=(m, c)) * rng.uniform(0.5, 2.0, c) + rng.normal(size=c) * 2.0).astype(np.float32)
    ty = torch.from_numpy(y).to(dt).cuda()
    got = [torch.full((c,), float("nan"), dtype=torch.float32, device="cuda") for _ in range(4)]
    if with_sums:
        nb.nb_bn_stats_static(ty, tag, m, c, EPS, *got)
    else:
        nb.nb_bn_stats_static(ty, tag, m, c, EPS, got[0], got[1])  # sum and sumsq are optional (NULL)
    torch.cuda.synchronize()
    # (a) the CPU oracle on the very values the GPU read (the 16-bit tensor widened): only the order of the fp32 / fp64
    # additions differs, so the results agree to about 1e-6
    yd = ty.double().cpu().numpy()
    o_mean, o_var, o_invstd = oracle.bn_stats(yd, EPS)
    rms = np.sqrt(o_mean**2 + o_var)
    g_mean, g_invstd = got[0].cpu().numpy().astype(np.float64), got[1].cpu().numpy().astype(np.float64)
    assert np.isfinite(g_mean).all() and np.isfinite(g_invstd).all()
    assert (np.abs(g_mean - o_mean) / rms).max() <= 2e-6
    # (single-pass variance from fp32 partial sums: the relative error of var, hence of invstd, grows with mean^2 / var)
    assert (np.abs(g_invstd - o_invstd) / o_invstd / (1.0 + o_mean**2 / (o_var + EPS))).max() <= 1e-6
    if with_sums:
        np.testing.assert_allclose(got[2].cpu().numpy(), yd.sum(0), rtol=2e-6, atol=2e-6 * float((rms * m).max()))
        np.testing.assert_allclose(got[3].cpu().numpy(), (yd * yd).sum(0), rtol=2e-6)
    # (b) the existing entry point (plan + workspace), same tolerance as the other statistics tests
    want = _reference_stats(nb, torch, ty, m, c, mode, tag)
    for name, g, w in zip(("mean", "invstd", "sum", "sumsq"), got if with_sums else got[:2], want):
        g = g.cpu().numpy()
        atol = 1e-6 if name in ("mean", "invstd") else 1e-3 * max(1.0, float(np.abs(w).max()) * 1e-3)
        np.testing.assert_allclose(g, w, rtol=1e-5, atol=atol, err_msg=name)


def _dtype_args(nb, torch, dtype_name):
    if dtype_name == "f16":
        return torch.float16, nb.NB_DTYPE_F16, nb.NB_MODE_BF16_TC
    return torch.float32, nb.NB_DTYPE_F32, nb.NB_MODE_F32_REF


@pytest.mark.parametrize("dtype_name", ["f16", "f32"])
def test_static_scratch_stats_match_workspace_stats_twice_in_a_row(dtype_name):
    import torch

    from paper_2609_10632_b200 import binding as nb

    dt, tag, mode = _dtype_args(nb, torch, dtype_name)
    rng = np.random.default_rng(7)
    for m, c in ((50_000, 192), (3_001, 48)):  # second call: fewer rows and channels than the first
        _check_against_oracle_and_workspace_call(nb, torch, dt, tag, mode, m, c, rng)


@pytest.mark.parametrize("dtype_name,m,c,with_sums", [("f16", 700, 1024, True), ("f32", 700, 1024, True), ("f16", 999, 24, True), ("f16", 4_000, 96, False)],
                         ids=["f16-c1024", "f32-c1024", "f16-c24", "f16-no-sums"])
def test_static_scratch_stats_at_the_limits(dtype_name, m, c, with_sums):
    """The documented maximum of 1024 channels in both dtypes (one and two rows of vectors per block), a channel-group
    count that does not divide the block size (c = 24 in fp16: 255 threads), and the optional outputs left out."""
    import torch

    from paper_2609_10632_b200 import binding as nb

    dt, tag, mode = _dtype_args(nb, torch, dtype_name)
    _check_against_oracle_and_workspace_call(nb, torch, dt, tag, mode, m, c, np.random.default_rng(11), with_sums)


def test_static_scratch_rejects_sizes_beyond_its_array():
    import torch

    from paper_2609_10632_b200 import binding as nb

    y = torch.zeros(4, 2048, dtype=torch.float16, device="cuda")
    mean = torch.full((2048,), 5.0, dtype=torch.float32, device="cuda")
    invstd = torch.full((2048,), 5.0, dtype=torch.float32, device="cuda")
    with pytest.raises(nb.NbError) as ei:
        nb.nb_bn_stats_static(y, nb.NB_DTYPE_F16, 4, 2048, EPS, mean, invstd)
    assert ei.value.status == nb.NB_ERR_UNSUPPORTED and "1024" in str(ei.value)
    with pytest.raises(nb.NbError) as ei:
        nb.nb_bn_stats_static(y, nb.NB_DTYPE_F16, 1, 64, EPS, mean, invstd)
    assert ei.value.status == nb.NB_ERR_INVALID_ARG
    with pytest.raises(nb.NbError) as ei:
        nb.nb_bn_stats_static(y, nb.NB_DTYPE_BF16, 4, 64, EPS, mean, invstd)
    assert ei.value.status == nb.NB_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert bool((mean == 5.0).all()) and bool((invstd == 5.0).all())
