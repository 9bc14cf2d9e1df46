"""nb_bn_stats_static: the batch-statistics entry point for callers that cannot allocate device memory.

Hosts that run under an allocator they do not control (or under a fixed memory budget) can neither create a plan
nor hand over a workspace; this entry point keeps its partial sums in an array built into the library instead.
The test calls it through the C ABI twice in a row -- the second time on a different, smaller tensor, so that stale
contents of the shared array from the first call would show -- and checks each result against nb_bn_stats (the
plan + workspace entry point) within the tolerance the other statistics tests use.  It also checks that sizes
beyond the built-in array are refused.  This file is collected last on purpose.
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


@pytest.mark.parametrize("dtype_name", ["f16", "f32"])
def test_static_scratch_stats_match_workspace_stats_twice_in_a_row(dtype_name):
    import torch

    from paper_2609_10632_b200 import binding as nb

    dt, tag, mode = (torch.float16, nb.NB_DTYPE_F16, nb.NB_MODE_BF16_TC) if dtype_name == "f16" else (torch.float32, nb.NB_DTYPE_F32, nb.NB_MODE_F32_REF)
    rng = np.random.default_rng(7)
    for m, c in ((50_000, 192), (3_001, 48)):  # second call: fewer rows and channels than the first
        y = (rng.normal(size=(m, c)) * rng.uniform(0.5, 2.0, c) + rng.normal(size=c) * 2.0).astype(np.float32)
        ty = torch.from_numpy(y).to(dt).cuda()
        got = [torch.full((c,), float("nan"), dtype=torch.float32, device="cuda") for _ in range(4)]
        nb.nb_bn_stats_static(ty, tag, m, c, EPS, *got)
        torch.cuda.synchronize()
        want = _reference_stats(nb, torch, ty, m, c, mode, tag)
        for name, g, w in zip(("mean", "invstd", "sum", "sumsq"), got, want):
            g = g.cpu().numpy()
            assert np.isfinite(g).all(), name
            atol = 1e-6 if name in ("mean", "invstd") else 1e-3 * max(1.0, float(np.abs(w).max()) * 1e-3)
            np.testing.assert_allclose(g, w, rtol=1e-5, atol=atol, err_msg=name)


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
