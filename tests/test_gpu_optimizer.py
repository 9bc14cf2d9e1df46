"""Fused global-norm clip + SGD-Nesterov step (include/nb_sgd.h) on the GPU against the fp64 oracle, element by element.

fp32 arithmetic on the GPU: relative L2 <= 1e-5 per tensor (the fp32 bar of the block calls; observed ~1e-7); the bf16
working copy must be bit-exactly the round-to-nearest-even of the GPU's own fp32 parameter (an integer decision taken
in the kernel's precision) and two runs must agree bit for bit (fixed-order sums)."""
import numpy as np
import pytest

from oracle import optimizer as opt
from paper_2609_10632_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

LR = [0.01, 0.02, 0.1]
WD = [3.75e-4, 0.0, 0.0]  # Table 1: 5e-4 scaled by the effective batch 48/64
MOM = 0.937
MAX_NORM = 10.0


class State:
    def __init__(self, sizes, groups, cfg_id, with_bf16=True):
        import torch

        from paper_2609_10632_b200 import binding as nb

        self.torch, self.nb = torch, nb
        dev = torch.device("cuda", 0)
        self.sizes, self.groups, self.cfg_id = list(sizes), list(groups), cfg_id
        params, _ = wl.make_optimizer_inputs(self.sizes, cfg_id, 0)
        self.h_params = [p.astype(np.float64) for p in params]
        self.h_bufs = [None] * len(sizes)
        self.p = [torch.from_numpy(p).to(dev) for p in params]
        self.g = [torch.empty(n, dtype=torch.float32, device=dev) for n in sizes]
        self.m = [torch.full((n,), float("nan"), dtype=torch.float32, device=dev) for n in sizes]  # first_step must ignore the contents
        self.lp = [torch.empty(n, dtype=torch.bfloat16, device=dev) if (with_bf16 and grp == 0) else None for n, grp in zip(sizes, groups)]
        self.plan = nb.SgdPlan(zip(self.g, self.p, self.m, self.lp, self.groups))
        self.ws = torch.empty(self.plan.workspace_bytes, dtype=torch.uint8, device=dev)
        self.plan.upload(self.ws)
        self.norm = torch.zeros(1, dtype=torch.float32, device=dev)

    def step(self, k, grad_scale, check=True):
        torch = self.torch
        _, grads = wl.make_optimizer_inputs(self.sizes, self.cfg_id, k, grad_scale)
        for d, h in zip(self.g, grads):
            d.copy_(torch.from_numpy(h))
        self.plan.step(self.ws, LR, WD, MOM, MAX_NORM, first_step=(k == 0), total_norm=self.norm)
        torch.cuda.synchronize()
        self.h_params, self.h_bufs, total = opt.clip_sgd_step(self.h_params, grads, self.h_bufs, self.groups, LR, WD, MOM, MAX_NORM, first_step=(k == 0))
        if check:
            assert float(self.norm.item()) == pytest.approx(total, rel=2e-6)
            for i in range(len(self.sizes)):
                parity.check(f"param[{i}]", self.p[i].double().cpu().numpy(), self.h_params[i], "f32")
                parity.check(f"momentum[{i}]", self.m[i].double().cpu().numpy(), self.h_bufs[i], "f32")
                if self.lp[i] is not None:
                    assert torch.equal(self.lp[i], self.p[i].to(torch.bfloat16)), f"bf16 copy of tensor {i}"
        return total


def test_small_lists_ragged_sizes_three_steps():
    sizes = [5000, 3, 4096, 4097, 12289, 1, 8, 640]  # tails of 0..3 elements, tensors below one vector, several chunks
    groups = [0, 2, 0, 1, 0, 2, 1, 0]
    st = State(sizes, groups, cfg_id=31)
    totals = [st.step(0, 0.5), st.step(1, 0.01), st.step(2, 0.2)]
    assert totals[0] > MAX_NORM > totals[1]  # the first step clips, the second does not


def test_clipping_disabled_and_single_tensor():
    import torch

    st = State([1000], [0], cfg_id=32, with_bf16=False)
    _, grads = wl.make_optimizer_inputs(st.sizes, 32, 0, 5.0)
    st.g[0].copy_(torch.from_numpy(grads[0]))
    p0 = st.h_params[0].copy()
    st.plan.step(st.ws, LR, WD, 0.0, 0.0, first_step=True, total_norm=None)  # max_norm 0: no clipping; momentum 0: plain descent
    torch.cuda.synchronize()
    want = p0 - LR[0] * (grads[0].astype(np.float64) + WD[0] * p0)
    parity.check("param", st.p[0].double().cpu().numpy(), want, "f32")


def test_detector_parameter_list_full_size_and_reproducible():
    """The 243 tensors / 25.9 M parameters of the detector: two steps against the oracle, then bitwise reproducibility."""
    import torch

    tensors = wl.detector_parameter_tensors()
    sizes, groups = [n for _, n, _ in tensors], [g for _, _, g in tensors]
    assert len(sizes) == 243
    st = State(sizes, groups, cfg_id=33)
    assert st.step(0, 0.01) > MAX_NORM  # sqrt(25.9e6) * 0.01 = 51: clipped
    st.step(1, 0.001)                   # 5.1: not clipped
    snap = [p.clone() for p in st.p]
    st2 = State(sizes, groups, cfg_id=33)
    st2.step(0, 0.01, check=False)
    st2.step(1, 0.001, check=False)
    for a, b in zip(snap, st2.p):
        assert torch.equal(a, b)


def test_step_inside_a_cuda_graph():
    import torch

    sizes, groups = [20000, 64, 64], [0, 1, 2]
    st = State(sizes, groups, cfg_id=34)
    st.step(0, 0.3)
    _, grads = wl.make_optimizer_inputs(sizes, 34, 1, 0.3)
    for d, h in zip(st.g, grads):
        d.copy_(torch.from_numpy(h))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            st.plan.step(st.ws, LR, WD, MOM, MAX_NORM, first_step=False, total_norm=st.norm)
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    torch.cuda.synchronize()
    want_p, want_b, total = opt.clip_sgd_step(st.h_params, grads, st.h_bufs, groups, LR, WD, MOM, MAX_NORM, first_step=False)
    for i in range(3):
        parity.check(f"param[{i}]", st.p[i].double().cpu().numpy(), want_p[i], "f32")
    assert float(st.norm.item()) == pytest.approx(total, rel=2e-6)


def test_argument_checks():
    import torch

    from paper_2609_10632_b200 import binding as nb

    dev = torch.device("cuda", 0)
    t = torch.zeros(64, dtype=torch.float32, device=dev)
    with pytest.raises(nb.NbError) as e:
        nb.SgdPlan([(t, t, t, None, 3)])
    assert e.value.status == nb.NB_ERR_INVALID_ARG
    with pytest.raises(nb.NbError) as e:
        nb.SgdPlan([(t[1:], t, t, None, 0, 8)])
    assert e.value.status == nb.NB_ERR_ALIGNMENT
    plan = nb.SgdPlan([(t, t.clone(), t.clone(), None, 0)])
    ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device=dev)
    with pytest.raises(nb.NbError) as e:
        plan.upload(ws[:256])
    assert e.value.status == nb.NB_ERR_WORKSPACE


def test_loss_scaled_steps_skip_on_overflow_and_follow_the_scaler_dynamics():
    """Gradients arrive multiplied by the loss scale; steps 1 and 4 carry an inf / a NaN and must be skipped (parameters,
    momentum and bf16 copies untouched, scale halved down to the floor); after two good steps in a row the scale doubles.
    Parameters against the oracle at the fp32 bar, scaler state exactly."""
    import struct

    import torch

    sizes, groups = [5000, 64, 4097], [0, 1, 2]
    st = State(sizes, groups, cfg_id=35)
    dev = st.p[0].device
    state = torch.zeros(4, dtype=torch.int32, device=dev)
    state[0] = struct.unpack("i", struct.pack("f", 1024.0))[0]
    scale, tracker, first = 1024.0, 0, True
    read = lambda: (struct.unpack("f", struct.pack("i", int(state[0].item())))[0], int(state[1].item()), int(state[2].item()))
    for k in range(7):
        _, grads = wl.make_optimizer_inputs(sizes, 35, k, 0.3)
        grads = [(g * np.float32(scale)).astype(np.float32) for g in grads]
        if k == 1:
            grads[0][123] = np.inf
        if k == 4:
            grads[2][4096] = np.nan
        for d, h in zip(st.g, grads):
            d.copy_(torch.from_numpy(h))
        before = [p.clone() for p in st.p], [m.clone() for m in st.m], [None if l is None else l.clone() for l in st.lp]
        st.plan.step_scaled(st.ws, state, LR, WD, MOM, 1.0, first_step=first, growth_interval=2, floor_scale=300.0, total_norm=st.norm)
        torch.cuda.synchronize()
        st.h_params, st.h_bufs, total, scale, tracker, skipped = opt.scaled_clip_sgd_step(st.h_params, grads, st.h_bufs, groups, LR, WD, MOM, 1.0, first, scale,
                                                                                          tracker, 2.0, 0.5, 2, floor=300.0)
        assert read() == (scale, tracker, int(skipped)), (k, read(), scale, tracker, skipped)
        if skipped:
            assert k in (1, 4)
            for i in range(len(sizes)):
                assert torch.equal(st.p[i], before[0][i]) and (first or torch.equal(st.m[i], before[1][i]))
                assert st.lp[i] is None or torch.equal(st.lp[i], before[2][i])
            assert not np.isfinite(float(st.norm.item()))
        else:
            first = False
            assert float(st.norm.item()) == pytest.approx(total, rel=2e-6)
            for i in range(len(sizes)):
                parity.check(f"param[{i}]", st.p[i].double().cpu().numpy(), st.h_params[i], "f32")
                parity.check(f"momentum[{i}]", st.m[i].double().cpu().numpy(), st.h_bufs[i], "f32")
    assert scale == 1024.0  # 1024 -> 512 (skip) -> 1024 (two good steps) -> 512 (skip) -> 1024 (two good steps)


def test_fp16_working_copy():
    import torch

    st = State([5000, 4097], [0, 0], cfg_id=36)
    st.lp = [torch.empty(n, dtype=torch.float16, device=st.p[0].device) for n in st.sizes]
    st.plan = st.nb.SgdPlan(zip(st.g, st.p, st.m, st.lp, st.groups))
    st.plan.upload(st.ws)
    _, grads = wl.make_optimizer_inputs(st.sizes, 36, 0, 0.1)
    for d, h in zip(st.g, grads):
        d.copy_(torch.from_numpy(h))
    st.plan.step(st.ws, LR, WD, MOM, MAX_NORM, first_step=True)
    torch.cuda.synchronize()
    for p, lp in zip(st.p, st.lp):
        assert torch.equal(lp, p.to(torch.float16))
