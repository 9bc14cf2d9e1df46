"""Device-buffer holder for one Conv-BN-SiLU block: allocates torch tensors and calls the C ABI.

No arithmetic happens here; torch is used for ``torch.empty`` / ``copy_`` only.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as nb


class CbsBlock:
    """All tensors of one block on one device plus its plan; forward()/backward() are the three C-ABI calls."""

    def __init__(self, shape, mode=nb.NB_MODE_BF16_TC, eps=1e-3, momentum=0.03, flags=0, device=0, running_stats=False,
                 need_dx=True, workspace=None):
        self.shape = s = shape
        self.mode = mode
        self.dev = torch.device("cuda", device)
        self.plan = nb.Plan.for_shape(s, eps=eps, momentum=momentum, mode=mode, flags=flags, device=device)
        f32 = mode == nb.NB_MODE_F32_REF
        self.act_dtype = torch.float32 if f32 else (torch.float16 if mode == nb.NB_MODE_F16_TC else torch.bfloat16)
        self.y_dtype = torch.float32 if f32 else torch.float16
        e = lambda *sz, dtype: torch.empty(*sz, dtype=dtype, device=self.dev)
        self.x = e(s.n, s.h, s.w, s.c_in, dtype=self.act_dtype)
        self.w = e(s.c_out, s.k, s.k, s.c_in, dtype=self.act_dtype)
        self.gamma = e(s.c_out, dtype=torch.float32)
        self.beta = e(s.c_out, dtype=torch.float32)
        self.g = e(s.n, s.ho, s.wo, s.c_out, dtype=self.act_dtype)
        self.y = e(s.n, s.ho, s.wo, s.c_out, dtype=self.y_dtype)
        self.a = e(s.n, s.ho, s.wo, s.c_out, dtype=self.act_dtype)
        self.dy = e(s.n, s.ho, s.wo, s.c_out, dtype=self.act_dtype)
        self.dx = e(s.n, s.h, s.w, s.c_in, dtype=self.act_dtype) if need_dx else None
        self.dw = e(s.c_out, s.k, s.k, s.c_in, dtype=torch.float32)
        self.mean = e(s.c_out, dtype=torch.float32)
        self.invstd = e(s.c_out, dtype=torch.float32)
        self.dgamma = e(s.c_out, dtype=torch.float32)
        self.dbeta = e(s.c_out, dtype=torch.float32)
        self.running_mean = torch.zeros(s.c_out, dtype=torch.float32, device=self.dev) if running_stats else None
        self.running_var = torch.ones(s.c_out, dtype=torch.float32, device=self.dev) if running_stats else None
        need = max(self.plan.fwd_bytes, self.plan.bwd_bytes)
        if workspace is None:
            workspace = torch.empty(need, dtype=torch.uint8, device=self.dev)
        assert workspace.numel() >= need
        self.ws = workspace

    def upload(self, inp):
        """Copy a workloads.BlockInputs (fp32 numpy) to the device tensors."""
        for name in ("x", "w", "gamma", "beta", "g"):
            dst = getattr(self, name)
            dst.copy_(torch.from_numpy(np.ascontiguousarray(getattr(inp, name))).to(dst.dtype))

    def fill_random(self, seed=0):
        """Device-side random fill of the same distributions (for timing runs of large layers)."""
        gen = torch.Generator(device=self.dev)
        gen.manual_seed(seed)
        s = self.shape
        if s.image_input:
            self.x.copy_(torch.rand(self.x.shape, generator=gen, device=self.dev))
        else:
            self.x.copy_(torch.randn(self.x.shape, generator=gen, device=self.dev))
        bound = 1.0 / float(np.sqrt(s.c_in * s.k * s.k))
        self.w.copy_((torch.rand(self.w.shape, generator=gen, device=self.dev) * 2 - 1) * bound)
        self.g.copy_(torch.randn(self.g.shape, generator=gen, device=self.dev))
        self.gamma.fill_(1.0)
        self.beta.zero_()

    def forward(self, stream=None):
        nb.nb_conv_bn_silu_fwd(self.plan, self.x, self.w, self.gamma, self.beta, self.running_mean, self.running_var, self.y,
                               self.mean, self.invstd, self.a, self.ws, stream)

    def backward_data(self, stream=None):
        nb.nb_conv_bn_silu_bwd_data(self.plan, self.g, self.y, self.mean, self.invstd, self.gamma, self.beta, self.w, self.dx,
                                    self.dgamma, self.dbeta, self.dy, self.ws, stream)

    def backward_weight(self, stream=None, workspace=None):
        nb.nb_conv_bn_silu_bwd_weight(self.plan, self.x, self.dy, self.dw, self.ws if workspace is None else workspace, stream)

    def step(self, stream=None, wgrad_stream=None, wgrad_workspace=None):
        """Forward, data gradient, weight gradient.  With `wgrad_stream` (and a workspace of its own) the weight gradient
        is queued on that stream behind an event that follows the data-gradient call, so it overlaps whatever the caller
        queues next on `stream`; the caller joins the two streams."""
        self.forward(stream)
        self.backward_data(stream)
        if wgrad_stream is None:
            self.backward_weight(stream)
            return
        assert wgrad_workspace is not None and wgrad_workspace.numel() >= self.plan.bwd_bytes
        ev = torch.cuda.Event()
        ev.record(torch.cuda.current_stream(self.dev) if stream is None else stream)
        wgrad_stream.wait_event(ev)
        self.backward_weight(wgrad_stream, wgrad_workspace)

    def poll(self):
        return nb.nb_cbs_poll_status(self.plan)

    def download(self):
        """Results as fp64 numpy arrays."""
        torch.cuda.synchronize(self.dev)
        out = {}
        for name in ("y", "a", "dy", "dx", "dw", "mean", "invstd", "dgamma", "dbeta", "running_mean", "running_var"):
            t = getattr(self, name)
            if t is not None:
                out[name] = t.detach().to(torch.float64).cpu().numpy()
        return out
