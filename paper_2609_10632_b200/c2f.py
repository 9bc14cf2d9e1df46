"""A chained C2f unit (Sec. 6 of the paper: the detector's repeated building block) on the GPU: 2 + 2n Conv-BN-SiLU blocks
joined by a channel split, residual additions and a concatenation, forward and backward.

Only wiring happens here: every arithmetic step is a C-ABI call (the block calls of nb_cbs.h and nb_slice_add of
nb_glue.h); torch allocates the buffers.  Layout of the concatenation buffer `cat` [M][(2+n)c]: channels [0, 2c) = output
of cv1, channels [(2+i)c, (3+i)c) = output of bottleneck i.  A bottleneck reads its input as a dense copy of the
previous part (the convolution calls take dense tensors) and writes t + v (or v) back into its slice; in the backward
pass the gradient of the concatenation is cv2's dx, and each bottleneck adds its input gradient (and, with the
shortcut, its output gradient) into the previous part's slice.
"""
from __future__ import annotations

import torch

from . import binding as nb
from . import workloads as wl
from .block import CbsBlock


class C2fChain:
    def __init__(self, batch, h, w, c1, c2, n, shortcut=True, eps=1e-3, device=0):
        assert c2 % 2 == 0
        self.n, self.shortcut, self.c = n, shortcut, c2 // 2
        c = self.c
        self.ctot = (2 + n) * c
        shape = lambda name, ci, co, k: wl.ConvShape(name, batch, h, w, ci, co, k, 1)
        self.cv1 = CbsBlock(shape("cv1", c1, 2 * c, 1), eps=eps, device=device)
        self.m = [(CbsBlock(shape(f"m{i}.cv1", c, c, 3), eps=eps, device=device), CbsBlock(shape(f"m{i}.cv2", c, c, 3), eps=eps, device=device))
                  for i in range(n)]
        self.cv2 = CbsBlock(shape("cv2", self.ctot, c2, 1), eps=eps, device=device)
        self.rows = batch * h * w
        for b1, b2 in self.m:  # the second convolution of a bottleneck reads the first one's activations; gradients flow back the same way
            b2.x = b1.a
            b1.g = b2.dx
        self.cat = self.cv2.x    # [N][H][W][(2+n)c]
        self.dcat = self.cv2.dx  # gradient of the concatenation

    @property
    def blocks(self):
        out = [self.cv1]
        for b1, b2 in self.m:
            out += [b1, b2]
        return out + [self.cv2]

    def _slice(self, t, first_channel):
        return t.data_ptr() + first_channel * t.element_size()

    def _add(self, out, ld_out, a, ld_a, channels, b=None, ld_b=0, accumulate=False, stream=None):
        nb.nb_slice_add(nb.NB_DTYPE_BF16, self.rows, channels, out, ld_out, a, ld_a, b, ld_b, accumulate, stream)

    def forward(self, stream=None):
        c, ct = self.c, self.ctot
        self.cv1.forward(stream)
        self._add(self._slice(self.cat, 0), ct, self.cv1.a, 2 * c, 2 * c, stream=stream)
        for i, (b1, b2) in enumerate(self.m):
            self._add(b1.x, c, self._slice(self.cat, (1 + i) * c), ct, c, stream=stream)  # dense copy of the previous part
            b1.forward(stream)
            b2.forward(stream)
            if self.shortcut:
                self._add(self._slice(self.cat, (2 + i) * c), ct, b2.a, c, c, b=b1.x, ld_b=c, stream=stream)
            else:
                self._add(self._slice(self.cat, (2 + i) * c), ct, b2.a, c, c, stream=stream)
        self.cv2.forward(stream)

    def backward(self, stream=None):
        """Expects cv2.g = dL/d out.  Leaves dL/dx in cv1.dx and every block's dw, dgamma, dbeta in the block."""
        c, ct = self.c, self.ctot
        self.cv2.backward_data(stream)
        self.cv2.backward_weight(stream)
        for i in reversed(range(self.n)):
            b1, b2 = self.m[i]
            self._add(b2.g, c, self._slice(self.dcat, (2 + i) * c), ct, c, stream=stream)  # dense copy of this part's gradient
            b2.backward_data(stream)
            b2.backward_weight(stream)
            b1.backward_data(stream)
            b1.backward_weight(stream)
            if self.shortcut:
                self._add(self._slice(self.dcat, (1 + i) * c), ct, b1.dx, c, c, b=self._slice(self.dcat, (2 + i) * c), ld_b=ct, accumulate=True, stream=stream)
            else:
                self._add(self._slice(self.dcat, (1 + i) * c), ct, b1.dx, c, c, accumulate=True, stream=stream)
        self._add(self.cv1.g, 2 * c, self._slice(self.dcat, 0), ct, 2 * c, stream=stream)
        self.cv1.backward_data(stream)
        self.cv1.backward_weight(stream)

    def poll(self):
        for b in self.blocks:
            b.poll()


class SppfChain:
    """The SPPF unit: 1x1 block, three chained 5x5 max-pools, concatenation of the four parts, 1x1 block; forward and
    backward.  Each pool writes a dense part buffer (the pool kernels take dense tensors); nb_slice_add moves the parts
    into, and the gradients out of, the concatenation buffer."""

    def __init__(self, batch, h, w, c1, c2, eps=1e-3, device=0):
        c = c1 // 2
        self.c, self.dims = c, (batch, h, w, c)
        shape = lambda name, ci, co: wl.ConvShape(name, batch, h, w, ci, co, 1, 1)
        self.cv1 = CbsBlock(shape("cv1", c1, c), eps=eps, device=device)
        self.cv2 = CbsBlock(shape("cv2", 4 * c, c2), eps=eps, device=device)
        self.rows = batch * h * w
        dev = self.cv1.dev
        self.pool = [torch.empty(batch, h, w, c, dtype=torch.bfloat16, device=dev) for _ in range(3)]
        self.idx = [torch.empty(batch, h, w, c, dtype=torch.uint8, device=dev) for _ in range(3)]
        self.dpart = [torch.empty(batch, h, w, c, dtype=torch.bfloat16, device=dev) for _ in range(4)]  # dense gradients of the parts
        self.cat, self.dcat = self.cv2.x, self.cv2.dx

    @property
    def blocks(self):
        return [self.cv1, self.cv2]

    def _slice(self, t, first_channel):
        return t.data_ptr() + first_channel * t.element_size()

    def forward(self, stream=None):
        n, h, w, c = self.dims
        self.cv1.forward(stream)
        src = self.cv1.a
        nb.nb_slice_add(nb.NB_DTYPE_BF16, self.rows, c, self._slice(self.cat, 0), 4 * c, src, c, stream=stream)
        for j in range(3):
            nb.nb_maxpool5_fwd(nb.NB_DTYPE_BF16, n, h, w, c, src, self.pool[j], self.idx[j], stream)
            nb.nb_slice_add(nb.NB_DTYPE_BF16, self.rows, c, self._slice(self.cat, (1 + j) * c), 4 * c, self.pool[j], c, stream=stream)
            src = self.pool[j]
        self.cv2.forward(stream)

    def backward(self, stream=None):
        n, h, w, c = self.dims
        self.cv2.backward_data(stream)
        self.cv2.backward_weight(stream)
        for j in range(4):
            nb.nb_slice_add(nb.NB_DTYPE_BF16, self.rows, c, self.dpart[j], c, self._slice(self.dcat, j * c), 4 * c, stream=stream)
        for j in (3, 2, 1):  # part j = pool(part j-1)
            nb.nb_maxpool5_bwd(nb.NB_DTYPE_BF16, n, h, w, c, self.dpart[j], self.idx[j - 1], self.dpart[j - 1], True, stream)
        self.cv1.g = self.dpart[0]
        self.cv1.backward_data(stream)
        self.cv1.backward_weight(stream)

    def poll(self):
        for b in self.blocks:
            b.poll()
