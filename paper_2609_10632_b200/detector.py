"""Run a dataflow description of chained Conv-BN-SiLU blocks and glue (workloads.detector_graph: the paper's detector,
Sec. 6, up to the last block of every head branch) on the GPU, forward and backward.

Only wiring happens here: every arithmetic step is a C-ABI call (block calls of nb_cbs.h, glue calls of nb_glue.h);
torch allocates the buffers, zeroes gradient accumulators and owns the stream.

Every named tensor is a dense NHWC bf16 buffer.  A block reads its input tensor's buffer directly and writes its
activations into its output tensor's buffer.  Gradients: a tensor whose only consumer is a block takes that block's dx
buffer as its gradient (no copy); every other tensor owns a gradient buffer to which each consumer contributes its share
(several consumers: the sum of their gradients).  The first contribution to a channel range OVERWRITES it and later ones
add to it (decided once, from the order of the backward pass); a buffer is zeroed beforehand only if the overwriting
contributions do not cover all of its channels.
"""
from __future__ import annotations

import torch

from . import binding as nb
from .block import CbsBlock


class GraphRunner:
    def __init__(self, ops, layers, outputs, eps=1e-3, device=0, plain_layers=None):
        """plain_layers: shapes of the plain convolutions (bias, no BN, no activation) that "plain" ops refer to; their
        parameters and gradients live in self.plain[k] (dict with plan, w, bias, dw, dbias, dx, ws)."""
        self.ops, self.layers, self.outputs = ops, layers, list(outputs)
        self.plain = []
        self.dev = torch.device("cuda", device)
        s0 = layers[0]
        self.shape = {"img": (s0.n, s0.h, s0.w, s0.c_in)}
        self.buf = {"img": torch.empty(self.shape["img"], dtype=torch.bfloat16, device=self.dev)}
        self.blocks = [None] * len(layers)
        self.idx = {}
        consumers = {}
        for o in ops:
            for name in o["ins"]:
                consumers.setdefault(name, []).append(o)
        # ---- forward buffers
        for o in ops:
            ins = [self.shape[i] for i in o["ins"]]
            kind = o["op"]
            if kind == "cbs":
                s = layers[o["layer"]]
                assert ins[0] == (s.n, s.h, s.w, s.c_in), (o["out"], ins[0])
                blk = CbsBlock(s, eps=eps, device=device)
                blk.x = self.buf[o["ins"][0]]
                self.blocks[o["layer"]] = blk
                shp, buf = (s.n, s.ho, s.wo, s.c_out), blk.a
            elif kind == "plain":
                s = plain_layers[o["layer"]]
                assert o["layer"] == len(self.plain) and ins[0] == (s.n, s.h, s.w, s.c_in), o["out"]
                plan = nb.Plan.for_shape(s, eps=eps, device=device)
                e = lambda *sz, dtype: torch.empty(*sz, dtype=dtype, device=self.dev)
                shp = (s.n, s.ho, s.wo, s.c_out)
                buf = e(shp, dtype=torch.bfloat16)
                self.plain.append({"plan": plan, "shape": s, "w": e(s.c_out, s.k, s.k, s.c_in, dtype=torch.bfloat16), "bias": e(s.c_out, dtype=torch.float32),
                                   "dw": e(s.c_out, s.k, s.k, s.c_in, dtype=torch.float32), "dbias": e(s.c_out, dtype=torch.float32),
                                   "dx": e(s.n, s.h, s.w, s.c_in, dtype=torch.bfloat16),
                                   "ws": e(max(plan.infer_bytes, plan.bwd_bytes, 256), dtype=torch.uint8)})
            else:
                n, h, w, c = ins[0]
                if kind == "slice":
                    shp = (n, h, w, o["c1"] - o["c0"])
                elif kind == "add" or kind == "maxpool":
                    shp = ins[0]
                elif kind == "concat":
                    shp = (n, h, w, sum(i[3] for i in ins))
                elif kind == "upsample":
                    shp = (n, 2 * h, 2 * w, c)
                else:
                    raise ValueError(kind)
                buf = torch.empty(shp, dtype=torch.bfloat16, device=self.dev)
                if kind == "maxpool":
                    self.idx[o["out"]] = torch.empty(shp, dtype=torch.uint8, device=self.dev)
            self.shape[o["out"]], self.buf[o["out"]] = shp, buf
        # ---- gradient buffers
        self.grad, self.owned = {}, []
        by_out = {o["out"]: o for o in ops}
        for name in list(self.buf):
            cons = consumers.get(name, [])
            if len(cons) == 1 and cons[0]["op"] == "plain":
                self.grad[name] = self.plain[cons[0]["layer"]]["dx"]
            elif len(cons) == 1 and cons[0]["op"] == "cbs":
                self.grad[name] = self.blocks[cons[0]["layer"]].dx
            else:
                self.grad[name] = torch.zeros(self.shape[name], dtype=torch.bfloat16, device=self.dev)
                if name not in self.outputs:
                    self.owned.append(name)
        for o in ops:
            if o["op"] == "cbs":
                self.blocks[o["layer"]].g = self.grad[o["out"]]
        self.aliased = {name for name in self.buf if name not in self.owned and name not in self.outputs}
        # ---- which contributions overwrite and which add: walk the backward order once
        covered = {name: [] for name in self.owned}  # channel intervals already written
        self.acc = {}                                  # (op index, input position) -> accumulate?
        for oi in reversed(range(len(ops))):
            o = ops[oi]
            for pos, src in enumerate(o["ins"]):
                if src not in covered:
                    continue  # aliased to a block's dx, or the block writes there directly
                c = self.shape[src][3]
                lo, hi = (o["c0"], o["c1"]) if o["op"] == "slice" else (0, c)
                inside = any(a <= lo and hi <= b for a, b in covered[src])
                disjoint = all(hi <= a or b <= lo for a, b in covered[src])
                if inside:
                    self.acc[(oi, pos)] = True
                elif disjoint:
                    self.acc[(oi, pos)] = False
                    covered[src].append((lo, hi))
                else:  # partial overlap: give up on this tensor, zero it and add everything
                    covered[src] = [(0, 0)]
                    self.acc[(oi, pos)] = True
        self.zeroed = []
        for name, iv in covered.items():
            full = sorted(iv) and sum(b - a for a, b in iv) == self.shape[name][3] and (0, 0) not in iv
            if not full:
                self.zeroed.append(name)
                for key in [k for k in self.acc if ops[k[0]]["ins"][k[1]] == name]:
                    self.acc[key] = True

    # ------------------------------------------------------------------ helpers
    def _rows(self, name):
        n, h, w, _ = self.shape[name]
        return n * h * w

    @staticmethod
    def _at(t, channel):
        return t.data_ptr() + channel * t.element_size()

    def _copy(self, out, ld_out, a, ld_a, rows, channels, b=None, ld_b=0, accumulate=False, stream=None):
        nb.nb_slice_add(nb.NB_DTYPE_BF16, rows, channels, out, ld_out, a, ld_a, b, ld_b, accumulate, stream)

    # ------------------------------------------------------------------ passes
    def forward(self, stream=None):
        B = self.buf
        for o in self.ops:
            kind, out, ins = o["op"], o["out"], o["ins"]
            rows = self._rows(out)
            c_out = self.shape[out][3]
            if kind == "cbs":
                self.blocks[o["layer"]].forward(stream)
            elif kind == "plain":
                pl = self.plain[o["layer"]]
                nb.nb_conv_bias_act(pl["plan"], B[ins[0]], pl["w"], pl["bias"], 0, B[out], pl["ws"], stream)
            elif kind == "slice":
                self._copy(B[out], c_out, self._at(B[ins[0]], o["c0"]), self.shape[ins[0]][3], rows, c_out, stream=stream)
            elif kind == "add":
                self._copy(B[out], c_out, B[ins[0]], c_out, rows, c_out, b=B[ins[1]], ld_b=c_out, stream=stream)
            elif kind == "concat":
                c0 = 0
                for name in ins:
                    c = self.shape[name][3]
                    self._copy(self._at(B[out], c0), c_out, B[name], c, rows, c, stream=stream)
                    c0 += c
            elif kind == "maxpool":
                n, h, w, c = self.shape[out]
                nb.nb_maxpool5_fwd(nb.NB_DTYPE_BF16, n, h, w, c, B[ins[0]], B[out], self.idx[out], stream)
            elif kind == "upsample":
                n, h, w, c = self.shape[ins[0]]
                nb.nb_upsample2(nb.NB_DTYPE_BF16, n, h, w, c, B[ins[0]], B[out], stream=stream)

    def backward(self, stream=None, wgrad_stream=None, wgrad_workspace=None):
        """Expects the gradients of the output tensors in self.grad[name]; leaves dL/d img in self.grad['img'] and every
        block's dw, dgamma, dbeta in the block.  With wgrad_stream (and a workspace for it) every weight gradient is queued
        on that stream behind an event that follows the block's data-gradient call (it only reads the block's input
        activations and dy, which nothing overwrites during the backward pass); the caller joins the streams."""
        G = self.grad
        for name in self.zeroed:
            G[name].zero_()
        for oi in reversed(range(len(self.ops))):
            o = self.ops[oi]
            kind, out, ins = o["op"], o["out"], o["ins"]
            c_out = self.shape[out][3]
            if kind == "cbs":
                blk = self.blocks[o["layer"]]
                blk.backward_data(stream)
                if wgrad_stream is None:
                    blk.backward_weight(stream)
                else:
                    ev = torch.cuda.Event()
                    ev.record(torch.cuda.current_stream(self.dev) if stream is None else stream)
                    wgrad_stream.wait_event(ev)
                    blk.backward_weight(wgrad_stream, wgrad_workspace)
                src = ins[0]
                if G[src] is not blk.dx:
                    c = self.shape[src][3]
                    self._copy(G[src], c, blk.dx, c, self._rows(src), c, accumulate=self.acc[(oi, 0)], stream=stream)
            elif kind == "plain":
                pl = self.plain[o["layer"]]
                nb.nb_conv_bias_bwd(pl["plan"], self.buf[ins[0]], pl["w"], G[out], pl["dx"], pl["dw"], pl["dbias"], pl["ws"], stream)
                assert G[ins[0]] is pl["dx"]  # a plain convolution is the only consumer of its input in this dataflow
            elif kind == "slice":
                src = ins[0]
                self._copy(self._at(G[src], o["c0"]), self.shape[src][3], G[out], c_out, self._rows(out), c_out, accumulate=self.acc[(oi, 0)], stream=stream)
            elif kind == "add":
                for pos, src in enumerate(ins):
                    self._copy(G[src], c_out, G[out], c_out, self._rows(out), c_out, accumulate=self.acc[(oi, pos)], stream=stream)
            elif kind == "concat":
                c0 = 0
                for pos, src in enumerate(ins):
                    c = self.shape[src][3]
                    self._copy(G[src], c, self._at(G[out], c0), c_out, self._rows(out), c, accumulate=self.acc[(oi, pos)], stream=stream)
                    c0 += c
            elif kind == "maxpool":
                n, h, w, c = self.shape[out]
                nb.nb_maxpool5_bwd(nb.NB_DTYPE_BF16, n, h, w, c, G[out], self.idx[out], G[ins[0]], self.acc[(oi, 0)], stream)
            elif kind == "upsample":
                n, h, w, c = self.shape[ins[0]]
                nb.nb_upsample2(nb.NB_DTYPE_BF16, n, h, w, c, G[out], G[ins[0]], backward=True, accumulate=self.acc[(oi, 0)], stream=stream)

    def poll(self):
        for b in self.blocks:
            b.poll()

    def glue_launches(self):
        glue = [o for o in self.ops if o["op"] not in ("cbs", "plain")]
        fwd = sum(len(o["ins"]) if o["op"] == "concat" else 1 for o in glue)
        bwd = sum(len(o["ins"]) if o["op"] in ("concat", "add") else 1 for o in glue)
        bwd += sum(1 for o in self.ops if o["op"] == "cbs" and self.grad[o["ins"][0]] is not self.blocks[o["layer"]].dx)
        return fwd, bwd
