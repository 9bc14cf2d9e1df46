"""Run a dataflow description of chained Conv-BN-SiLU blocks and glue (workloads.detector_graph: the paper's detector,
Sec. 6, from the image to the raw head outputs) on the GPU, forward and backward.

Only wiring happens here: every arithmetic step is a C-ABI call (block calls of nb_cbs.h, glue calls of nb_glue.h);
torch allocates the buffers, zeroes gradient accumulators where needed and owns the streams.

Every named tensor is an NHWC bf16 tensor, dense or -- with views=True -- a CHANNEL SLICE of a wider buffer (a torch
view: data_ptr() is the slice's first channel, stride(-2) its row pitch), which the block calls accept through
nb_cbs_plan_set_pitches and the glue calls through their pitch arguments:
  * a "slice" output is a view of its input (no copy) when all its consumers take pitched operands;
  * a tensor that feeds a concatenation is PLACED inside the concatenation buffer when its producer can write there (a
    block or an add), every other consumer takes pitched operands and runs before the block that consumes the
    concatenation; consecutive slices that make up a whole tensor place that tensor.  Placed inputs need no copy.
Gradients mirror this: the gradient of a placed tensor (or of a slice view) is the same channel range of the gradient of
the buffer it lives in, so the concatenation's / slice's backward step is free and the other consumers ADD their share
there.  A dense tensor whose only consumer is a block takes that block's dx buffer as its gradient; any other tensor
owns a gradient buffer in which the first contribution to a channel range overwrites and later ones add (decided once,
from the order of the backward pass; zeroed beforehand only if the overwriting contributions leave a gap).
"""
from __future__ import annotations

import torch

from . import binding as nb
from .block import CbsBlock

_PITCH_IN = ("slice", "add", "concat", "upsample", "maxpool")  # glue ops that read pitched operands (blocks do when their plan says so)


class GraphRunner:
    def __init__(self, ops, layers, outputs, eps=1e-3, device=0, plain_layers=None, views=True, direct_dx=True, fuse_residual=True,
                 fuse_shortcut_grad=True):
        """plain_layers: shapes of the plain convolutions (bias, no BN, no activation) that "plain" ops refer to; their
        parameters and gradients live in self.plain[k] (dict with plan, w, bias, dw, dbias, dx, ws).
        views=False: every tensor dense, split / concat by copies (the reference behaviour of the views).
        direct_dx=False: every block writes its data gradient to a buffer of its own and a glue launch adds it to the
        input's gradient (the reference behaviour of nb_cbs_plan_set_dx_target).
        fuse_residual=False: every residual add is a glue launch of its own (the reference behaviour of
        nb_cbs_plan_set_fwd_residual, up to one rounding: the fused add rounds the sum once, the separate one rounds the
        block's output first).
        fuse_shortcut_grad=False: the shortcut's share of a fused residual add's gradient is a glue launch of its own (the
        reference behaviour of nb_cbs_plan_set_bwd_residual)."""
        self.ops, self.layers, self.outputs = ops, layers, list(outputs)
        self.dev = torch.device("cuda", device)
        self.plain, self.idx = [], {}
        self.glue_fwd = self.glue_bwd = 0
        new = lambda shp, dtype=torch.bfloat16: torch.empty(shp, dtype=dtype, device=self.dev)
        prod = {o["out"]: (i, o) for i, o in enumerate(ops)}
        cons = {}
        for i, o in enumerate(ops):
            for pos, name in enumerate(o["ins"]):
                cons.setdefault(name, []).append((i, o, pos))
        # ---- residual adds "out = shortcut + v" whose v is a block's output with no other consumer: that block performs the
        # add itself (its normalise + SiLU pass adds the shortcut), v and out are one tensor, and so are their gradients
        self.fused_v = {}  # name of v -> the add op
        if fuse_residual:
            for o in ops:
                if o["op"] == "add":
                    v = o["ins"][1]
                    if v in prod and prod[v][1]["op"] == "cbs" and len(cons[v]) == 1 and v not in self.outputs and o["ins"][0] != v:
                        self.fused_v[v] = o
        self.fused_adds = {id(o) for o in self.fused_v.values()}
        # ---- shapes, blocks, plain convolutions
        s0 = layers[0]
        shape = self.shape = {"img": (s0.n, s0.h, s0.w, s0.c_in)}
        self.blocks = [None] * len(layers)
        takes_pitch = {}
        for o in ops:
            ins = [shape[i] for i in o["ins"]]
            kind = o["op"]
            if kind == "cbs":
                s = layers[o["layer"]]
                assert ins[0] == (s.n, s.h, s.w, s.c_in), (o["out"], ins[0])
                blk = self.blocks[o["layer"]] = CbsBlock(s, eps=eps, device=device)
                try:  # can this block read its input as a channel slice? (needs the tensor-core forward and weight gradient)
                    blk.plan.set_pitches(ld_x=s.c_in + 8)
                    takes_pitch[o["layer"]] = True
                except nb.NbError:
                    takes_pitch[o["layer"]] = False
                blk.plan.set_pitches()
                shape[o["out"]] = (s.n, s.ho, s.wo, s.c_out)
            elif kind == "plain":
                s = plain_layers[o["layer"]]
                assert o["layer"] == len(self.plain) and ins[0] == (s.n, s.h, s.w, s.c_in), o["out"]
                plan = nb.Plan.for_shape(s, eps=eps, device=device)
                self.plain.append({"plan": plan, "shape": s, "w": new((s.c_out, s.k, s.k, s.c_in)), "bias": new((s.c_out,), torch.float32),
                                   "dw": new((s.c_out, s.k, s.k, s.c_in), torch.float32), "dbias": new((s.c_out,), torch.float32),
                                   "dx": new((s.n, s.h, s.w, s.c_in)), "ws": new((max(plan.infer_bytes, plan.bwd_bytes, 256),), torch.uint8)})
                shape[o["out"]] = (s.n, s.ho, s.wo, s.c_out)
            else:
                n, h, w, c = ins[0]
                shape[o["out"]] = {"slice": lambda: (n, h, w, o["c1"] - o["c0"]), "add": lambda: ins[0], "maxpool": lambda: ins[0],
                                   "concat": lambda: (n, h, w, sum(i[3] for i in ins)), "upsample": lambda: (n, 2 * h, 2 * w, c)}[kind]()
        reads_pitched = lambda o: o["op"] in _PITCH_IN or (o["op"] == "cbs" and takes_pitch[o["layer"]])
        # ---- views: which slices are views, which tensors live inside a concatenation buffer
        slice_view, placed = set(), {}
        if views:
            for o in ops:
                if o["op"] == "slice" and all(reads_pitched(c) for _, c, _ in cons.get(o["out"], [])):
                    slice_view.add(o["out"])
            for ci, o in enumerate(ops):
                if o["op"] != "concat" or len(cons.get(o["out"], [])) != 1 or cons[o["out"]][0][1]["op"] != "cbs":
                    continue
                bi = cons[o["out"]][0][0]  # the block that consumes the concatenation (its dx is the concatenation's gradient)

                def others_ok(name, skip):  # every consumer except `skip` reads pitched operands and runs before that block
                    return all((c is skip) or (reads_pitched(c) and i < bi) for i, c, _ in cons.get(name, []))

                off, k, ins = 0, 0, o["ins"]
                while k < len(ins):
                    t = ins[k]
                    _, po = prod.get(t, (None, {"op": "input"}))
                    if po["op"] in ("cbs", "add", "upsample", "maxpool") and t not in placed and t not in self.outputs and others_ok(t, o):
                        placed[t] = (o["out"], off)
                    elif po["op"] == "slice" and t in slice_view and po["c0"] == 0:
                        src = po["ins"][0]  # consecutive slices of one tensor that together are that tensor: place the tensor
                        run, width = [], 0
                        while k + len(run) < len(ins) and width < shape[src][3]:
                            q = ins[k + len(run)]
                            qo = prod[q][1]
                            if qo["op"] != "slice" or qo["ins"][0] != src or qo["c0"] != width or q not in slice_view:
                                break
                            run.append(q)
                            width = qo["c1"]
                        spo = prod.get(src, (None, {"op": "input"}))[1]
                        if (width == shape[src][3] and spo["op"] in ("cbs", "add") and src not in placed and src not in self.outputs
                                and all(c["op"] == "slice" and c["out"] in run for _, c, _ in cons[src]) and all(others_ok(q, o) for q in run)):
                            placed[src] = (o["out"], off)
                            off += width
                            k += len(run)
                            continue
                    off += shape[t][3]
                    k += 1
        self.placed, self.slice_view = placed, slice_view
        # ---- forward tensors
        buf = self.buf = {"img": new(shape["img"])}
        storage = {}

        def cat_storage(name):
            if name not in storage:
                storage[name] = new(shape[name])
            return storage[name]

        for o in ops:
            out, kind, c = o["out"], o["op"], shape[o["out"]][3]
            if out in self.fused_v:
                continue  # lives in the add's output tensor (set when that op is reached)
            if out in placed:
                cat, off = placed[out]
                buf[out] = cat_storage(cat)[..., off:off + c]
            elif kind == "slice" and out in slice_view:
                buf[out] = buf[o["ins"][0]][..., o["c0"]:o["c1"]]
            elif kind == "concat":
                buf[out] = cat_storage(out)
            elif kind == "cbs":
                buf[out] = self.blocks[o["layer"]].a
            else:
                buf[out] = new(shape[out])
            if kind == "maxpool":
                self.idx[out] = new(shape[out], torch.uint8)
            if id(o) in self.fused_adds:
                buf[o["ins"][1]] = buf[out]
        # ---- gradients
        grad = self.grad = {}
        self.owned = []

        def grad_of(name):
            if name in grad:
                return grad[name]
            c = shape[name][3]
            po = prod.get(name, (None, {"op": "input"}))[1]
            cs = cons.get(name, [])
            if name in self.fused_v:
                g = grad_of(self.fused_v[name]["out"])
            elif name in placed:
                cat, off = placed[name]
                g = grad_of(cat)[..., off:off + c]
            elif po["op"] == "slice" and name in slice_view:
                g = grad_of(po["ins"][0])[..., po["c0"]:po["c1"]]
            elif len(cs) == 1 and cs[0][1]["op"] == "plain":
                g = self.plain[cs[0][1]["layer"]]["dx"]
            elif len(cs) == 1 and cs[0][1]["op"] == "cbs":
                g = self.blocks[cs[0][1]["layer"]].dx
            else:
                g = torch.zeros(shape[name], dtype=torch.bfloat16, device=self.dev)
                if name not in self.outputs:
                    self.owned.append(name)
            grad[name] = g
            return g

        for name in buf:
            grad_of(name)
        # ---- wire the blocks: input, output and upstream gradient as (possibly pitched) views
        for o in ops:
            if o["op"] != "cbs":
                continue
            blk, s = self.blocks[o["layer"]], layers[o["layer"]]
            blk.x, blk.a, blk.g = buf[o["ins"][0]], buf[o["out"]], grad[o["out"]]
            blk.plan.set_pitches(ld_x=blk.x.stride(-2), ld_a=blk.a.stride(-2), ld_g=blk.g.stride(-2))
            if o["out"] in self.fused_v:
                blk.res = buf[self.fused_v[o["out"]]["ins"][0]]
                blk.plan.set_fwd_residual(blk.res, blk.res.stride(-2))
        # ---- which contributions overwrite and which add: walk the backward order once over the OWNED buffers
        def root(name):  # (owned tensor whose buffer holds this gradient, channel offset in it) or (None, 0)
            po = prod.get(name, (None, {"op": "input"}))[1]
            if name in placed:
                r, off = root(placed[name][0])
                return r, off + placed[name][1]
            if po["op"] == "slice" and name in slice_view:
                r, off = root(po["ins"][0])
                return r, off + po["c0"]
            return (name, 0) if name in self.owned else (None, 0)

        covered = {name: [] for name in self.owned}
        self.acc, pending = {}, {}
        for oi in reversed(range(len(ops))):
            o = ops[oi]
            for pos, src in enumerate(o["ins"]):
                if self._implicit(o, pos):
                    continue
                r, off = root(src)
                if r is None:
                    self.acc[(oi, pos)] = True  # lands in a buffer that a block's backward wrote whole (a block's dx): add
                    continue
                lo = off + (o["c0"] if o["op"] == "slice" else 0)
                hi = lo + (o["c1"] - o["c0"] if o["op"] == "slice" else shape[src][3])
                inside = any(a <= lo and hi <= b for a, b in covered[r])
                disjoint = all(hi <= a or b <= lo for a, b in covered[r])
                self.acc[(oi, pos)] = not disjoint
                pending.setdefault(r, []).append((oi, pos))
                if disjoint:
                    covered[r].append((lo, hi))
                elif not inside:
                    covered[r] = [(0, 0)]  # partial overlap: zero the buffer and add everything
        self.zeroed = []
        for name, iv in covered.items():
            if (0, 0) in iv or sum(b - a for a, b in iv) != shape[name][3]:
                self.zeroed.append(name)
                for key in pending.get(name, []):
                    self.acc[key] = True
        # ---- a block whose input's gradient lives in a buffer other than its own dx writes (or adds) there itself: its data
        # gradient kernel stores through TMA into the channel slice, as a reduction when other consumers contributed before
        self.direct_dx = set()
        if direct_dx:
            for oi, o in enumerate(ops):
                if o["op"] != "cbs":
                    continue
                blk, target = self.blocks[o["layer"]], grad[o["ins"][0]]
                if target is blk.dx:
                    continue
                try:
                    blk.plan.set_dx_target(ld_dx=target.stride(-2), accumulate=self.acc[(oi, 0)])
                except nb.NbError:
                    continue  # (stride-2 layers and layers off the tensor-core path keep the glue launch)
                blk.dx = target
                self.direct_dx.add(oi)
        # ---- the shortcut's share of a fused residual add's gradient: the block that performs the add also hands its
        # incoming gradient (the sum's gradient) to the shortcut's gradient buffer, inside its dy pass
        self.shortcut_by_block = {}  # index of the add op -> the block that does its backward
        if fuse_shortcut_grad:
            for oi, o in enumerate(ops):
                if o["op"] != "add" or id(o) not in self.fused_adds:
                    continue
                vi, vo = prod[o["ins"][1]]
                if any(vi < i < oi for i, _, _ in cons[o["ins"][0]]):
                    continue  # another contribution to the same gradient would change places with this one
                blk = self.blocks[vo["layer"]]
                gres = grad[o["ins"][0]]
                try:
                    blk.plan.set_bwd_residual(gres, gres.stride(-2), accumulate=self.acc[(oi, 0)])
                except nb.NbError:
                    continue
                blk.gres = gres
                self.shortcut_by_block[oi] = blk

    # ------------------------------------------------------------------ helpers
    def _implicit(self, o, pos):
        """True when op o's backward contribution to its input `pos` needs no work: a slice view, a placed concat input."""
        src = o["ins"][pos]
        if o["op"] == "add" and id(o) in self.fused_adds:
            return pos == 1  # the block's output IS the sum: its gradient is the sum's gradient
        if o["op"] == "slice":
            return o["out"] in self.slice_view
        if o["op"] == "concat":
            off = sum(self.shape[t][3] for t in o["ins"][:pos])
            return self._in_place(self.buf[src], self.buf[o["out"]], off)
        return False

    @staticmethod
    def _in_place(t, cat, off):
        return t.untyped_storage().data_ptr() == cat.untyped_storage().data_ptr() and t.data_ptr() == cat.data_ptr() + off * cat.element_size()

    def _rows(self, name):
        n, h, w, _ = self.shape[name]
        return n * h * w

    def _sadd(self, out, a, rows, channels, b=None, accumulate=False, stream=None):
        nb.nb_slice_add(nb.NB_DTYPE_BF16, rows, channels, out, out.stride(-2), a, a.stride(-2), b, b.stride(-2) if b is not None else 0, accumulate, stream)

    # ------------------------------------------------------------------ passes
    def forward(self, stream=None):
        B, n_glue = self.buf, 0
        for o in self.ops:
            kind, out, ins = o["op"], o["out"], o["ins"]
            rows, c_out = self._rows(out), self.shape[out][3]
            if kind == "cbs":
                self.blocks[o["layer"]].forward(stream)
            elif kind == "plain":
                pl = self.plain[o["layer"]]
                nb.nb_conv_bias_act(pl["plan"], B[ins[0]], pl["w"], pl["bias"], 0, B[out], pl["ws"], stream)
            elif kind == "slice":
                if out not in self.slice_view:
                    self._sadd(B[out], B[ins[0]][..., o["c0"]:o["c1"]], rows, c_out, stream=stream)
                    n_glue += 1
            elif kind == "add":
                if id(o) not in self.fused_adds:
                    self._sadd(B[out], B[ins[0]], rows, c_out, b=B[ins[1]], stream=stream)
                    n_glue += 1
            elif kind == "concat":
                c0 = 0
                for name in ins:
                    c = self.shape[name][3]
                    if not self._in_place(B[name], B[out], c0):
                        self._sadd(B[out][..., c0:c0 + c], B[name], rows, c, stream=stream)
                        n_glue += 1
                    c0 += c
            elif kind == "maxpool":
                n, h, w, c = self.shape[out]
                nb.nb_maxpool5_fwd(nb.NB_DTYPE_BF16, n, h, w, c, B[ins[0]], B[out], self.idx[out], stream, ld_x=B[ins[0]].stride(-2), ld_y=B[out].stride(-2))
                n_glue += 1
            elif kind == "upsample":
                n, h, w, c = self.shape[ins[0]]
                nb.nb_upsample2(nb.NB_DTYPE_BF16, n, h, w, c, B[ins[0]], B[out], ld_small=B[ins[0]].stride(-2), ld_large=B[out].stride(-2), stream=stream)
                n_glue += 1
        self.glue_fwd = n_glue

    def backward(self, stream=None, wgrad_stream=None, wgrad_workspace=None):
        """Expects the gradients of the output tensors in self.grad[name]; leaves dL/d img in self.grad['img'] and every
        block's dw, dgamma, dbeta in the block.  With wgrad_stream (and a workspace for it) every weight gradient is queued
        on that stream behind an event that follows the block's data-gradient call (it only reads the block's input
        activations and dy, which nothing overwrites during the backward pass); the caller joins the streams."""
        G, n_glue = self.grad, 0
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
                    self._sadd(G[src], blk.dx, self._rows(src), self.shape[src][3], accumulate=self.acc[(oi, 0)], stream=stream)
                    n_glue += 1
            elif kind == "plain":
                pl = self.plain[o["layer"]]
                nb.nb_conv_bias_bwd(pl["plan"], self.buf[ins[0]], pl["w"], G[out], pl["dx"], pl["dw"], pl["dbias"], pl["ws"], stream)
                assert G[ins[0]] is pl["dx"]  # a plain convolution is the only consumer of its input in this dataflow
            elif kind == "slice":
                if out not in self.slice_view:
                    self._sadd(G[ins[0]][..., o["c0"]:o["c1"]], G[out], self._rows(out), c_out, accumulate=self.acc[(oi, 0)], stream=stream)
                    n_glue += 1
            elif kind == "add":
                for pos, src in enumerate(ins):
                    if not self._implicit(o, pos) and not (pos == 0 and oi in self.shortcut_by_block):
                        self._sadd(G[src], G[out], self._rows(out), c_out, accumulate=self.acc[(oi, pos)], stream=stream)
                        n_glue += 1
            elif kind == "concat":
                c0 = 0
                for pos, src in enumerate(ins):
                    c = self.shape[src][3]
                    if not self._implicit(o, pos):
                        self._sadd(G[src], G[out][..., c0:c0 + c], self._rows(out), c, accumulate=self.acc[(oi, pos)], stream=stream)
                        n_glue += 1
                    c0 += c
            elif kind == "maxpool":
                n, h, w, c = self.shape[out]
                nb.nb_maxpool5_bwd(nb.NB_DTYPE_BF16, n, h, w, c, G[out], self.idx[out], G[ins[0]], self.acc[(oi, 0)], stream, ld_g=G[out].stride(-2),
                                   ld_dx=G[ins[0]].stride(-2))
                n_glue += 1
            elif kind == "upsample":
                n, h, w, c = self.shape[ins[0]]
                nb.nb_upsample2(nb.NB_DTYPE_BF16, n, h, w, c, G[out], G[ins[0]], backward=True, accumulate=self.acc[(oi, 0)], ld_small=G[ins[0]].stride(-2),
                                ld_large=G[out].stride(-2), stream=stream)
                n_glue += 1
        self.glue_bwd = n_glue

    def fill_parameters(self, seed=0):
        """Random filters (Kaiming-uniform bound), gamma = 1, beta = 0 for every block (timing runs)."""
        gen = torch.Generator(device=self.dev)
        for i, b in enumerate(self.blocks):
            gen.manual_seed(seed + i)
            s = b.shape
            bound = 1.0 / float((s.c_in * s.k * s.k) ** 0.5)
            b.w.copy_((torch.rand(b.w.shape, generator=gen, device=self.dev) * 2 - 1) * bound)
            b.gamma.fill_(1.0)
            b.beta.zero_()

    def poll(self):
        for b in self.blocks:
            b.poll()

    def glue_launches(self):
        """(forward, backward) glue launches of the last passes."""
        return self.glue_fwd, self.glue_bwd
