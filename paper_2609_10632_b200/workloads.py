"""Seeded synthetic workloads: shapes of the detector's Conv-BN-SiLU layers and host-side input generators.

This module holds no arithmetic of the method (no convolution, normalisation or activation): it only
names shapes, draws random numbers and converts between fp32 and bf16 bit patterns.  It is the one
module that both the tests of the CPU oracle and the callers of the CUDA library may import, so both
sides see bit-identical inputs.

Shapes follow the paper's case-study detector (Sec. 6: a YOLOv8m-class network with CSP backbone,
PAN-FPN neck, decoupled head, DFL with reg_max = 16, strides {8, 16, 32}, 80 classes, about 25.9 M
parameters, batch 16 at 640 x 640; Table 1).  The images the paper trains on are not available here:
uniform[0, 1] images and N(0, 1) activations stand in for them.  Convolution weights are drawn
Kaiming-uniform with a = sqrt(5), the initialiser Table 2 (row 3) says the reference uses, i.e.
U(-b, b) with b = 1/sqrt(fan_in).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


# ----------------------------------------------------------------------------- shapes
@dataclass(frozen=True)
class ConvShape:
    """One Conv(k x k, stride, pad k//2) -> BN -> SiLU block on an NHWC batch."""

    name: str
    n: int
    h: int
    w: int
    c_in: int
    c_out: int
    k: int
    stride: int
    image_input: bool = False  # True: x ~ U[0,1] (network input); False: x ~ N(0,1)

    @property
    def pad(self) -> int:
        return self.k // 2

    @property
    def ho(self) -> int:
        return (self.h + 2 * self.pad - self.k) // self.stride + 1

    @property
    def wo(self) -> int:
        return (self.w + 2 * self.pad - self.k) // self.stride + 1

    @property
    def m(self) -> int:
        return self.n * self.ho * self.wo

    @property
    def kdim(self) -> int:
        return self.k * self.k * self.c_in

    @property
    def gemm_flops(self) -> int:
        """Multiply-adds x 2 of ONE of the three GEMMs (fprop, dgrad and wgrad cost the same)."""
        return 2 * self.m * self.kdim * self.c_out

    @property
    def key(self):
        return (self.n, self.h, self.w, self.c_in, self.c_out, self.k, self.stride)

    def with_batch(self, n: int) -> "ConvShape":
        return ConvShape(self.name, n, self.h, self.w, self.c_in, self.c_out, self.k, self.stride, self.image_input)


def detector_layers(batch: int = 16, image: int = 640):
    """The 77 Conv-BN-SiLU layers of the YOLOv8m-class detector, in network order.

    Width multiple 0.75 / depth multiple 0.67 give stage channels 48/96/192/384/576 and C2f repeats
    2/4/4/2.  C2f(c1 -> c2, n): 1x1 c1 -> c2, then n bottlenecks of two 3x3 (c2/2 -> c2/2) on one half,
    then 1x1 (2+n)*c2/2 -> c2.  SPPF: 1x1 c -> c/2, three chained 5x5 max-pools, 1x1 2c -> c.  Head per
    level: box branch 3x3 ch -> 64, 3x3 64 -> 64; class branch 3x3 ch -> 192, 3x3 192 -> 192 (their final
    plain 1x1 convolutions carry a bias and no BN/SiLU and are listed by `detector_plain_head_convs`).
    """
    layers: list[ConvShape] = []

    def conv(name, cin, cout, k, s, hin, image_input=False):
        layers.append(ConvShape(name, batch, hin, hin, cin, cout, k, s, image_input))
        return (hin + 2 * (k // 2) - k) // s + 1

    def c2f(name, c1, c2, n, h):
        c = c2 // 2
        conv(f"{name}.cv1", c1, 2 * c, 1, 1, h)
        for i in range(n):
            conv(f"{name}.m{i}.cv1", c, c, 3, 1, h)
            conv(f"{name}.m{i}.cv2", c, c, 3, 1, h)
        conv(f"{name}.cv2", (2 + n) * c, c2, 1, 1, h)

    h = image
    h = conv("b0.stem", 3, 48, 3, 2, h, image_input=True)
    h = conv("b1.down", 48, 96, 3, 2, h)
    c2f("b2.c2f", 96, 96, 2, h)
    h3 = h = conv("b3.down", 96, 192, 3, 2, h)
    c2f("b4.c2f", 192, 192, 4, h)
    h4 = h = conv("b5.down", 192, 384, 3, 2, h)
    c2f("b6.c2f", 384, 384, 4, h)
    h5 = h = conv("b7.down", 384, 576, 3, 2, h)
    c2f("b8.c2f", 576, 576, 2, h)
    conv("b9.sppf.cv1", 576, 288, 1, 1, h5)
    conv("b9.sppf.cv2", 4 * 288, 576, 1, 1, h5)
    c2f("n12.c2f", 576 + 384, 384, 2, h4)
    c2f("n15.c2f", 384 + 192, 192, 2, h3)
    conv("n16.down", 192, 192, 3, 2, h3)
    c2f("n18.c2f", 192 + 384, 384, 2, h4)
    conv("n19.down", 384, 384, 3, 2, h4)
    c2f("n21.c2f", 384 + 576, 576, 2, h5)
    for lvl, (ch, hh) in enumerate([(192, h3), (384, h4), (576, h5)]):
        conv(f"h22.box{lvl}.0", ch, 64, 3, 1, hh)
        conv(f"h22.box{lvl}.1", 64, 64, 3, 1, hh)
        conv(f"h22.cls{lvl}.0", ch, 192, 3, 1, hh)
        conv(f"h22.cls{lvl}.1", 192, 192, 3, 1, hh)
    return layers


def detector_plain_head_convs():
    """(c_in, c_out) of the six bias-carrying 1x1 output convolutions of the head (no BN, no SiLU)."""
    return [(64, 64), (192, 80)] * 3


def detector_graph(batch: int = 16, image: int = 640, plain_head: bool = False):
    """The detector's dataflow up to the last Conv-BN-SiLU block of every head branch, as a list of primitive operations
    over named tensors (a description only: no arithmetic here, both the GPU runner and the CPU oracle interpret it).

    Returns (ops, layers, outputs): `layers` = detector_layers(batch, image); every op is a dict with "out", "op" and
    "ins": op "cbs" (+ "layer": index into layers), "slice" (+ "c0", "c1": channel range), "add", "concat", "maxpool"
    (5x5, stride 1), "upsample" (nearest 2x); tensor "img" is the input image batch; `outputs` names the six head tensors
    (box and class branch of the three levels), which feed the plain output convolutions and the loss.
    Backbone C2f units have the residual shortcut, neck units do not.

    plain_head=True appends the six plain 1x1 output convolutions (bias, no BN, no activation): op "plain" with "layer" =
    index into a fourth return value, the list of their ConvShapes; `outputs` then names the six raw head outputs
    (64 box-distribution channels and 80 class logits per level).
    """
    layers = detector_layers(batch, image)
    index = {s.name: i for i, s in enumerate(layers)}
    ops = []

    def cbs(name, src):
        ops.append({"out": name, "op": "cbs", "ins": [src], "layer": index[name]})
        return name

    def c2f(name, src, n, shortcut):
        c = layers[index[f"{name}.cv1"]].c_out // 2
        a0 = cbs(f"{name}.cv1", src)
        parts = []
        for j in range(2):
            ops.append({"out": f"{name}.p{j}", "op": "slice", "ins": [a0], "c0": j * c, "c1": (j + 1) * c})
            parts.append(f"{name}.p{j}")
        for i in range(n):
            v = cbs(f"{name}.m{i}.cv2", cbs(f"{name}.m{i}.cv1", parts[-1]))
            if shortcut:
                ops.append({"out": f"{name}.p{2 + i}", "op": "add", "ins": [parts[-1], v]})
                v = f"{name}.p{2 + i}"
            parts.append(v)
        ops.append({"out": f"{name}.cat", "op": "concat", "ins": list(parts)})
        return cbs(f"{name}.cv2", f"{name}.cat")

    def cat(name, srcs):
        ops.append({"out": name, "op": "concat", "ins": list(srcs)})
        return name

    t = cbs("b1.down", cbs("b0.stem", "img"))
    t = cbs("b3.down", c2f("b2.c2f", t, 2, True))
    p3 = c2f("b4.c2f", t, 4, True)
    p4 = c2f("b6.c2f", cbs("b5.down", p3), 4, True)
    t = c2f("b8.c2f", cbs("b7.down", p4), 2, True)
    a0 = cbs("b9.sppf.cv1", t)
    pools = [a0]
    for j in range(3):
        ops.append({"out": f"b9.sppf.pool{j}", "op": "maxpool", "ins": [pools[-1]]})
        pools.append(f"b9.sppf.pool{j}")
    p5 = cbs("b9.sppf.cv2", cat("b9.sppf.cat", pools))
    ops.append({"out": "n10.up", "op": "upsample", "ins": [p5]})
    n12 = c2f("n12.c2f", cat("n11.cat", ["n10.up", p4]), 2, False)
    ops.append({"out": "n13.up", "op": "upsample", "ins": [n12]})
    n15 = c2f("n15.c2f", cat("n14.cat", ["n13.up", p3]), 2, False)
    n18 = c2f("n18.c2f", cat("n17.cat", [cbs("n16.down", n15), n12]), 2, False)
    n21 = c2f("n21.c2f", cat("n20.cat", [cbs("n19.down", n18), p5]), 2, False)
    outputs = []
    for lvl, src in enumerate([n15, n18, n21]):
        outputs.append(cbs(f"h22.box{lvl}.1", cbs(f"h22.box{lvl}.0", src)))
        outputs.append(cbs(f"h22.cls{lvl}.1", cbs(f"h22.cls{lvl}.0", src)))
    if not plain_head:
        return ops, layers, outputs
    plain, raw = [], []
    for j, (src, (cin, cout)) in enumerate(zip(outputs, detector_plain_head_convs())):
        s = layers[index[src]]
        assert s.c_out == cin
        name = src.replace(".1", ".out")
        plain.append(ConvShape(name, batch, s.ho, s.wo, cin, cout, 1, 1))
        ops.append({"out": name, "op": "plain", "ins": [src], "layer": j})
        raw.append(name)
    return ops, layers, raw, plain


def detector_parameter_tensors():
    """[(name, numel, group)] of the detector's trainable tensors in network order: per Conv-BN-SiLU layer the filter
    (group 0: decayed weights), the BN gain (group 1) and the BN shift (group 2: biases); per plain head convolution its
    filter (group 0) and bias (group 2).  243 tensors, about 25.9 M elements (Sec. 3.2 / Sec. 6; pinned in tests)."""
    out = []
    for s in detector_layers():
        out.append((f"{s.name}.w", s.c_out * s.k * s.k * s.c_in, 0))
        out.append((f"{s.name}.gamma", s.c_out, 1))
        out.append((f"{s.name}.beta", s.c_out, 2))
    for i, (cin, cout) in enumerate(detector_plain_head_convs()):
        out.append((f"h22.out{i}.w", cout * cin, 0))
        out.append((f"h22.out{i}.bias", cout, 2))
    return out


def distinct_shapes(layers):
    """[(shape, multiplicity)] in first-appearance order."""
    seen: dict = {}
    for s in layers:
        if s.key in seen:
            seen[s.key][1] += 1
        else:
            seen[s.key] = [s, 1]
    return [(v[0], v[1]) for v in seen.values()]


def config_shapes(cfg: int):
    """Shapes of the benchmark configurations 1-5 (cfg 4 is a pair of layers, cfg 5 the 77 layers)."""
    if cfg == 1:
        return [ConvShape("cfg1", 2, 32, 32, 16, 32, 3, 1)]
    if cfg == 2:
        return [ConvShape("cfg2.stem", 16, 640, 640, 3, 48, 3, 2, True)]
    if cfg == 3:
        return [ConvShape("cfg3.c2f", 16, 160, 160, 96, 96, 3, 1)]
    if cfg == 4:
        return [ConvShape("cfg4a.1x1", 16, 40, 40, 384, 384, 1, 1), ConvShape("cfg4b.down", 16, 80, 80, 192, 384, 3, 2)]
    if cfg == 5:
        return detector_layers(16, 640)
    raise ValueError(f"unknown config {cfg}")


# ----------------------------------------------------------------------------- bf16 <-> fp32 bit patterns
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even), returned as uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """fp32 values that are exactly representable in bf16."""
    return bf16_bits_to_f32(f32_to_bf16_bits(a))


# ----------------------------------------------------------------------------- generators
_ROLES = {"x": 0, "w": 1, "gamma": 2, "beta": 3, "g": 4, "rm": 5, "rv": 6, "bias": 7}


def _rng(cfg_id: int, layer_id: int, role: str) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(cfg_id), int(layer_id) * 8 + _ROLES[role]]))


@dataclass
class BlockInputs:
    """fp32 host arrays for one block.  With bf16=True, x, w and g hold bf16-representable values."""

    shape: ConvShape
    x: np.ndarray
    w: np.ndarray
    gamma: np.ndarray
    beta: np.ndarray
    g: np.ndarray
    meta: dict = field(default_factory=dict)


def make_inputs(shape: ConvShape, cfg_id: int = 0, layer_id: int = 0, bf16: bool = True, affine: str = "init") -> BlockInputs:
    """Draw x, w, gamma, beta and the upstream gradient g for one block.

    x: U[0,1) for the image layer, N(0,1) otherwise.  w: U(-b, b), b = 1/sqrt(c_in * k * k).
    affine="init": gamma = 1, beta = 0 (fresh BN); affine="random": gamma ~ U[0.5,1.5], beta ~ N(0, 0.1).
    g ~ N(0,1).  Values are drawn in fp32 (from fp64 draws) and, if bf16, rounded to bf16 precision.
    """
    s = shape
    rx = _rng(cfg_id, layer_id, "x")
    if s.image_input:
        x = rx.random((s.n, s.h, s.w, s.c_in), dtype=np.float32)
    else:
        x = rx.standard_normal((s.n, s.h, s.w, s.c_in), dtype=np.float32)
    bound = 1.0 / np.sqrt(s.c_in * s.k * s.k)
    w = (_rng(cfg_id, layer_id, "w").random((s.c_out, s.k, s.k, s.c_in), dtype=np.float32) * 2.0 - 1.0) * np.float32(bound)
    g = _rng(cfg_id, layer_id, "g").standard_normal((s.n, s.ho, s.wo, s.c_out), dtype=np.float32)
    if affine == "init":
        gamma = np.ones(s.c_out, dtype=np.float32)
        beta = np.zeros(s.c_out, dtype=np.float32)
    elif affine == "random":
        gamma = (0.5 + _rng(cfg_id, layer_id, "gamma").random(s.c_out, dtype=np.float32)).astype(np.float32)
        beta = (0.1 * _rng(cfg_id, layer_id, "beta").standard_normal(s.c_out, dtype=np.float32)).astype(np.float32)
    else:
        raise ValueError(affine)
    if bf16:
        x, w, g = round_to_bf16(x), round_to_bf16(w), round_to_bf16(g)
    return BlockInputs(s, x, w, gamma, beta, g, {"cfg_id": cfg_id, "layer_id": layer_id, "bf16": bf16, "affine": affine})


def make_eval_stats(shape: ConvShape, cfg_id: int = 0, layer_id: int = 0):
    """Running statistics and a bias for the evaluation-mode / plain variants of one block (fp32 [c_out] each).

    A unit-variance input through a filter drawn as in make_inputs gives a convolution output of variance 1/3, so the
    running variance is U[0.25, 0.75), the running mean 0.2 * N(0,1); the bias of a plain layer is 0.5 * N(0,1).
    """
    c = shape.c_out
    rm = (0.2 * _rng(cfg_id, layer_id, "rm").standard_normal(c, dtype=np.float32)).astype(np.float32)
    rv = (0.25 + 0.5 * _rng(cfg_id, layer_id, "rv").random(c, dtype=np.float32)).astype(np.float32)
    bias = (0.5 * _rng(cfg_id, layer_id, "bias").standard_normal(c, dtype=np.float32)).astype(np.float32)
    return rm, rv, bias


def make_optimizer_inputs(sizes, cfg_id: int, step: int, grad_scale: float = 1.0):
    """Seeded fp32 gradients for optimiser step `step` over tensors of the given sizes, plus (for step 0) parameters.

    Parameters: 0.05 * N(0,1); gradients: grad_scale * N(0,1).  Returns (params or None, grads) as lists of fp32 arrays.
    """
    params = None
    if step == 0:
        params = [(0.05 * _rng(cfg_id, i, "w").standard_normal(n, dtype=np.float32)).astype(np.float32) for i, n in enumerate(sizes)]
    grads = [(np.float32(grad_scale) * _rng(cfg_id + 1000 * (step + 1), i, "g").standard_normal(n, dtype=np.float32)).astype(np.float32)
             for i, n in enumerate(sizes)]
    return params, grads
