"""fp64 CPU oracle of a CHAINED group of Conv-BN-SiLU blocks: the C2f unit of the paper's detector (Sec. 6), forward and
backward, composed from the single-block stage functions of this package and plain numpy slicing.

TEST INFRASTRUCTURE ONLY (same rules as the rest of this package).

C2f(c1 -> c2, n bottlenecks, shortcut): with c = c2 / 2
    a0 = CBS_1x1(x)                      [.., 2c]
    parts = [a0[.., :c], a0[.., c:]]
    for i < n:  t = parts[-1];  v = CBS_3x3(CBS_3x3(t));  parts.append(t + v if shortcut else v)
    out = CBS_1x1(concat(parts))         [.., c2]
Every CBS is conv -> BN(batch statistics) -> SiLU.  In the backward pass a tensor with several consumers receives the
sum of their gradients (a part feeds the concatenation, the next bottleneck and, with the shortcut, that bottleneck's sum).

Pins (tests/test_oracle_pins_chain.py): central finite differences of the whole unit with respect to inputs and filters,
n = 0 reducing to two blocks in sequence, and the shortcut's effect on a linearised case.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

import oracle


@dataclass
class BlockParams:
    w: np.ndarray
    gamma: np.ndarray
    beta: np.ndarray


@dataclass
class C2fResult:
    out: np.ndarray
    parts: list
    dx: np.ndarray | None = None
    grads: list = field(default_factory=list)  # per block, in layer order: (dw, dgamma, dbeta)


def _block_bwd(x_in, prm: BlockParams, fwd, g, stride=1):
    dy, dgamma, dbeta = oracle.bn_silu_bwd(g, fwd.y, fwd.mean, fwd.invstd, prm.gamma, prm.beta)
    dx = oracle.conv_dgrad(dy, prm.w, np.shape(x_in), stride)
    dw = oracle.conv_wgrad(x_in, dy, np.shape(prm.w)[1], stride)
    return dx, (dw, dgamma, dbeta)


def c2f_fwd_bwd(x, params, n: int, shortcut: bool, eps: float, g_out=None) -> C2fResult:
    """params: BlockParams in layer order cv1, m0.cv1, m0.cv2, ..., cv2.  g_out = dL/d out (None: forward only)."""
    assert len(params) == 2 + 2 * n
    x = np.asarray(x, dtype=np.float64)
    f_cv1 = oracle.cbs_fwd(x, params[0].w, params[0].gamma, params[0].beta, 1, eps)
    c = f_cv1.a.shape[-1] // 2
    parts = [f_cv1.a[..., :c], f_cv1.a[..., c:]]
    inner = []  # per bottleneck: (input t, fwd of cv1, fwd of cv2)
    for i in range(n):
        t = parts[-1]
        f1 = oracle.cbs_fwd(t, params[1 + 2 * i].w, params[1 + 2 * i].gamma, params[1 + 2 * i].beta, 1, eps)
        f2 = oracle.cbs_fwd(f1.a, params[2 + 2 * i].w, params[2 + 2 * i].gamma, params[2 + 2 * i].beta, 1, eps)
        inner.append((t, f1, f2))
        parts.append(t + f2.a if shortcut else f2.a)
    cat = np.concatenate(parts, axis=-1)
    f_cv2 = oracle.cbs_fwd(cat, params[-1].w, params[-1].gamma, params[-1].beta, 1, eps)
    res = C2fResult(out=f_cv2.a, parts=parts)
    if g_out is None:
        return res
    grads = [None] * len(params)
    dcat, grads[-1] = _block_bwd(cat, params[-1], f_cv2, np.asarray(g_out, dtype=np.float64))
    dparts = [dcat[..., j * c:(j + 1) * c].copy() for j in range(2 + n)]
    for i in reversed(range(n)):
        t, f1, f2 = inner[i]
        dv = dparts[2 + i]  # complete: the concatenation's share plus whatever bottleneck i+1 added
        du, grads[2 + 2 * i] = _block_bwd(f1.a, params[2 + 2 * i], f2, dv)
        dt, grads[1 + 2 * i] = _block_bwd(t, params[1 + 2 * i], f1, du)
        dparts[1 + i] = dparts[1 + i] + dt + (dv if shortcut else 0.0)
    da0 = np.concatenate(dparts[:2], axis=-1)
    res.dx, grads[0] = _block_bwd(x, params[0], f_cv1, da0)
    res.grads = grads
    return res


# ------------------------------------------------------------------ the other glue of the detector (Sec. 6): SPPF, upsampling
def maxpool5(x):
    """5x5 max-pool, stride 1, padding 2 (padding never wins), NHWC.  Returns (y, idx) with idx = r*5 + t of the FIRST
    maximum of the window in row-major order (r, t = offsets 0..4 from the window's top-left corner at (p-2, q-2))."""
    x = np.asarray(x, dtype=np.float64)
    N, H, W, C = x.shape
    y = np.full_like(x, -np.inf)
    idx = np.zeros(x.shape, dtype=np.int64)
    for r in range(5):
        for t in range(5):
            shifted = np.full_like(x, -np.inf)
            h0, h1 = max(0, 2 - r), min(H, H + 2 - r)  # output rows p with 0 <= p - 2 + r < H
            w0, w1 = max(0, 2 - t), min(W, W + 2 - t)
            shifted[:, h0:h1, w0:w1, :] = x[:, h0 - 2 + r:h1 - 2 + r, w0 - 2 + t:w1 - 2 + t, :]
            better = shifted > y  # strict: an equal later element does not replace the first maximum
            y = np.where(better, shifted, y)
            idx = np.where(better, r * 5 + t, idx)
    return y, idx


def maxpool5_bwd(g, idx):
    """Gradient of maxpool5: every output's gradient goes to the input element its window's first maximum came from."""
    g = np.asarray(g, dtype=np.float64)
    N, H, W, C = g.shape
    dx = np.zeros_like(g)
    n, p, q, c = np.meshgrid(np.arange(N), np.arange(H), np.arange(W), np.arange(C), indexing="ij")
    np.add.at(dx, (n, p - 2 + idx // 5, q - 2 + idx % 5, c), g)
    return dx


def upsample2(x):
    """Nearest-neighbour 2x upsampling, NHWC: y[n, 2h+a, 2w+b, c] = x[n, h, w, c]."""
    return np.repeat(np.repeat(np.asarray(x, dtype=np.float64), 2, axis=1), 2, axis=2)


def upsample2_bwd(g):
    g = np.asarray(g, dtype=np.float64)
    N, H2, W2, C = g.shape
    return g.reshape(N, H2 // 2, 2, W2 // 2, 2, C).sum(axis=(2, 4))


def round_bf16(a):
    """Round fp64 values to the nearest bf16 (ties to even), returned as fp64: the storage precision of activations."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    bits = f.view(np.uint32).astype(np.uint64)
    bits = (bits + 0x7FFF + ((bits >> 16) & 1)) & 0xFFFF0000
    return bits.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(a))


def sppf_fwd_bwd(x, params, eps: float, g_out=None, pool_in_bf16: bool = False):
    """SPPF unit (Sec. 6): a0 = CBS_1x1(x); p1 = pool(a0); p2 = pool(p1); p3 = pool(p2); out = CBS_1x1(concat(a0, p1, p2, p3)).
    Returns (out, parts, dx, grads) with grads per block (cv1, cv2) = (dw, dgamma, dbeta); dx, grads None without g_out.

    pool_in_bf16: which element of a window is the maximum is an integer decision taken on floating-point values; a
    16-bit implementation takes it on bf16-rounded activations, where near-equal candidates become exact ties (first
    one wins).  With this flag the first block's activations are rounded to bf16 before the pools, so that both sides
    decide in the same precision; everything else stays fp64."""
    assert len(params) == 2
    x = np.asarray(x, dtype=np.float64)
    f1 = oracle.cbs_fwd(x, params[0].w, params[0].gamma, params[0].beta, 1, eps)
    parts, idxs = [round_bf16(f1.a) if pool_in_bf16 else f1.a], []
    for _ in range(3):
        y, idx = maxpool5(parts[-1])
        parts.append(y)
        idxs.append(idx)
    cat = np.concatenate(parts, axis=-1)
    f2 = oracle.cbs_fwd(cat, params[1].w, params[1].gamma, params[1].beta, 1, eps)
    if g_out is None:
        return f2.a, parts, None, None
    c = f1.a.shape[-1]
    dcat, g2 = _block_bwd(cat, params[1], f2, np.asarray(g_out, dtype=np.float64))
    d = [dcat[..., j * c:(j + 1) * c].copy() for j in range(4)]
    for j in (3, 2, 1):  # part j = pool(part j-1): its complete gradient flows back into part j-1
        d[j - 1] += maxpool5_bwd(d[j], idxs[j - 1])
    dx, g1 = _block_bwd(x, params[0], f1, d[0])
    return f2.a, parts, dx, [g1, g2]


# ------------------------------------------------------------------ a whole dataflow graph of blocks and glue
def graph_fwd_bwd(ops, layers, params, x, eps: float, out_grads=None, pool_in_bf16: bool = False, storage_16bit: bool = False,
                  plain_layers=None, plain_params=None):
    """Interpret a dataflow description (a list of op dicts: "cbs" with a layer index, "slice", "add", "concat", "maxpool",
    "upsample"; see the detector's description in the workload module) forwards and, given gradients for some tensors,
    backwards.  layers[k] gives block k's stride; params[k] its BlockParams.  A tensor with several consumers receives
    the sum of their gradients.  Returns (tensors, grads, block_grads): dicts name -> array, and per layer (dw, dgamma, dbeta).
    pool_in_bf16: inputs of max-pools are rounded to bf16 first (see sppf_fwd_bwd).
    Op "plain" (convolution + bias, no BN, no activation) takes its shape from plain_layers[k] and (w, bias) from
    plain_params[k]; its gradients (dw, dbias) are returned in a fourth value when plain_layers is given.

    storage_16bit: model the STORAGE precision the benchmark spec fixes for a chained run -- activations, upstream gradients,
    dy and dx are bf16 tensors, the saved convolution output is fp16 -- by rounding exactly where a tensor is stored
    (after the convolution: fp16; after SiLU, after a residual add, after dy, after dx, after every accumulation into a
    gradient: bf16), while all arithmetic in between stays fp64.  A deep randomly initialised network amplifies
    perturbations from layer to layer, so two runs that round at different points drift apart geometrically; with the
    same rounding points the remaining differences are the arithmetic's alone."""
    r16 = round_bf16 if storage_16bit else (lambda a: a)
    T = {"img": np.asarray(x, dtype=np.float64)}
    saved = {}
    for o in ops:
        ins = [T[i] for i in o["ins"]]
        kind = o["op"]
        if kind == "cbs":
            k = o["layer"]
            if storage_16bit:
                y = oracle.conv_fwd(ins[0], params[k].w, layers[k].stride).astype(np.float16).astype(np.float64)
                mean, var, invstd = oracle.bn_stats(y, eps)
                f = oracle.BlockResult(y=y, mean=mean, var=var, invstd=invstd,
                                       a=round_bf16(oracle.bn_silu_fwd(y, mean, invstd, params[k].gamma, params[k].beta)))
            else:
                f = oracle.cbs_fwd(ins[0], params[k].w, params[k].gamma, params[k].beta, layers[k].stride, eps)
            saved[o["out"]] = f
            T[o["out"]] = f.a
        elif kind == "slice":
            T[o["out"]] = ins[0][..., o["c0"]:o["c1"]]
        elif kind == "add":
            T[o["out"]] = r16(ins[0] + ins[1])
        elif kind == "concat":
            T[o["out"]] = np.concatenate(ins, axis=-1)
        elif kind == "maxpool":
            src = round_bf16(ins[0]) if pool_in_bf16 else ins[0]
            T[o["out"]], saved[o["out"]] = maxpool5(src)
        elif kind == "upsample":
            T[o["out"]] = upsample2(ins[0])
        elif kind == "plain":
            w, bias = plain_params[o["layer"]]
            T[o["out"]] = r16(oracle.conv_bias_act(ins[0], w, bias, plain_layers[o["layer"]].stride))
        else:
            raise ValueError(kind)
    if out_grads is None:
        return (T, None, None) if plain_layers is None else (T, None, None, None)
    G = {k: np.asarray(v, dtype=np.float64).copy() for k, v in out_grads.items()}

    def give(name, g):
        G[name] = r16(G[name] + g) if name in G else r16(g)

    block_grads = [None] * len(layers)
    plain_grads = [None] * (len(plain_layers) if plain_layers is not None else 0)
    for o in reversed(ops):
        if o["out"] not in G:
            continue  # nothing downstream needs this tensor
        g = G[o["out"]]
        kind = o["op"]
        if kind == "cbs":
            k = o["layer"]
            if storage_16bit:
                f, prm = saved[o["out"]], params[k]
                dy, dgamma, dbeta = oracle.bn_silu_bwd(g, f.y, f.mean, f.invstd, prm.gamma, prm.beta)
                dy = round_bf16(dy)
                dx = round_bf16(oracle.conv_dgrad(dy, prm.w, np.shape(T[o["ins"][0]]), layers[k].stride))
                block_grads[k] = (oracle.conv_wgrad(T[o["ins"][0]], dy, np.shape(prm.w)[1], layers[k].stride), dgamma, dbeta)
            else:
                dx, block_grads[k] = _block_bwd(T[o["ins"][0]], params[k], saved[o["out"]], g, layers[k].stride)
            give(o["ins"][0], dx)
        elif kind == "slice":
            full = np.zeros_like(T[o["ins"][0]])
            full[..., o["c0"]:o["c1"]] = g
            give(o["ins"][0], full)
        elif kind == "add":
            give(o["ins"][0], g)
            give(o["ins"][1], g)
        elif kind == "concat":
            c0 = 0
            for name in o["ins"]:
                c = T[name].shape[-1]
                give(name, g[..., c0:c0 + c])
                c0 += c
        elif kind == "maxpool":
            give(o["ins"][0], maxpool5_bwd(g, saved[o["out"]]))
        elif kind == "upsample":
            give(o["ins"][0], upsample2_bwd(g))
        elif kind == "plain":
            k = o["layer"]
            dx, dw, db = oracle.conv_bias_bwd(T[o["ins"][0]], plain_params[k][0], g, plain_layers[k].stride)
            plain_grads[k] = (dw, db)
            give(o["ins"][0], r16(dx))
    return (T, G, block_grads) if plain_layers is None else (T, G, block_grads, plain_grads)
