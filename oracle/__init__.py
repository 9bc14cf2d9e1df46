"""fp64 CPU oracle of the Conv2d -> BatchNorm(batch statistics) -> SiLU block (forward and backward).

TEST INFRASTRUCTURE ONLY.  Importers allowed: ``tests/``, ``__graft_entry__.smoke()`` and the
``cpu_baseline`` / ``--impl reference`` legs of ``bench.py``.  The product package never imports this
module and this module never imports the product package; the two share no code.

The arithmetic lives in ``oracle.c`` (direct loops, double precision); this file only compiles it with
gcc, loads it through ctypes and composes the stage functions in the order the definitions give:
conv -> batch statistics -> normalise+affine+SiLU, and backwards SiLU' -> BN backward -> dgrad, wgrad.
The paper (Sec. 3.2, Sec. 6, Table 2 rows 2-3) names these operators without printing formulas; the
definitions are those of the works it cites, with eps and momentum passed explicitly.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile oracle.c into liboracle.so next to it (gcc, OpenMP, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        dp = ctypes.POINTER(ctypes.c_double)
        ci = ctypes.c_int
        for name in ("oracle_conv_fwd", "oracle_conv_dgrad", "oracle_conv_wgrad"):
            getattr(lib, name).argtypes = [dp, dp, dp, ci, ci, ci, ci, ci, ci, ci]
            getattr(lib, name).restype = None
        lib.oracle_bn_stats.argtypes = [dp, ctypes.c_longlong, ci, ctypes.c_double, dp, dp, dp, dp, dp, ctypes.c_double]
        lib.oracle_bn_stats.restype = None
        lib.oracle_bn_silu_fwd.argtypes = [dp, ctypes.c_longlong, ci, dp, dp, dp, dp, dp]
        lib.oracle_bn_silu_fwd.restype = None
        lib.oracle_bn_silu_bwd.argtypes = [dp, dp, ctypes.c_longlong, ci, dp, dp, dp, dp, dp, dp, dp]
        lib.oracle_bn_silu_bwd.restype = None
        dbl = ctypes.c_double
        lib.oracle_bn_eval_act.argtypes = [dp, ctypes.c_longlong, ci, dp, dp, dp, dp, dbl, ci, dp]
        lib.oracle_bn_eval_act.restype = None
        lib.oracle_bias_act.argtypes = [dp, ctypes.c_longlong, ci, dp, ci, dp]
        lib.oracle_bias_act.restype = None
        lib.oracle_bn_fold.argtypes = [dp, ci, ctypes.c_longlong, dp, dp, dp, dp, dbl, dp, dp]
        lib.oracle_bn_fold.restype = None
        lib.oracle_out_extent.argtypes = [ci, ci, ci]
        lib.oracle_out_extent.restype = ci
        lib.oracle_num_threads.argtypes = []
        lib.oracle_num_threads.restype = ci
        _lib = lib
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double)) if a is not None else None


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def out_extent(size: int, k: int, stride: int) -> int:
    return int(_load().oracle_out_extent(size, k, stride))


def conv_fwd(x, w, stride: int):
    """x [N,H,W,Cin], w [Cout,k,k,Cin] -> y [N,Ho,Wo,Cout]; cross-correlation, zero pad k//2."""
    x, w = _f64(x), _f64(w)
    N, H, W, Cin = x.shape
    Cout, k, k2, Cin2 = w.shape
    assert k == k2 and Cin == Cin2
    Ho, Wo = out_extent(H, k, stride), out_extent(W, k, stride)
    y = np.empty((N, Ho, Wo, Cout), dtype=np.float64)
    _load().oracle_conv_fwd(_p(x), _p(w), _p(y), N, H, W, Cin, Cout, k, stride)
    return y


def conv_dgrad(dy, w, x_shape, stride: int):
    dy, w = _f64(dy), _f64(w)
    N, H, W, Cin = x_shape
    Cout, k, _, _ = w.shape
    assert dy.shape == (N, out_extent(H, k, stride), out_extent(W, k, stride), Cout)
    dx = np.empty((N, H, W, Cin), dtype=np.float64)
    _load().oracle_conv_dgrad(_p(dy), _p(w), _p(dx), N, H, W, Cin, Cout, k, stride)
    return dx


def conv_wgrad(x, dy, k: int, stride: int):
    x, dy = _f64(x), _f64(dy)
    N, H, W, Cin = x.shape
    Cout = dy.shape[-1]
    assert dy.shape == (N, out_extent(H, k, stride), out_extent(W, k, stride), Cout)
    dw = np.empty((Cout, k, k, Cin), dtype=np.float64)
    _load().oracle_conv_wgrad(_p(x), _p(dy), _p(dw), N, H, W, Cin, Cout, k, stride)
    return dw


def bn_stats(y, eps: float, running_mean=None, running_var=None, momentum: float = 0.0):
    """Per-channel mean, biased variance and invstd over all leading dims; running stats updated in place."""
    y = _f64(y)
    C = y.shape[-1]
    M = y.size // C
    mean, var, invstd = (np.empty(C, dtype=np.float64) for _ in range(3))
    if running_mean is not None:
        assert running_mean.dtype == np.float64 and running_var.dtype == np.float64
    _load().oracle_bn_stats(_p(y), M, C, float(eps), _p(mean), _p(var), _p(invstd),
                            _p(running_mean), _p(running_var), float(momentum))
    return mean, var, invstd


def bn_silu_fwd(y, mean, invstd, gamma, beta):
    y = _f64(y)
    C = y.shape[-1]
    a = np.empty_like(y)
    _load().oracle_bn_silu_fwd(_p(y), y.size // C, C, _p(_f64(mean)), _p(_f64(invstd)), _p(_f64(gamma)), _p(_f64(beta)), _p(a))
    return a


def bn_silu_bwd(g, y, mean, invstd, gamma, beta):
    g, y = _f64(g), _f64(y)
    C = y.shape[-1]
    dy = np.empty_like(y)
    dgamma, dbeta = np.empty(C, dtype=np.float64), np.empty(C, dtype=np.float64)
    _load().oracle_bn_silu_bwd(_p(g), _p(y), y.size // C, C, _p(_f64(mean)), _p(_f64(invstd)),
                               _p(_f64(gamma)), _p(_f64(beta)), _p(dy), _p(dgamma), _p(dbeta))
    return dy, dgamma, dbeta


@dataclass
class BlockResult:
    y: np.ndarray
    mean: np.ndarray
    var: np.ndarray
    invstd: np.ndarray
    a: np.ndarray
    dy: np.ndarray | None = None
    dgamma: np.ndarray | None = None
    dbeta: np.ndarray | None = None
    dx: np.ndarray | None = None
    dw: np.ndarray | None = None


def cbs_fwd(x, w, gamma, beta, stride: int, eps: float, running_mean=None, running_var=None, momentum: float = 0.0):
    """Whole block forward from (x, w, gamma, beta)."""
    y = conv_fwd(x, w, stride)
    mean, var, invstd = bn_stats(y, eps, running_mean, running_var, momentum)
    a = bn_silu_fwd(y, mean, invstd, gamma, beta)
    return BlockResult(y=y, mean=mean, var=var, invstd=invstd, a=a)


def cbs_fwd_bwd(x, w, gamma, beta, g, stride: int, eps: float, need_dx: bool = True):
    """Whole block forward and backward from (x, w, gamma, beta, g = dL/da); never from any other intermediates."""
    res = cbs_fwd(x, w, gamma, beta, stride, eps)
    k = np.shape(w)[1]
    res.dy, res.dgamma, res.dbeta = bn_silu_bwd(g, res.y, res.mean, res.invstd, gamma, beta)
    if need_dx:
        res.dx = conv_dgrad(res.dy, w, np.shape(x), stride)
    res.dw = conv_wgrad(x, res.dy, k, stride)
    return res


# ------------------------------------------------------------------ evaluation-mode and plain variants
def bn_eval_act(y, gamma, beta, running_mean, running_var, eps: float, act: bool = True):
    """Evaluation-mode BN (running statistics, Table 2 row 9) then SiLU when `act`."""
    y = _f64(y)
    C = y.shape[-1]
    a = np.empty_like(y)
    _load().oracle_bn_eval_act(_p(y), y.size // C, C, _p(_f64(gamma)), _p(_f64(beta)), _p(_f64(running_mean)), _p(_f64(running_var)),
                               float(eps), int(bool(act)), _p(a))
    return a


def bias_act(y, bias, act: bool):
    y = _f64(y)
    C = y.shape[-1]
    out = np.empty_like(y)
    _load().oracle_bias_act(_p(y), y.size // C, C, _p(_f64(bias)) if bias is not None else None, int(bool(act)), _p(out))
    return out


def bn_fold(w, gamma, beta, running_mean, running_var, eps: float):
    """Filter and bias of the convolution that equals conv -> evaluation-mode BN."""
    w = _f64(w)
    Cout = w.shape[0]
    wf, bf = np.empty_like(w), np.empty(Cout, dtype=np.float64)
    _load().oracle_bn_fold(_p(w), Cout, w.size // Cout, _p(_f64(gamma)), _p(_f64(beta)), _p(_f64(running_mean)), _p(_f64(running_var)),
                           float(eps), _p(wf), _p(bf))
    return wf, bf


def cbs_infer(x, w, gamma, beta, running_mean, running_var, stride: int, eps: float, act: bool = True):
    """Evaluation-mode block from (x, w, gamma, beta, running statistics): conv -> BN(running) -> SiLU."""
    return bn_eval_act(conv_fwd(x, w, stride), gamma, beta, running_mean, running_var, eps, act)


def conv_bias_act(x, w, bias, stride: int, act: bool = False):
    """Convolution with a per-channel bias and no normalisation (the head's output layers, Table 2 row 3)."""
    return bias_act(conv_fwd(x, w, stride), bias, act)


def conv_bias_bwd(x, w, g, stride: int):
    """Backward of conv_bias_act(act=False) given g = dL/d out: (dx, dw, dbias) with dbias_c = sum of g over all pixels."""
    g = _f64(g)
    k = np.shape(w)[1]
    return conv_dgrad(g, w, np.shape(x), stride), conv_wgrad(x, g, k, stride), g.reshape(-1, g.shape[-1]).sum(axis=0)
