"""ctypes binding of libnb_cbs.so: the same names as include/nb_cbs.h, argument marshalling only.

Every step of the path runs inside the library's CUDA kernels.  PyTorch appears only as the owner of
device memory (``tensor.data_ptr()``) and streams.  There is no fallback: if the shared library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_float, c_int, c_int32, c_size_t, c_uint32, c_void_p

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("NB_CBS_LIBRARY") or os.path.join(HERE, "libnb_cbs.so")  # (the variable: another build of the same library, for A/B timing)

NB_OK = 0
NB_ERR_INVALID_ARG, NB_ERR_UNSUPPORTED, NB_ERR_WORKSPACE, NB_ERR_ALIGNMENT = 1, 2, 3, 4
NB_ERR_CUDA, NB_ERR_ARCH, NB_ERR_TIMEOUT, NB_ERR_INTERNAL = 5, 6, 7, 8
NB_DTYPE_F32, NB_DTYPE_BF16, NB_DTYPE_F16 = 0, 1, 2
NB_MODE_BF16_TC, NB_MODE_F32_REF, NB_MODE_F16_TC = 0, 1, 2
NB_CBS_FLAG_FORCE_SIMT = 1
NB_CBS_FLAG_SEPARATE_FINALIZE = 2

EXPORTS = (
    "nb_abi_version", "nb_last_error", "nb_cbs_plan_create", "nb_cbs_plan_destroy", "nb_cbs_out_shape",
    "nb_cbs_workspace_bytes", "nb_cbs_plan_paths", "nb_cbs_poll_status", "nb_conv_bn_silu_fwd", "nb_bn_stats",
    "nb_conv_bn_silu_bwd_data", "nb_conv_bn_silu_bwd_weight", "nb_cbs_step_host_scratch_bytes",
    "nb_conv_bn_silu_step_host", "nb_cbs_launch_count", "nb_cbs_profile_enable", "nb_cbs_profile_site_name",
    "nb_cbs_profile_read", "nb_bn_stats_static", "nb_cbs_infer_workspace_bytes", "nb_conv_bn_silu_infer", "nb_conv_bias_act",
    "nb_bn_fold", "nb_sgd_plan_create", "nb_sgd_plan_destroy", "nb_sgd_workspace_bytes", "nb_sgd_upload", "nb_sgd_clip_nesterov_step", "nb_sgd_clip_nesterov_step_scaled",
    "nb_slice_add", "nb_maxpool5_fwd", "nb_maxpool5_bwd", "nb_upsample2", "nb_conv_bias_bwd", "nb_cbs_plan_set_pitches",
    "nb_cbs_plan_set_dx_target", "nb_cbs_plan_set_fwd_residual", "nb_cbs_plan_set_bwd_residual",
)


class nb_cbs_desc(Structure):
    _fields_ = [
        ("struct_size", c_uint32), ("n", c_int32), ("h", c_int32), ("w", c_int32), ("c_in", c_int32), ("c_out", c_int32),
        ("ksize", c_int32), ("stride", c_int32), ("eps", c_float), ("momentum", c_float), ("mode", c_int32), ("flags", c_uint32),
    ]


class nb_sgd_tensor(Structure):
    _fields_ = [("grad", c_void_p), ("param", c_void_p), ("momentum", c_void_p), ("param_bf16", c_void_p), ("numel", ctypes.c_int64),
                ("group", c_int32), ("copy_dtype", c_int32)]


class nb_sgd_hyper(Structure):
    _fields_ = [("struct_size", c_uint32), ("momentum", c_float), ("max_norm", c_float), ("lr", c_float * 3), ("weight_decay", c_float * 3),
                ("first_step", c_int32)]


class nb_scaler_hyper(Structure):
    _fields_ = [("struct_size", c_uint32), ("growth_factor", c_float), ("backoff_factor", c_float), ("floor_scale", c_float), ("growth_interval", c_int32)]


class NbError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"nb_cbs status {status}: {message}")
        self.status = status


_lib = None


def load() -> ctypes.CDLL:
    """Load the library (raises if it has not been built: there is no other implementation to fall back to)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2609_10632_b200.build` (nvcc, sm_100a)")
        lib = ctypes.CDLL(LIB_PATH)
        V = c_void_p
        FP = c_void_p  # float* passed as raw addresses
        lib.nb_abi_version.restype = c_uint32
        lib.nb_abi_version.argtypes = []
        lib.nb_last_error.restype = c_char_p
        lib.nb_last_error.argtypes = []
        lib.nb_cbs_plan_create.argtypes = [POINTER(nb_cbs_desc), c_int, POINTER(V)]
        lib.nb_cbs_plan_destroy.argtypes = [V]
        lib.nb_cbs_out_shape.argtypes = [V, POINTER(c_int32), POINTER(c_int32)]
        lib.nb_cbs_workspace_bytes.argtypes = [V, POINTER(c_size_t), POINTER(c_size_t)]
        lib.nb_cbs_plan_paths.argtypes = [V, POINTER(c_int32)]
        lib.nb_cbs_plan_set_pitches.argtypes = [V, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64]
        lib.nb_cbs_poll_status.argtypes = [V, V]
        lib.nb_cbs_plan_set_dx_target.argtypes = [V, ctypes.c_int64, c_int32]
        lib.nb_cbs_plan_set_fwd_residual.argtypes = [V, V, ctypes.c_int64]
        lib.nb_cbs_plan_set_bwd_residual.argtypes = [V, V, ctypes.c_int64, c_int32]
        lib.nb_conv_bn_silu_fwd.argtypes = [V, V, V, FP, FP, FP, FP, V, FP, FP, V, V, c_size_t, V]
        lib.nb_bn_stats.argtypes = [V, V, c_int32, FP, FP, FP, FP, V, c_size_t, V]
        lib.nb_conv_bn_silu_bwd_data.argtypes = [V, V, V, FP, FP, FP, FP, V, V, FP, FP, V, V, c_size_t, V]
        lib.nb_conv_bn_silu_bwd_weight.argtypes = [V, V, V, FP, V, c_size_t, V]
        lib.nb_cbs_step_host_scratch_bytes.argtypes = [V, POINTER(c_size_t)]
        lib.nb_conv_bn_silu_step_host.argtypes = [V, V, V, FP, FP, V, V, V, FP, FP, FP, V, c_size_t, V]
        lib.nb_bn_stats_static.argtypes = [V, c_int32, ctypes.c_int64, c_int32, c_float, FP, FP, FP, FP, V]
        lib.nb_cbs_infer_workspace_bytes.argtypes = [V, POINTER(c_size_t), POINTER(c_int32)]
        lib.nb_conv_bn_silu_infer.argtypes = [V, V, V, FP, FP, FP, FP, V, V, c_size_t, V]
        lib.nb_conv_bias_act.argtypes = [V, V, V, FP, c_int32, V, V, c_size_t, V]
        lib.nb_bn_fold.argtypes = [V, V, FP, FP, FP, FP, V, FP, V]
        lib.nb_conv_bias_bwd.argtypes = [V, V, V, V, V, FP, FP, V, c_size_t, V]
        lib.nb_sgd_plan_create.argtypes = [POINTER(nb_sgd_tensor), c_int32, c_int, POINTER(V)]
        lib.nb_sgd_plan_destroy.argtypes = [V]
        lib.nb_sgd_workspace_bytes.argtypes = [V, POINTER(c_size_t)]
        lib.nb_sgd_upload.argtypes = [V, V, c_size_t, V]
        lib.nb_sgd_clip_nesterov_step.argtypes = [V, V, c_size_t, POINTER(nb_sgd_hyper), FP, V]
        lib.nb_sgd_clip_nesterov_step_scaled.argtypes = [V, V, c_size_t, POINTER(nb_sgd_hyper), POINTER(nb_scaler_hyper), V, FP, V]
        lib.nb_slice_add.argtypes = [c_int32, ctypes.c_int64, c_int32, V, ctypes.c_int64, V, ctypes.c_int64, V, ctypes.c_int64, c_int32, V]
        lib.nb_maxpool5_fwd.argtypes = [c_int32, c_int32, c_int32, c_int32, c_int32, V, V, V, ctypes.c_int64, ctypes.c_int64, V]
        lib.nb_maxpool5_bwd.argtypes = [c_int32, c_int32, c_int32, c_int32, c_int32, V, V, V, c_int32, ctypes.c_int64, ctypes.c_int64, V]
        lib.nb_upsample2.argtypes = [c_int32, c_int32, c_int32, c_int32, c_int32, V, V, c_int32, c_int32, ctypes.c_int64, ctypes.c_int64, V]
        lib.nb_cbs_launch_count.argtypes = []
        lib.nb_cbs_launch_count.restype = ctypes.c_ulonglong
        lib.nb_cbs_profile_enable.argtypes = [V, c_int32]
        lib.nb_cbs_profile_site_name.argtypes = [c_int32]
        lib.nb_cbs_profile_site_name.restype = c_char_p
        lib.nb_cbs_profile_read.argtypes = [V, c_int32, POINTER(ctypes.c_double), POINTER(ctypes.c_int64)]
        for name in EXPORTS:
            if name not in ("nb_abi_version", "nb_last_error", "nb_cbs_launch_count", "nb_cbs_profile_site_name"):
                getattr(lib, name).restype = c_int32
        _lib = lib
    return _lib


def nb_last_error() -> str:
    return load().nb_last_error().decode()


def _check(status: int):
    if status != NB_OK:
        raise NbError(status, nb_last_error())


def _ptr(t):
    """Device (or host) address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    if hasattr(t, "ctypes"):
        return t.ctypes.data
    raise TypeError(type(t))


def _nbytes(t) -> int:
    if t is None:
        return 0
    if hasattr(t, "element_size"):
        return t.numel() * t.element_size()
    return t.nbytes


def _stream(stream):
    if stream is None:
        import torch

        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def nb_abi_version() -> int:
    return int(load().nb_abi_version())


class Plan:
    """Owner of one nb_cbs_plan handle."""

    def __init__(self, n, h, w, c_in, c_out, ksize, stride, eps=1e-3, momentum=0.03, mode=NB_MODE_BF16_TC, flags=0, device=0):
        self.desc = nb_cbs_desc(ctypes.sizeof(nb_cbs_desc), n, h, w, c_in, c_out, ksize, stride, eps, momentum, mode, flags)
        self.handle = c_void_p()
        self.device = device
        _check(load().nb_cbs_plan_create(byref(self.desc), device, byref(self.handle)))
        ho, wo = c_int32(), c_int32()
        _check(load().nb_cbs_out_shape(self.handle, byref(ho), byref(wo)))
        self.ho, self.wo = ho.value, wo.value
        f, b = c_size_t(), c_size_t()
        _check(load().nb_cbs_workspace_bytes(self.handle, byref(f), byref(b)))
        self.fwd_bytes, self.bwd_bytes = f.value, b.value
        p3 = (c_int32 * 3)()
        _check(load().nb_cbs_plan_paths(self.handle, p3))
        self.paths = {"fprop": p3[0], "dgrad": p3[1], "wgrad": p3[2]}
        ib, fused = c_size_t(), c_int32()
        _check(load().nb_cbs_infer_workspace_bytes(self.handle, byref(ib), byref(fused)))
        self.infer_bytes, self.infer_fused = ib.value, bool(fused.value)

    def set_pitches(self, ld_x=0, ld_a=0, ld_g=0):
        """x, a_out, g of the training calls are channel slices with these row pitches in elements (0 = dense)."""
        _check(load().nb_cbs_plan_set_pitches(self.handle, int(ld_x), int(ld_a), int(ld_g)))

    def set_fwd_residual(self, res=None, ld_res=0):
        """The forward call adds `res` (a tensor of the output's shape; row pitch ld_res elements, 0 = dense) to its output."""
        _check(load().nb_cbs_plan_set_fwd_residual(self.handle, _ptr(res), int(ld_res)))

    def set_bwd_residual(self, gres=None, ld_gres=0, accumulate=True):
        """The data-gradient call also adds (accumulate) or copies its incoming gradient g into `gres` (row pitch ld_gres, 0 = dense)."""
        _check(load().nb_cbs_plan_set_bwd_residual(self.handle, _ptr(gres), int(ld_gres), 1 if accumulate else 0))

    def set_dx_target(self, ld_dx=0, accumulate=False):
        """dx of the data-gradient call is a channel slice with this row pitch (0 = dense) and is added to, not overwritten."""
        _check(load().nb_cbs_plan_set_dx_target(self.handle, int(ld_dx), 1 if accumulate else 0))

    @classmethod
    def for_shape(cls, s, **kw):
        return cls(s.n, s.h, s.w, s.c_in, s.c_out, s.k, s.stride, **kw)

    @property
    def m(self):
        return self.desc.n * self.ho * self.wo

    def step_host_scratch_bytes(self) -> int:
        b = c_size_t()
        _check(load().nb_cbs_step_host_scratch_bytes(self.handle, byref(b)))
        return b.value

    def close(self):
        if self.handle:
            load().nb_cbs_plan_destroy(self.handle)
            self.handle = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def nb_cbs_launch_count() -> int:
    return int(load().nb_cbs_launch_count())


def nb_cbs_profile_enable(plan: Plan, enable: bool):
    _check(load().nb_cbs_profile_enable(plan.handle, 1 if enable else 0))


def nb_cbs_profile_read(plan: Plan) -> dict:
    """{site name: (total_ms, launches)} accumulated since profiling was enabled on this plan."""
    out = {}
    i = 0
    while True:
        name = load().nb_cbs_profile_site_name(i)
        if name is None:
            return out
        ms, n = ctypes.c_double(), ctypes.c_int64()
        _check(load().nb_cbs_profile_read(plan.handle, i, byref(ms), byref(n)))
        out[name.decode()] = (ms.value, n.value)
        i += 1


def nb_cbs_poll_status(plan: Plan, stream=None):
    _check(load().nb_cbs_poll_status(plan.handle, _stream(stream)))
    return nb_last_error()


def nb_conv_bn_silu_fwd(plan: Plan, x, w, gamma, beta, running_mean, running_var, y_saved, save_mean, save_invstd, a_out,
                        workspace, stream=None):
    _check(load().nb_conv_bn_silu_fwd(plan.handle, _ptr(x), _ptr(w), _ptr(gamma), _ptr(beta), _ptr(running_mean), _ptr(running_var),
                                      _ptr(y_saved), _ptr(save_mean), _ptr(save_invstd), _ptr(a_out), _ptr(workspace),
                                      _nbytes(workspace), _stream(stream)))


def nb_bn_stats(plan: Plan, y, y_dtype, mean, invstd, sum_, sumsq, workspace, stream=None):
    _check(load().nb_bn_stats(plan.handle, _ptr(y), y_dtype, _ptr(mean), _ptr(invstd), _ptr(sum_), _ptr(sumsq), _ptr(workspace),
                              _nbytes(workspace), _stream(stream)))


def nb_bn_stats_static(y, y_dtype, m, c, eps, mean, invstd, sum_=None, sumsq=None, stream=None):
    """Plan-free, workspace-free batch statistics on the current device (scratch is an array inside the library)."""
    _check(load().nb_bn_stats_static(_ptr(y), y_dtype, m, c, eps, _ptr(mean), _ptr(invstd), _ptr(sum_), _ptr(sumsq), _stream(stream)))


def nb_conv_bn_silu_bwd_data(plan: Plan, g, y_saved, save_mean, save_invstd, gamma, beta, w, dx, dgamma, dbeta, dy_out,
                             workspace, stream=None):
    _check(load().nb_conv_bn_silu_bwd_data(plan.handle, _ptr(g), _ptr(y_saved), _ptr(save_mean), _ptr(save_invstd), _ptr(gamma),
                                           _ptr(beta), _ptr(w), _ptr(dx), _ptr(dgamma), _ptr(dbeta), _ptr(dy_out), _ptr(workspace),
                                           _nbytes(workspace), _stream(stream)))


def nb_conv_bn_silu_bwd_weight(plan: Plan, x, dy, dw, workspace, stream=None):
    _check(load().nb_conv_bn_silu_bwd_weight(plan.handle, _ptr(x), _ptr(dy), _ptr(dw), _ptr(workspace), _nbytes(workspace),
                                             _stream(stream)))


def nb_conv_bn_silu_infer(plan: Plan, x, w, gamma, beta, running_mean, running_var, a_out, workspace, stream=None):
    _check(load().nb_conv_bn_silu_infer(plan.handle, _ptr(x), _ptr(w), _ptr(gamma), _ptr(beta), _ptr(running_mean), _ptr(running_var),
                                        _ptr(a_out), _ptr(workspace), _nbytes(workspace), _stream(stream)))


def nb_conv_bias_act(plan: Plan, x, w, bias, act, out, workspace, stream=None):
    _check(load().nb_conv_bias_act(plan.handle, _ptr(x), _ptr(w), _ptr(bias), int(act), _ptr(out), _ptr(workspace), _nbytes(workspace),
                                   _stream(stream)))


def nb_conv_bias_bwd(plan: Plan, x, w, dout, dx, dw, dbias, workspace, stream=None):
    _check(load().nb_conv_bias_bwd(plan.handle, _ptr(x), _ptr(w), _ptr(dout), _ptr(dx), _ptr(dw), _ptr(dbias), _ptr(workspace), _nbytes(workspace),
                                   _stream(stream)))


def nb_bn_fold(plan: Plan, w, gamma, beta, running_mean, running_var, w_folded, bias_folded, stream=None):
    _check(load().nb_bn_fold(plan.handle, _ptr(w), _ptr(gamma), _ptr(beta), _ptr(running_mean), _ptr(running_var), _ptr(w_folded),
                             _ptr(bias_folded), _stream(stream)))


def nb_conv_bn_silu_step_host(plan: Plan, host_x, host_w, host_gamma, host_beta, host_g, host_a, host_dx, host_dw, host_dgamma,
                              host_dbeta, device_scratch, stream=None):
    _check(load().nb_conv_bn_silu_step_host(plan.handle, _ptr(host_x), _ptr(host_w), _ptr(host_gamma), _ptr(host_beta), _ptr(host_g),
                                            _ptr(host_a), _ptr(host_dx), _ptr(host_dw), _ptr(host_dgamma), _ptr(host_dbeta),
                                            _ptr(device_scratch), _nbytes(device_scratch), _stream(stream)))


def nb_slice_add(dtype, rows, channels, out, ld_out, a, ld_a, b=None, ld_b=0, accumulate=False, stream=None):
    """out/a/b: raw device addresses (ints) of the slices' first elements, or tensors whose data_ptr is that address."""
    _check(load().nb_slice_add(int(dtype), int(rows), int(channels), _ptr(out), int(ld_out), _ptr(a), int(ld_a), _ptr(b), int(ld_b),
                               1 if accumulate else 0, _stream(stream)))


def nb_maxpool5_fwd(dtype, n, h, w, c, x, y, idx=None, stream=None, ld_x=0, ld_y=0):
    _check(load().nb_maxpool5_fwd(int(dtype), n, h, w, c, _ptr(x), _ptr(y), _ptr(idx), int(ld_x), int(ld_y), _stream(stream)))


def nb_maxpool5_bwd(dtype, n, h, w, c, g, idx, dx, accumulate=False, stream=None, ld_g=0, ld_dx=0):
    _check(load().nb_maxpool5_bwd(int(dtype), n, h, w, c, _ptr(g), _ptr(idx), _ptr(dx), 1 if accumulate else 0, int(ld_g), int(ld_dx), _stream(stream)))


def nb_upsample2(dtype, n, h, w, c, src, dst, backward=False, accumulate=False, ld_small=0, ld_large=0, stream=None):
    """2x nearest-neighbour upsampling (or its gradient); n, h, w, c and ld_small describe the SMALL tensor, ld_large the large one (pixel pitches, 0 = dense)."""
    _check(load().nb_upsample2(int(dtype), n, h, w, c, _ptr(src), _ptr(dst), 1 if backward else 0, 1 if accumulate else 0, int(ld_small), int(ld_large),
                               _stream(stream)))


class SgdPlan:
    """Owner of one nb_sgd_plan handle.  `tensors`: iterable of (grad, param, momentum, param_bf16 or None, group), each a
    device tensor (or a raw address with an explicit numel as a sixth item)."""

    def __init__(self, tensors, device=0):
        items = list(tensors)
        arr = (nb_sgd_tensor * max(len(items), 1))()
        for i, it in enumerate(items):
            grad, param, mom, lp, group = it[:5]
            numel = it[5] if len(it) > 5 else param.numel()
            copy_dtype = NB_DTYPE_F16 if (lp is not None and hasattr(lp, "dtype") and "float16" in str(lp.dtype) and "bfloat16" not in str(lp.dtype)) else 0
            arr[i] = nb_sgd_tensor(_ptr(grad), _ptr(param), _ptr(mom), _ptr(lp), int(numel), int(group), copy_dtype)
        self.count = len(items)
        self.handle = c_void_p()
        _check(load().nb_sgd_plan_create(arr, self.count, device, byref(self.handle)))
        b = c_size_t()
        _check(load().nb_sgd_workspace_bytes(self.handle, byref(b)))
        self.workspace_bytes = b.value

    def upload(self, workspace, stream=None):
        _check(load().nb_sgd_upload(self.handle, _ptr(workspace), _nbytes(workspace), _stream(stream)))

    def step(self, workspace, lr, weight_decay, momentum, max_norm, first_step, total_norm=None, stream=None):
        h = nb_sgd_hyper(ctypes.sizeof(nb_sgd_hyper), momentum, max_norm, (c_float * 3)(*lr), (c_float * 3)(*weight_decay), 1 if first_step else 0)
        _check(load().nb_sgd_clip_nesterov_step(self.handle, _ptr(workspace), _nbytes(workspace), byref(h), _ptr(total_norm), _stream(stream)))

    def step_scaled(self, workspace, state, lr, weight_decay, momentum, max_norm, first_step, growth_factor=2.0, backoff_factor=0.5, floor_scale=0.0,
                    growth_interval=2000, total_norm=None, stream=None):
        """`state`: a 16-byte device buffer laid out as nb_loss_scaler (float scale, int32 growth_tracker, int32 skipped, int32 reserved)."""
        h = nb_sgd_hyper(ctypes.sizeof(nb_sgd_hyper), momentum, max_norm, (c_float * 3)(*lr), (c_float * 3)(*weight_decay), 1 if first_step else 0)
        sc = nb_scaler_hyper(ctypes.sizeof(nb_scaler_hyper), growth_factor, backoff_factor, floor_scale, growth_interval)
        _check(load().nb_sgd_clip_nesterov_step_scaled(self.handle, _ptr(workspace), _nbytes(workspace), byref(h), byref(sc), _ptr(state), _ptr(total_norm),
                                                       _stream(stream)))

    def close(self):
        if self.handle:
            load().nb_sgd_plan_destroy(self.handle)
            self.handle = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
