"""The built shared library, interrogated without a GPU: it loads, exports every symbol the header declares,
reports its ABI revision, and rejects bad descriptors before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2609_10632_b200 import binding as nb
from paper_2609_10632_b200 import build as nbbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    nbbuild.build()
    return nb.load()


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(nb_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(lib):
    declared = _declared()
    assert declared == set(nb.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_abi_version_matches_header(lib):
    text = open(os.path.join(ROOT, "include", "nb_cbs.h")).read()
    want = int(re.search(r"#define NB_CBS_ABI_VERSION (\d+)u", text).group(1))
    assert nb.nb_abi_version() == want


def test_desc_struct_matches_header_size(lib):
    assert ctypes.sizeof(nb.nb_cbs_desc) == 48


def _create(lib, **over):
    d = dict(n=2, h=8, w=8, c_in=16, c_out=32, ksize=3, stride=1, eps=1e-3, momentum=0.1, mode=nb.NB_MODE_BF16_TC, flags=0)
    size = over.pop("struct_size", ctypes.sizeof(nb.nb_cbs_desc))
    d.update(over)
    desc = nb.nb_cbs_desc(size, d["n"], d["h"], d["w"], d["c_in"], d["c_out"], d["ksize"], d["stride"], d["eps"], d["momentum"], d["mode"], d["flags"])
    h = ctypes.c_void_p()
    st = lib.nb_cbs_plan_create(ctypes.byref(desc), 0, ctypes.byref(h))
    return st, h, nb.nb_last_error()


def test_bad_descriptors_are_rejected_before_any_cuda_call(lib):
    h = ctypes.c_void_p()
    assert lib.nb_cbs_plan_create(None, 0, ctypes.byref(h)) == nb.NB_ERR_INVALID_ARG
    assert "NULL" in nb.nb_last_error()
    for over, code, word in [
        (dict(struct_size=8), nb.NB_ERR_INVALID_ARG, "struct_size"),
        (dict(ksize=5), nb.NB_ERR_INVALID_ARG, "ksize"),
        (dict(stride=3), nb.NB_ERR_INVALID_ARG, "stride"),
        (dict(n=0), nb.NB_ERR_INVALID_ARG, "positive"),
        (dict(mode=7), nb.NB_ERR_INVALID_ARG, "mode"),
        (dict(eps=0.0), nb.NB_ERR_INVALID_ARG, "eps"),
        (dict(c_out=12), nb.NB_ERR_UNSUPPORTED, "c_out"),
        (dict(c_out=6, mode=nb.NB_MODE_F32_REF), nb.NB_ERR_UNSUPPORTED, "c_out"),
        (dict(n=1, h=1, w=1), nb.NB_ERR_INVALID_ARG, "at least 2"),
    ]:
        st, handle, msg = _create(lib, **over)
        assert st == code, (over, st, msg)
        assert word in msg, (over, msg)
        assert not handle.value


def test_null_plan_arguments(lib):
    assert lib.nb_cbs_plan_destroy(None) == nb.NB_OK
    ho, wo = ctypes.c_int32(), ctypes.c_int32()
    assert lib.nb_cbs_out_shape(None, ctypes.byref(ho), ctypes.byref(wo)) == nb.NB_ERR_INVALID_ARG
    assert lib.nb_conv_bn_silu_fwd(None, *([None] * 11), 0, None) == nb.NB_ERR_INVALID_ARG
    assert lib.nb_conv_bn_silu_bwd_data(None, *([None] * 12), 0, None) == nb.NB_ERR_INVALID_ARG
    assert lib.nb_conv_bn_silu_bwd_weight(None, None, None, None, None, 0, None) == nb.NB_ERR_INVALID_ARG
    assert lib.nb_bn_stats(None, None, 0, None, None, None, None, None, 0, None) == nb.NB_ERR_INVALID_ARG


def test_plan_create_without_a_device_fails_loudly(lib):
    import torch

    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    st, handle, msg = _create(lib)
    assert st == nb.NB_ERR_CUDA and msg
    with pytest.raises(nb.NbError):
        nb.Plan(2, 8, 8, 16, 32, 3, 1)


def test_sgd_plan_rejects_bad_lists_before_any_cuda_call(lib):
    h = ctypes.c_void_p()
    assert lib.nb_sgd_plan_create(None, 1, 0, ctypes.byref(h)) == nb.NB_ERR_INVALID_ARG
    arr = (nb.nb_sgd_tensor * 1)()
    arr[0] = nb.nb_sgd_tensor(0x1000, 0x2000, 0x3000, None, 16, 0, 0)
    assert lib.nb_sgd_plan_create(arr, 0, 0, ctypes.byref(h)) == nb.NB_ERR_INVALID_ARG
    arr[0].numel = 0
    assert lib.nb_sgd_plan_create(arr, 1, 0, ctypes.byref(h)) == nb.NB_ERR_INVALID_ARG
    arr[0].numel = 16
    arr[0].group = 3
    assert lib.nb_sgd_plan_create(arr, 1, 0, ctypes.byref(h)) == nb.NB_ERR_INVALID_ARG
    assert "group" in nb.nb_last_error()
    arr[0].group = 0
    arr[0].copy_dtype = 7
    assert lib.nb_sgd_plan_create(arr, 1, 0, ctypes.byref(h)) == nb.NB_ERR_INVALID_ARG
    arr[0].copy_dtype = nb.NB_DTYPE_F16
    arr[0].grad = 0x1004
    assert lib.nb_sgd_plan_create(arr, 1, 0, ctypes.byref(h)) == nb.NB_ERR_ALIGNMENT
    assert ctypes.sizeof(nb.nb_sgd_tensor) == 48 and ctypes.sizeof(nb.nb_sgd_hyper) == 40 and ctypes.sizeof(nb.nb_scaler_hyper) == 20


def test_status_codes_of_the_binding_match_the_header():
    text = open(os.path.join(ROOT, "include", "nb_cbs.h")).read()
    codes = dict((k, int(v)) for k, v in re.findall(r"\b(NB_(?:OK|ERR_[A-Z_]+)) = (\d+)", text))
    assert codes["NB_ERR_TIMEOUT"] == 7 and len(codes) == 9
    for name, value in codes.items():
        assert getattr(nb, name) == value, name


def test_device_code_reports_give_ups_through_the_named_constant_only():
    """The status word that nb_cbs_poll_status returns is written in ONE place (report_timeout in common.cuh, with
    NB_ERR_TIMEOUT from the header); no kernel source writes a literal code there.  And no kernel source contains a wait
    of one block for another (a spin on a global counter or flag): the only bounded waits are those of a CTA on its own
    mbarriers."""
    csrc = os.path.join(ROOT, "paper_2609_10632_b200", "csrc")
    writers = []
    for fn in sorted(os.listdir(csrc)):
        text = open(os.path.join(csrc, fn)).read()
        for m in re.finditer(r"atomicCAS\([^;]*ST_ERR[^;]*;", text):
            writers.append((fn, m.group(0)))
    assert len(writers) == 1 and writers[0][0] == "common.cuh" and "(int)NB_ERR_TIMEOUT" in writers[0][1], writers
    for fn in sorted(os.listdir(csrc)):
        text = open(os.path.join(csrc, fn)).read()
        assert "ld.acquire.gpu" not in text and "grid_wait" not in text and "cooperative" not in text, fn
