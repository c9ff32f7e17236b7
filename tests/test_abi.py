"""The C ABI library: it builds for sm_100a, loads without a GPU, exports every symbol the header
declares, and refuses to work (rather than falling back to anything) when there is no device."""
import ctypes
import os
import re

import pytest
import torch

from paper_2601_12917_b200 import build as zbuild
from paper_2601_12917_b200 import zgr

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "zgr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(zgr_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = zbuild.build()
    assert os.path.exists(path)
    L = ctypes.CDLL(path)
    names = _declared_symbols()
    assert {"zgr_init", "zgr_perturb", "zgr_restore_update", "zgr_set_coeffs_dtc", "zgr_destroy"} <= set(names)
    for name in names:
        assert hasattr(L, name), f"{name} is declared in zgr.h but not exported"


def test_error_strings_and_null_arguments():
    L = zgr.lib()
    assert zgr.strerror(zgr.OK) == "ok"
    for code in (zgr.EINVAL, zgr.ESTATE, zgr.ECUDA, zgr.ENOMEM, -99):
        assert isinstance(zgr.strerror(code), str) and zgr.strerror(code)
    h = ctypes.c_void_p()
    assert L.zgr_init(ctypes.byref(h), None, 0, None) == zgr.EINVAL
    assert L.zgr_perturb(None, 0, 1.0, None) == zgr.EINVAL
    assert L.zgr_restore_update(None, 0, 1.0, 1.0, 0.1, None) == zgr.EINVAL
    assert L.zgr_set_coeffs_dtc(None, 0, None, None, None, 8) == zgr.EINVAL
    assert L.zgr_launch_count(None) == -1
    L.zgr_destroy(None)


def test_current_device_check_of_the_launching_calls():
    # Every call that enqueues work compares the context's device with the current one through this host-only
    # function and returns ZGR_EINVAL on a mismatch, before anything is launched (a context's tables, tensor
    # maps and borrowed pointers are addresses of its own device).
    L = zgr.lib()
    assert L.zgr_debug_check_device(0, 0) == zgr.OK
    assert L.zgr_debug_check_device(3, 3) == zgr.OK
    assert L.zgr_debug_check_device(0, 1) == zgr.EINVAL
    assert L.zgr_debug_check_device(1, 0) == zgr.EINVAL
    assert L.zgr_debug_check_device(-1, -1) == zgr.EINVAL       # no valid device was current at zgr_init


def test_argument_validation_happens_before_any_device_work():
    L = zgr.lib()
    h = ctypes.c_void_p()
    fake = 0x10000  # never dereferenced on the host
    def init(t, cfg):
        arr = (zgr.ZgrTensor * 1)(t)
        return L.zgr_init(ctypes.byref(h), arr, 1, ctypes.byref(cfg))
    good_cfg = zgr.ZgrConfig(0.5, 1e-3, zgr.SCALE_UNIT, 32)
    assert init(zgr.ZgrTensor(fake, 4, 4, 9, 0, None), good_cfg) == zgr.EINVAL          # dtype
    assert init(zgr.ZgrTensor(fake, 0, 4, zgr.F32, 0, None), good_cfg) == zgr.EINVAL    # rows
    assert init(zgr.ZgrTensor(fake, 4, 4, zgr.F32, 2, None), good_cfg) == zgr.EINVAL    # rank without U
    assert init(zgr.ZgrTensor(fake, 4, 4, zgr.F32, 0, fake), good_cfg) == zgr.EINVAL    # U without rank
    assert init(zgr.ZgrTensor(fake + 2, 4, 4, zgr.F32, 0, None), good_cfg) == zgr.EINVAL  # misaligned for fp32
    assert init(zgr.ZgrTensor(fake, 4, 4, zgr.F32, 0, None), zgr.ZgrConfig(-0.1, 1e-3, 1, 32)) == zgr.EINVAL
    assert init(zgr.ZgrTensor(fake, 4, 4, zgr.F32, 0, None), zgr.ZgrConfig(0.5, 1e-3, 1, 8)) == zgr.EINVAL


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful on a machine without a GPU")
def test_no_device_is_an_error_not_a_fallback():
    L = zgr.lib()
    h = ctypes.c_void_p()
    arr = (zgr.ZgrTensor * 1)(zgr.ZgrTensor(0x10000, 4, 4, zgr.F32, 0, None))
    cfg = zgr.ZgrConfig(0.5, 1e-3, zgr.SCALE_UNIT, 32)
    rc = L.zgr_init(ctypes.byref(h), arr, 1, ctypes.byref(cfg))
    assert rc in (zgr.ECUDA, zgr.ENOMEM)
    assert not h.value
