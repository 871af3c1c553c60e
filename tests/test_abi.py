"""CPU-side checks of the C-ABI library: it builds for sm_100a, loads without a GPU and
exports every function include/wrnn.h declares; argument errors are reported without a device."""
import ctypes as C
import os
import re

import pytest

from paper_1802_08435_b200 import build as wbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    return wbuild.build()


def declared_functions():
    src = open(os.path.join(ROOT, "include", "wrnn.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    names = re.findall(r"\b(wrnn_[a-z_0-9]+)\s*\(", src)
    return sorted(set(names))


def test_header_declares_the_expected_entry_points():
    names = declared_functions()
    for n in ("wrnn_create", "wrnn_destroy", "wrnn_sample", "wrnn_step_teacher_forced", "wrnn_fold", "wrnn_unfold",
              "wrnn_sample_subscale", "wrnn_sample_host", "wrnn_poll_status", "wrnn_last_error"):
        assert n in names


def test_library_loads_and_exports_every_declared_symbol(libpath):
    L = C.CDLL(libpath)
    for n in declared_functions():
        assert hasattr(L, n), n


def test_binding_lists_the_same_names():
    from paper_1802_08435_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()
    for n in binding.EXPORTS:
        assert callable(getattr(binding, n))


def test_argument_errors_need_no_device(libpath):
    L = C.CDLL(libpath)
    L.wrnn_last_error.restype = C.c_char_p
    out = C.c_void_p()
    assert L.wrnn_create(None, 1, C.byref(out)) == 1 and not out.value
    assert b"null" in L.wrnn_last_error(None)
    assert L.wrnn_fold(None, 10, 3, None, None) == 1          # B must divide n_total
    assert L.wrnn_unfold(None, -1, 1, None, None) == 1
    assert L.wrnn_sample(None, None, 1, 1, 0, None, None, None) == 1
    assert L.wrnn_poll_status(None) == 1
    L.wrnn_destroy(None)
    L.wrnn_launch_count.restype = C.c_int64
    assert L.wrnn_launch_count() == 0


def test_create_without_a_device_fails_loudly(libpath):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    import numpy as np
    from paper_1802_08435_b200 import binding, synth
    w = synth.make_weights(8, cond_dim=0)
    with pytest.raises(binding.WrnnError) as e:
        binding.wrnn_create(w, "f32")
    assert e.value.code in (binding.WRNN_ERR_CUDA, binding.WRNN_ERR_UNSUPPORTED)
