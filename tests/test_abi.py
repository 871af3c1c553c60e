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


@pytest.mark.parametrize("B,L,F,chunk,lag", [(16, 1500, 128, 128, 256), (4, 90, 6, 3, 9), (5, 64, 8, 8, 16), (3, 10, 2, 4, 8),
                                           (4, 40, 4, 4, 64), (1, 33, 5, 8, 16), (8, 1000, 128, 64, 192)])
def test_staggered_subscale_schedule(B, L, F, chunk, lag):
    """Host logic of the staggered schedule (Section 4.2): every (row, position) is generated exactly once, in order;
    whenever row r generates positions up to p, row r - 1 has already finished position p + F (the future horizon),
    i.e. the conditioning of a whole call can be computed before it starts; the batch ramps up to min(B, ...) rows."""
    from paper_1802_08435_b200 import binding
    assert lag >= F + chunk and lag % chunk == 0
    calls = binding.wrnn_subscale_schedule(B, L, chunk, lag)
    done = [0] * B                       # positions finished per row
    active = {}                          # rows stepping at a global time (a row that ends inside a chunk has a call of its own)
    for (r_lo, n_rows, p_lo, n) in calls:
        assert n_rows >= 1 and 1 <= n <= chunk and 0 <= r_lo and r_lo + n_rows <= B
        t = p_lo + r_lo * lag
        active[t] = active.get(t, 0) + n_rows
        for b in range(n_rows):          # check against the state BEFORE this call (all its rows advance together)
            r, p = r_lo + b, p_lo - b * lag
            assert p == done[r], "rows advance contiguously"
            assert p + n <= L
            if r > 0:
                need = min(L, p + n - 1 + F + 1)          # positions [0, need) of row r - 1 feed this call's conditioning
                assert done[r - 1] >= need, (r, p, n, done[r - 1])
        for b in range(n_rows):
            done[r_lo + b] += n
    assert done == [L] * B
    assert max(active.values()) == min(B, (L + lag - 1) // lag)
    with pytest.raises(binding.WrnnError):
        binding.wrnn_subscale_schedule(B, L, chunk, lag + 1)
