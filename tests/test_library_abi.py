"""The C-ABI library builds, loads without a GPU and exports every symbol the public header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    from paper_2511_20390_b200.build import build
    return build()


def _declared():
    text = open(os.path.join(ROOT, "include", "free_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"^(?:int|size_t|const char\*)\s+(\w+)\s*\(", text, flags=re.M)
    assert len(names) >= 10
    return names


def test_header_symbols_are_exported(libpath):
    L = ctypes.CDLL(libpath)
    for name in _declared():
        assert hasattr(L, name), f"{name} declared in include/free_b200.h but not exported"


def test_binding_covers_the_header(libpath):
    from paper_2511_20390_b200 import binding
    assert sorted(_declared()) == binding.exported_symbols()
    L = binding.lib()
    assert L.free_strerror(0) == b"ok" and b"variance" in L.free_strerror(-5)
    assert b"unknown" in L.free_strerror(-99)


def test_struct_layouts_match_the_header(libpath):
    # sizes follow from the field lists of the header (LP64): guards against drift between the two
    from paper_2511_20390_b200 import binding as b
    assert ctypes.sizeof(b.BlockWeights) == 10 * 8
    assert ctypes.sizeof(b.ModelDesc) == 12 * 4 + 8 * 8 + 80 + 4 * 8
    assert ctypes.sizeof(b.DrafterDesc) == 8 + 2 * 8 + 80 + 4 * 8
    assert ctypes.sizeof(b.ScheduleDesc) == 8 + 4 * 8
    assert ctypes.sizeof(b.TrajStats) == 5 * 8 + 65 * 8 + 8 + 8
    assert ctypes.sizeof(b.SpecParams) == 4 + 4 + 8 + 8            # K, cfg_scale, lambda, use_graph (+ padding)


def test_argument_errors_need_no_gpu(libpath):
    from paper_2511_20390_b200 import binding
    L = binding.lib()
    assert L.spec_verify(1, 4, 16, *([None] * 11)) == -1                      # null pointers
    p = ctypes.c_void_p(4096)
    assert L.spec_verify(1, 0, 16, p, p, p, p, None, p, None, p, p, None, None) == -2     # K out of range
    assert L.spec_verify(1, 65, 16, p, p, p, p, None, p, None, p, p, None, None) == -2
    assert L.spec_verify(1, 4, 0, p, p, p, p, None, p, None, p, p, None, None) == -2      # d < 1
    q = ctypes.c_void_p(4100)
    assert L.spec_verify(1, 4, 16, q, p, p, p, None, p, None, p, p, None, None) == -3     # misaligned
    assert L.spec_verify(0, 4, 16, p, p, p, p, None, p, None, p, p, None, None) == 0      # empty batch


def test_schedule_constructors_errors_and_closed_forms(libpath):
    # the library's host-side schedule constructors: argument errors, and values that follow from the definitions
    import numpy as np
    from paper_2511_20390_b200 import binding, linear_schedule, respaced_schedule
    L = binding.lib()
    buf = [np.empty(8) for _ in range(4)]
    ptr = [a.ctypes.data_as(ctypes.c_void_p) for a in buf]
    assert L.free_schedule_linear(8, 1e-4, 2e-2, 0, 0.0, -1.0, None, *ptr[1:]) == -1          # null table
    assert L.free_schedule_linear(8, 1e-4, 2e-2, 7, 0.0, -1.0, *ptr) == -1                     # unknown variance mode
    assert L.free_schedule_linear(1, 1e-4, 2e-2, 0, 0.0, -1.0, *ptr) == -2                     # N < 2
    assert L.free_schedule_linear(8, 0.0, 2e-2, 0, 0.0, -1.0, *ptr) == -2                      # beta must lie in (0, 1)
    assert L.free_schedule_linear(8, 1e-4, 1.5, 0, 0.0, -1.0, *ptr) == -2
    assert L.free_schedule_linear(8, 1e-4, 2e-2, 2, 1.5, -1.0, *ptr) == -2                     # interpolation weight outside [0, 1]
    assert L.free_schedule_respaced(8, 4, 1e-4, 2e-2, 0, 0.0, -1.0, *ptr) == -2                # fewer original steps than kept
    assert L.free_schedule_linear(8, 1e-4, 2e-2, 0, 0.0, -1.0, *ptr) == 0
    with pytest.raises(ValueError):
        linear_schedule(8, variance=1.5)
    # two-step schedule by hand: alpha = (1-b0, 1-b1); sigma2 = (0, b1 b0 / (1 - a0 a1))
    b0, b1 = 0.1, 0.3
    t = linear_schedule(2, b0, b1)
    assert np.allclose(t["coef_x"], [1 / np.sqrt(0.9), 1 / np.sqrt(0.7)], rtol=1e-15)
    assert np.allclose(t["coef_eps"], [b0 / np.sqrt(b0 * 0.9), b1 / np.sqrt((1 - 0.63) * 0.7)], rtol=1e-15)
    assert t["sigma2"][0] == 0.0 and np.isclose(t["sigma2"][1], b1 * b0 / (1 - 0.63), rtol=1e-15)
    assert np.array_equal(t["t_embed_value"], [0.0, 1.0])
    # keeping every step of the full schedule changes nothing; the kept indices of 1000 -> 250 are 4 or 5 apart
    full, same = linear_schedule(50), respaced_schedule(50, 50)
    for k in full:
        assert np.allclose(full[k], same[k], rtol=1e-12, atol=1e-300)
    keep = respaced_schedule(250)["t_embed_value"]
    assert keep[0] == 0 and keep[-1] == 999 and set(np.diff(keep)) <= {4.0, 5.0}
