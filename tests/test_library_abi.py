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
