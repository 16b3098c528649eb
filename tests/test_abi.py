"""CPU-only checks of the C-ABI: the library loads, exports everything the header declares, and
rejects invalid instances before touching a GPU."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2508_06133_b200 import binding as kv
from paper_2508_06133_b200 import build as kb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    kb.build()
    return kv.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "kvsched.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sched_[a-z_]+)\s*\(", text)))


def test_header_and_library_agree(lib):
    names = declared_functions()
    assert "sched_init" in names and "sched_eval_batch" in names and "sched_sorted_f" in names \
        and "sched_local_search" in names
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(kv.EXPORTS) == names


def test_error_strings(lib):
    assert lib.sched_strerror(0) == b"ok"
    for code in range(-6, 0):
        assert lib.sched_strerror(code) not in (b"ok", b"unknown error code")
    assert lib.sched_strerror(-99) == b"unknown error code"


@pytest.mark.parametrize("s,o,M,code", [
    ([], [], 10, kv.E_INVAL),                 # n = 0
    ([0, 1], [1, 1], 10, kv.E_INVAL),         # s < 1
    ([1, 1], [1, 0], 10, kv.E_INVAL),         # o < 1
    ([1, 1], [1, 1], 0, kv.E_INVAL),          # M < 1
    ([5, 1], [6, 1], 10, kv.E_INVAL),         # s + o > M: the request could never be admitted
    ([1], [1], 1 << 30, kv.E_UNSUPPORTED),    # M too large for 32-bit occupancy cells
])
def test_invalid_instances_are_rejected_before_any_launch(lib, s, o, M, code):
    with pytest.raises(kv.SchedError) as e:
        kv.Scheduler(np.array(s, dtype=np.int32), np.array(o, dtype=np.int32), M)
    assert e.value.code == code


def test_null_arguments(lib):
    assert lib.sched_init(None, 1, None, None, 10) == kv.E_INVAL
    assert lib.sched_destroy(None) == kv.E_INVAL
    assert lib.sched_sync(None) == kv.E_INVAL
    h = C.c_void_p()
    assert lib.sched_init(C.byref(h), 2, None, None, 10) == kv.E_INVAL and not h.value
    big = np.ones((2, 2000), dtype=np.int32)
    assert lib.sched_init_batch(C.byref(h), 2, 2000, big.ctypes.data, big.ctypes.data, 10) == kv.E_UNSUPPORTED


def test_sources_name_no_closed_calls():
    banned = ["cudaMemcpy" + "BatchAsync", "cudaMemcpy3D" + "BatchAsync", "multicast" + "::cluster"]
    for dirpath, _, files in os.walk(os.path.join(ROOT, "paper_2508_06133_b200")):
        for f in files:
            if f.endswith((".cu", ".cuh", ".py", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                for b in banned:
                    assert b not in text, (f, b)
