"""Host-only checks of the C ABI: the library loads without a GPU, exports every declared entry
point, and rejects bad arguments before touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_2504_17096_b200 import binding as B
from paper_2504_17096_b200 import build as cuda_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    cuda_build.build()
    return B.load()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "sailor.h")).read()
    declared = set(re.findall(r"\b(sailor_[a-z_]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_struct_sizes_match_the_header(lib):
    assert C.sizeof(B.PlanRec) == 72 and C.sizeof(B.Run) == 4
    assert C.sizeof(B.Result) == 120 and C.sizeof(B.Stats) == 104
    assert C.sizeof(B.Space) == 152 and C.sizeof(B.Objective) == 32 and C.sizeof(B.IssueRates) == 48


def test_error_strings_and_null_arguments(lib):
    assert B.sailor_strerror(0) == "ok"
    for code in (B.E_ARG, B.E_RANGE, B.E_CUDA, B.E_NOMEM, B.E_DEVICE):
        assert B.sailor_strerror(code) not in ("ok", "unknown error")
    assert B.sailor_strerror(-99) == "unknown error"
    out = C.c_void_p()
    assert lib.sailor_create(None, None, None, 0, None, C.byref(out)) == B.E_ARG
    assert lib.sailor_destroy(None) == B.OK
    assert lib.sailor_set_availability(None, None) == B.E_ARG
    assert lib.sailor_simulate(None, None, 0, 0, None, None, None, None) == B.E_ARG
    n = C.c_uint64()
    assert lib.sailor_space_size(None, None, C.byref(n)) == B.E_ARG
    assert lib.sailor_plan(None, None, None, 1, None, None, None) == B.E_ARG
    assert lib.sailor_last_cuda_error(None) == 0
    assert lib.sailor_measure_issue_rates(0, None, 3, None) == B.E_ARG
    assert lib.sailor_measure_issue_rates(0, None, 0, C.byref(B.IssueRates())) == B.E_ARG


def test_library_reads_no_environment_variable():
    """The interface is plain structs: nothing in the library's sources looks at the environment."""
    csrc = os.path.join(ROOT, "paper_2504_17096_b200", "csrc")
    for f in os.listdir(csrc):
        assert "getenv" not in open(os.path.join(csrc, f)).read(), f


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2504_17096_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f


def test_zone_order_helper():
    from paper_2504_17096_b200 import binding as B
    assert len(B.all_zone_orders(3)) == 15 and len(B.all_zone_orders(4)) == 64 and len(B.all_zone_orders(5)) == 325
    assert B.all_zone_orders(3, 1) == [[0], [1], [2]]
    assert all(len(set(o)) == len(o) for o in B.all_zone_orders(4))
