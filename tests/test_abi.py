"""The C-ABI library loads and exports every function include/retexo.h
declares; host-side argument validation rejects bad calls before any launch
(no GPU needed: these calls return before touching the device)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "retexo.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2302_13053_b200 import build
    return C.CDLL(build.build())


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(retexo_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_function_is_exported(lib):
    names = declared_functions()
    assert {"retexo_aggregate", "retexo_mlp_train_step", "retexo_embed", "retexo_cross_partition_bytes",
            "retexo_lmp_train"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name
    from paper_2302_13053_b200 import binding
    assert sorted(binding.EXPORTS) == names


def test_status_strings_and_sizes(lib):
    lib.retexo_status_string.restype = C.c_char_p
    assert lib.retexo_status_string(0) == b"ok"
    assert len({lib.retexo_status_string(i) for i in range(8)}) == 8
    lib.retexo_theta_size.restype = C.c_int64
    assert lib.retexo_theta_size(C.c_int32(10), C.c_int32(4), C.c_int32(3)) == 10 * 4 + 4 + 4 * 3 + 3
    assert lib.retexo_theta_size(C.c_int32(10), C.c_int32(0), C.c_int32(3)) == 33
    for fn in ("retexo_aggregate_workspace_size", "retexo_cross_partition_workspace_size"):
        getattr(lib, fn).restype = C.c_size_t
    assert lib.retexo_aggregate_workspace_size(C.c_int64(1000), C.c_int64(5000), C.c_int32(0), C.c_int32(64),
                                               C.c_int32(0)) >= 1000 * 4
    small = lib.retexo_cross_partition_workspace_size(C.c_int64(1000), C.c_int64(5000), C.c_int32(100))
    big = lib.retexo_cross_partition_workspace_size(C.c_int64(1000), C.c_int64(5000), C.c_int32(1000000))
    assert 0 < small < big


def test_bad_arguments_are_rejected_on_the_host(lib):
    from paper_2302_13053_b200.binding import _Csr, _Mlp
    INVALID, WORKSPACE = 1, 4
    g = _Csr(-1, 0, None, None)
    assert lib.retexo_aggregate(C.byref(g), 0, None, C.c_int64(4), 4, None, None, C.c_int64(4), 1, None,
                                C.c_int64(0), None, C.c_size_t(0), None) == INVALID
    g = _Csr(0, 0, None, None)       # an empty graph is a valid no-op
    assert lib.retexo_aggregate(C.byref(g), 0, None, C.c_int64(4), 4, None, None, C.c_int64(4), 1, None,
                                C.c_int64(0), None, C.c_size_t(0), None) == 0
    g = _Csr(4, 0, 1, None)          # null feature pointer, no outputs
    assert lib.retexo_aggregate(C.byref(g), 0, None, C.c_int64(4), 4, None, None, C.c_int64(4), 1, None,
                                C.c_int64(0), None, C.c_size_t(0), None) == INVALID
    assert lib.retexo_aggregate(C.byref(g), 7, C.c_void_p(256), C.c_int64(4), 4, None, C.c_void_p(256),
                                C.c_int64(4), 1, None, C.c_int64(0), None, C.c_size_t(0), None) == INVALID
    # valid shapes but no workspace
    assert lib.retexo_aggregate(C.byref(g), 0, C.c_void_p(256), C.c_int64(4), 4, None, C.c_void_p(256),
                                C.c_int64(4), 1, None, C.c_int64(0), None, C.c_size_t(0), None) == WORKSPACE
    dims = (C.c_int32 * 1)(4)
    assert lib.retexo_cross_partition_bytes(C.byref(g), C.c_void_p(256), 0, 1, dims, 4, None, None, None, None,
                                            None, None, None, C.c_size_t(0), None) == INVALID
    m = _Mlp(0, 4, 3, 256, None, None, 1, 0.1, 0.9, 0.999, 1e-8, 0)
    assert lib.retexo_mlp_train_step(C.byref(m), C.c_void_p(256), C.c_int64(8), C.c_int32(0),
                                     C.c_void_p(256), C.c_int64(4), None, None, None, C.c_int64(0), None, C.c_size_t(0), None) == INVALID
    m = _Mlp(8, 4, 3, 256, None, None, 1, 0.1, 0.9, 0.999, 1e-8, 0)      # Adam without moments
    assert lib.retexo_mlp_train_step(C.byref(m), C.c_void_p(256), C.c_int64(8), C.c_int32(0),
                                     C.c_void_p(256), C.c_int64(4), None, None, None, C.c_int64(0), None, C.c_size_t(0), None) == INVALID
    m = _Mlp(8, 4, 3, 256, None, None, 0, 0.1, 0.9, 0.999, 1e-8, 0)
    ALIGNMENT = 3
    assert lib.retexo_mlp_train_step(C.byref(m), C.c_void_p(256), C.c_int64(9), C.c_int32(0),
                                     C.c_void_p(256), C.c_int64(4), None, None, None, C.c_int64(0), None, C.c_size_t(0), None) == ALIGNMENT
    # a column of ones is claimed, but the rows have no room for it
    assert lib.retexo_mlp_train_step(C.byref(m), C.c_void_p(256), C.c_int64(8), C.c_int32(1),
                                     C.c_void_p(256), C.c_int64(4), None, None, None, C.c_int64(0), None, C.c_size_t(0), None) == INVALID
    assert lib.retexo_embed(C.byref(m), C.c_void_p(256), C.c_int64(8), None, C.c_int64(4), None, C.c_int64(0), None,
                            C.c_int64(0), None, C.c_int64(0), None, None, None, None, C.c_size_t(0), None) == WORKSPACE
