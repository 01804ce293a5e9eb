"""CPU-side checks of the C ABI: the library builds, loads, exports every symbol the header
declares, and rejects bad arguments on the host before anything is launched."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2512_19720_b200 import build
    path = build.build()
    from paper_2512_19720_b200 import api
    assert api.LIB_PATH == path
    return api.lib


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(pd_[a-z_0-9]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"pd_pack_delta", "pd_linear", "pd_linear_multivariant", "pd_merge"} <= names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/ but not exported"


def test_binding_lists_the_same_names(lib):
    from paper_2512_19720_b200 import api
    assert set(api.EXPORTS) <= declared_symbols()
    for n in ("pd_pack_delta", "pd_linear", "pd_linear_multivariant", "pd_merge"):
        assert callable(getattr(api, n))


def test_status_strings(lib):
    from paper_2512_19720_b200 import api
    seen = {api.status_string(c) for c in range(8)}
    assert len(seen) == 8 and api.status_string(0) == "ok"
    assert api.status_string(99) == "unknown status"


def test_workspace_sizes(lib):
    from paper_2512_19720_b200 import api
    assert api.workspace_bytes(api.OP_MERGE, 0, 0, 4096, 4096) == 0
    assert api.workspace_bytes(api.OP_PACK, 0, 0, 4096, 11008) >= 8 * (4096 + 11008)
    assert api.workspace_bytes(api.OP_LINEAR_MULTIVARIANT, 2112, 16, 4096, 4096) >= 4 * 2112 + 4 * 18
    assert api.workspace_bytes(api.OP_LINEAR, 16, 0, 4096, 4096) % 256 == 0


def test_host_side_argument_errors(lib):
    """None of these reaches a launch: the pointers are fake and never dereferenced on the host."""
    A = 0x10000  # aligned fake address
    INVALID, SHAPE, ALIGN, WS = 1, 2, 3, 4
    # pack
    assert lib.pd_pack_delta(None, A, 64, 64, A, A, A, A, 1 << 20, None) == INVALID
    assert lib.pd_pack_delta(A, A, 64, 64, A, None, None, A, 1 << 20, None) == INVALID
    assert lib.pd_pack_delta(A, A, 0, 64, A, A, A, A, 1 << 20, None) == INVALID
    assert lib.pd_pack_delta(A, A, 64, 48, A, A, A, A, 1 << 20, None) == SHAPE
    assert lib.pd_pack_delta(A + 2, A, 64, 64, A, A, A, A, 1 << 20, None) == ALIGN
    assert lib.pd_pack_delta(A, A, 64, 64, A, A, A, None, 0, None) == WS
    assert lib.pd_pack_delta(A, A, 64, 64, A, A, A, A, 16, None) == WS
    assert lib.pd_pack_delta(A, A, 64, 64, A, A, A, A + 16, 1 << 20, None) == WS
    # merge
    assert lib.pd_merge(A, A, None, 0, 64, 64, A, None) == INVALID
    assert lib.pd_merge(A, A, A, 7, 64, 64, A, None) == INVALID
    assert lib.pd_merge(A, A, A, 0, 64, 40, A, None) == SHAPE
    assert lib.pd_merge(A + 4, A, A, 0, 64, 64, A, None) == ALIGN
    # linear
    assert lib.pd_linear(None, 1, 64, A, A, A, 0, 64, 64, A, 64, A, 1 << 20, None) == INVALID
    assert lib.pd_linear(A, 0, 64, A, A, A, 0, 64, 64, A, 64, A, 1 << 20, None) == INVALID
    assert lib.pd_linear(A, 1, 32, A, A, A, 0, 64, 64, A, 64, A, 1 << 20, None) == INVALID  # ldx < d_in
    assert lib.pd_linear(A, 1, 64, A, A, None, 0, 64, 64, A, 64, A, 1 << 20, None) == INVALID  # mask without v
    assert lib.pd_linear(A, 1, 64, A, A, A, 0, 64, 70, A, 64, A, 1 << 20, None) == SHAPE
    assert lib.pd_linear(A, 1, 68, A, A, A, 0, 64, 64, A, 64, A, 1 << 20, None) == ALIGN  # ldx % 8
    assert lib.pd_linear(A, 1, 64, A, A, A, 0, 64, 64, A + 1, 64, A, 1 << 20, None) == ALIGN
    assert lib.pd_linear(A, 1, 64, A, A, A, 0, 64, 64, A, 64, None, 0, None) == WS
    # multivariant
    axes = (ctypes.c_uint8 * 2)(0, 1)
    bad_axes = (ctypes.c_uint8 * 2)(0, 5)
    assert lib.pd_linear_multivariant(A, 4, 64, None, A, A, A, 64, axes, 2, 64, 64, A, 64, A, 1 << 20, None) == INVALID
    assert lib.pd_linear_multivariant(A, 4, 64, A, A, A, A, 64, bad_axes, 2, 64, 64, A, 64, A, 1 << 20, None) == INVALID
    assert lib.pd_linear_multivariant(A, 4, 64, A, A, A, A, 32, axes, 2, 64, 64, A, 64, A, 1 << 20, None) == INVALID
    assert lib.pd_linear_multivariant(A, 4, 64, A, A, A, A, 64, axes, 2, 64, 64, A, 64, A, 64, None) == WS
    many = (ctypes.c_uint8 * 100)(*([0] * 100))
    assert lib.pd_linear_multivariant(A, 4, 64, A, A, A, A, 64, many, 100, 64, 64, A, 64, A, 1 << 20, None) == SHAPE
    assert lib.pd_launch_count() == 0


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2512_19720_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert not re.search(r"pd_oracle|libpd_oracle|from\s+oracle|import\s+oracle|oracle/", text), \
                    f"{fn} reaches into the oracle"
