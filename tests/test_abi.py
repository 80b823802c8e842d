"""The C-ABI library: it builds, loads without a GPU, and exports what include/tli.h declares."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2502_05202_b200 import build as tli_build, tli

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "tli.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tli_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    tli_build.build()
    lib = tli.load()
    names = declared_functions()
    assert set(tli.EXPORTS) <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_header_constants_match_the_binding():
    text = open(os.path.join(ROOT, "include", "tli.h")).read()
    for name in ("TLI_MAX_B", "TLI_MAX_K", "TLI_MAX_V"):
        assert int(re.search(r"#define\s+%s\s+(\d+)" % name, text).group(1)) == getattr(tli, name)
    for name, val in re.findall(r"\b(TLI_[A-Z0-9_]+)\s*=\s*(-?\d+)", text):
        assert getattr(tli, name) == int(val), name


def test_status_strings():
    lib = tli.load()
    for code in (0, -1, -2, -3, -4, -5):
        assert lib.tli_status_string(code)
    assert lib.tli_status_string(-99) == b"unknown code"


def test_id_map_is_validated_on_the_host_before_any_cuda_call():
    lib = tli.load()
    h = ctypes.c_void_p()

    def create(V_t, V_d, m):
        m = np.asarray(m, np.int32)
        return lib.tli_create(ctypes.byref(h), 0, V_t, V_d, m.ctypes.data)

    assert create(4, 3, [0, 0, -1]) == tli.TLI_ERR_BAD_MAP          # two drafter ids on one target id
    assert create(4, 3, [0, 4, -1]) == tli.TLI_ERR_BAD_MAP          # out of range
    assert create(4, 3, [0, -2, -1]) == tli.TLI_ERR_BAD_MAP
    assert create(0, 3, [0, 1, 2]) == tli.TLI_ERR_ARG
    assert create(tli.TLI_MAX_V + 1, 1, [0]) == tli.TLI_ERR_UNSUPPORTED
    assert lib.tli_create(None, 0, 1, 1, np.zeros(1, np.int32).ctypes.data) == tli.TLI_ERR_ARG
    assert lib.tli_create(ctypes.byref(h), 0, 1, 1, None) == tli.TLI_ERR_ARG
    assert lib.tli_destroy(None) == tli.TLI_ERR_ARG
    assert lib.tli_workspace_bytes(None, 1, 1, 0) == 0
    with pytest.raises(tli.TLIError):
        tli.tli_create(0, 4, 3, [0, 0, -1])
