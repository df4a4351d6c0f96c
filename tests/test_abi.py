"""The C-ABI library builds for sm_100a, loads without a GPU and exports every function the public
header declares; host-side argument checks that need no device."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def header_functions():
    text = open(os.path.join(ROOT, "include", "aquakv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(aquakv_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2501_19392_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = header_functions()
    assert {"aquakv_encode", "aquakv_decode", "aquakv_decode_attn", "aquakv_create"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    from paper_2501_19392_b200 import api
    assert sorted(api.SYMBOLS) == names


def test_host_side_checks_without_a_device():
    from paper_2501_19392_b200 import api
    assert api.code_bytes(1024, 16) == 256 and api.code_bytes(1024, 64) == 384 and api.code_bytes(512, 256) == 256
    assert api.code_bytes(1000, 16) == -2          # unsupported d_kv
    assert api.code_bytes(1024, 32) == -2          # unsupported grid size
    assert api.status_string(0) == "ok" and "workspace" in api.status_string(-4)
    p = api.Params(1024, 1024, 1024, 3, 16, api.BF16)
    assert api.lib.aquakv_code_bytes(ctypes.byref(p)) == -2      # grid_dim must be 2
    h = ctypes.c_void_p()
    assert api.lib.aquakv_create(None, None, None, None, ctypes.byref(h)) == -1
    g = np.zeros((16, 2), np.float32)
    s = np.ones(1024, np.int8)
    p = api.Params(1024, 1024, 1024, 2, 16, api.BF16)
    bad = s.copy()
    bad[3] = 0
    assert api.lib.aquakv_create(ctypes.byref(p), g.ctypes.data, bad.ctypes.data, s.ctypes.data, ctypes.byref(h)) == -1
    g2 = g.copy()
    g2[0, 0] = np.nan
    assert api.lib.aquakv_create(ctypes.byref(p), g2.ctypes.data, s.ctypes.data, s.ctypes.data, ctypes.byref(h)) == -1
    assert api.lib.aquakv_destroy(None) == 0
    assert api.lib.aquakv_workspace_bytes(None, 100, 0) == 0
    assert api.lib.aquakv_encode(None, 1, *([None] * 2), 0, None, None, 0, *([None] * 10), 0, None, 0, None) == -1


def test_product_path_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2501_19392_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text and "aqo_" not in text, f
    src = open(os.path.join(ROOT, "oracle", "aquakv_oracle.c")).read() + open(os.path.join(ROOT, "oracle", "__init__.py")).read()
    assert "paper_2501_19392_b200" not in src and "aquakv.h" not in src
