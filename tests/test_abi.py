"""CPU-only checks of the C-ABI library: it builds for sm_100a, loads, and
exports every symbol that include/tfps.h declares; host-side argument checks
that need no device answer with their error codes."""
from __future__ import annotations

import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "tfps.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tfps_[a-z0-9_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_1711_01912_b200 import build, tfps
    build.build_library()
    return tfps.lib()


def test_header_symbols_are_exported(lib):
    syms = declared_symbols()
    assert "tfps_eval_batch" in syms and "tfps_graph_create" in syms and len(syms) >= 12
    for s in syms:
        assert hasattr(lib, s), f"{s} declared in tfps.h but not exported"


def test_binding_lists_every_declared_symbol():
    from paper_1711_01912_b200 import tfps
    assert sorted(tfps.EXPORTS) == declared_symbols()
    for s in tfps.EXPORTS:
        assert callable(getattr(tfps, s)), f"binding lacks {s}"


def test_strerror_and_host_side_argument_checks(lib):
    from paper_1711_01912_b200 import tfps
    assert tfps.tfps_strerror(0) == "ok"
    assert "cycle" in tfps.tfps_strerror(tfps.ERR_CYCLE)
    h = ctypes.c_void_p()
    # negative size and missing arrays are rejected before any CUDA call
    assert lib.tfps_graph_create(ctypes.byref(h), -1, 0, None, None, None, None, None, None, 0, None, None, 0, 0, None) == tfps.ERR_INVALID_ARG
    assert lib.tfps_graph_create(ctypes.byref(h), 4, 0, None, None, None, None, None, None, 0, None, None, 0, 0, None) == tfps.ERR_INVALID_ARG
    assert h.value is None
    assert "required" in tfps.tfps_last_error()
    assert lib.tfps_graph_destroy(None) == 0
    assert lib.tfps_devices_set(None, 1, None, None, None, 1) == tfps.ERR_INVALID_ARG
    assert lib.tfps_eval_batch(None, 1, 16, None, None, None, None, None, None, None, None, 0, 0, None) == tfps.ERR_INVALID_ARG
    assert lib.tfps_transpose_u8(None, None, 4, 4, 2, None) == tfps.ERR_INVALID_ARG
    assert lib.tfps_eval_workspace_bytes(None, 4, 16, 0) == 0
