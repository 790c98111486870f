"""The C-ABI library builds, loads without a GPU, and exports every symbol include/fastvar.h declares;
host-only entry points and argument validation work with no device present (no compute calls here)."""
import ctypes
import os
import re

import pytest

from paper_2503_23367_b200 import binding as fv
from paper_2503_23367_b200 import build as fv_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    fv_build.build()
    return fv.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fastvar.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fv_[a-z0-9_]+)\s*\(", text)))


def test_header_and_binding_agree_and_symbols_exist(lib):
    names = declared_functions()
    assert len(names) >= 20
    assert sorted(fv.EXPORTS) == names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in fastvar.h but not exported"


def test_host_only_functions(lib):
    assert fv.fv_k_for(0.6, 13, 13) == 102
    assert fv.fv_k_for(0.6, 40, 40) == 960
    assert fv.fv_k_for(0.2, 128, 128) == 3277
    assert fv.fv_k_for(1.0, 5, 7) == 35
    assert fv.fv_k_for(1e-9, 5, 7) == 1
    assert lib.fv_status_string(0) == b"ok"
    assert lib.fv_status_string(6) == b"device-side wait expired"
    assert lib.fv_prune_select_workspace_bytes(2, 4096, 2048) >= 2 * 4096 * 4 + 2 * 128 * 2048 * 4


def test_argument_validation_happens_before_any_launch(lib):
    # NULL pointers and bad sizes are rejected on the host (no CUDA call is made)
    assert lib.fv_prune_select(None, 1, 2, 2, 8, 0.5, None, None, None, None, None, None, 0, None) == 1
    assert lib.fv_restore(None, 1, 1, None, None, 1, 1, 1, 1, 8, None, None, 0, None) == 1
    assert lib.fv_gather_ln(None, None, 1, 4, 4, 8, None, None, 0, None, None, None) == 1
    assert lib.fv_var_step(None, None, 1, 0, 1.0, None, None, None, None) == 1
    assert lib.fv_reset(None) == 1
    cfg = fv.fv_config(2, 256, 4, 4, 0, 1, 0, None, None, -1, 64)
    assert lib.fv_workspace_bytes(ctypes.byref(cfg)) == 0            # n_steps = 0 is invalid
    h = (ctypes.c_int32 * 2)(4, 8); w = (ctypes.c_int32 * 2)(4, 8)
    cfg = fv.fv_config(2, 256, 4, 4, 0, 1, 2, h, w, 0, 80)
    assert lib.fv_workspace_bytes(ctypes.byref(cfg)) > 64 * 256 * 2 * 4
    assert lib.fv_kv_bytes(ctypes.byref(cfg)) == 2 * 2 * 80 * 256 * 2
    assert lib.fv_cache_bytes(ctypes.byref(cfg)) == 16 * 256 * 4 + 2 * 2 * 16 * 256 * 2   # fp32 output map + sublayer caches


def test_struct_layouts_match_the_library(lib):
    import ctypes as C
    sizes = (C.c_size_t * 3)()
    lib.fv_struct_sizes(sizes)
    assert tuple(sizes) == (C.sizeof(fv.fv_config), C.sizeof(fv.fv_weights), C.sizeof(fv.fv_generator))
