"""CPU-side checks of the boundary: the C-ABI library builds, loads and exports what include/osscar.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "osscar.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(osscar_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    import paper_2403_12983_b200 as pkg
    L = pkg.lib()
    names = declared_functions()
    assert {"osscar_gram", "osscar_init_support", "osscar_local_search", "osscar_objective"} <= set(names)
    for name in names:
        assert hasattr(L, name), name
    assert set(pkg.binding.EXPORTS) == set(names)


def test_struct_layouts_match_header():
    import paper_2403_12983_b200.binding as b
    assert ctypes.sizeof(b.SearchParams) == 48
    assert b.SearchParams.accept_rel_tol.offset == 16 and b.SearchParams.loop_mode.offset == 32
    assert b.SearchParams.wait_limit_cycles.offset == 40
    assert ctypes.sizeof(b.SearchResult) == 96 and b.SearchResult.loop_driver.offset == 88
    assert b.SearchResult.obj_init.offset == 16 and b.SearchResult.ms_search.offset == 32


def test_host_side_argument_checks_need_no_gpu():
    import paper_2403_12983_b200 as pkg
    b = pkg.binding
    out = ctypes.c_size_t(0)
    L = pkg.lib()
    assert L.osscar_workspace_bytes(64, 64, 1, 32, ctypes.byref(out)) == b.OK and out.value > 0
    small = out.value
    assert L.osscar_workspace_bytes(28672, 7168, 1, 8602, ctypes.byref(out)) == b.OK
    assert 5e9 < out.value < 8e9 and out.value > small
    assert L.osscar_workspace_bytes(64, 64, 5, 3, ctypes.byref(out)) == b.E_SHAPE
    assert L.osscar_workspace_bytes(64, 64, 1, 0, ctypes.byref(out)) == b.E_SHAPE
    assert L.osscar_workspace_bytes(64, 64, 1, 65, ctypes.byref(out)) == b.E_SHAPE
    assert L.osscar_workspace_bytes(128 * 2, 64, 128, 1, ctypes.byref(out)) == b.E_SHAPE      # g above the supported maximum
    assert L.osscar_workspace_bytes(64, 64, 1, 32, None) == b.E_ARG
    assert L.osscar_destroy(None) == b.E_ARG
    assert L.osscar_status_string(b.E_NOTPD).decode().startswith("H restricted")


def test_no_cpu_fallback():
    import torch
    import paper_2403_12983_b200 as pkg
    if torch.cuda.is_available():
        pytest.skip("CUDA present")
    with pytest.raises(pkg.OsscarError):
        pkg.Solver()
    h = ctypes.c_void_p()
    assert pkg.lib().osscar_create(ctypes.byref(h), 0, None) == pkg.binding.E_CUDA


def test_product_does_not_import_the_oracle():
    pkg_dir = os.path.join(ROOT, "paper_2403_12983_b200")
    for dirpath, _, files in os.walk(pkg_dir):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower() or f == "__init__.py" and False, f
