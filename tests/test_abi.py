"""Host-side checks that need no GPU: the library builds, loads and exports the declared ABI."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__ as ge
    ge.build()
    import paper_2506_20818_b200 as pkg
    return pkg.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "lp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lp_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 20
    for name in names:
        assert hasattr(lib, name), f"{name} declared in include/lp.h but not exported"


def test_binding_covers_header():
    import paper_2506_20818_b200 as pkg
    assert sorted(pkg.EXPORTS) == declared_functions()


def test_struct_layouts_match_header():
    import paper_2506_20818_b200 as pkg
    # lp_model_desc: 2 + 5 + 1 + 4 + 5 int32; lp_stats: 1 + 5 + 4 + 2 int64
    assert ctypes.sizeof(pkg.ModelDesc) == 4 * 17
    assert ctypes.sizeof(pkg.Stats) == 8 * 12


def test_create_without_gpu_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = ctypes.c_void_p()
    st = lib.lp_create(ctypes.byref(h), 0, None)
    assert st != 0 and not h.value
    assert b"CUDA" in lib.lp_last_error(None) or b"device" in lib.lp_last_error(None)


def test_null_context_is_rejected(lib):
    assert lib.lp_get_stats(None, None) == -1
    assert lib.lp_param_count(None, None) == -1
    lib.lp_destroy(None)


def test_product_does_not_import_oracle():
    pkg_dir = os.path.join(ROOT, "paper_2506_20818_b200")
    for dirpath, _, files in os.walk(pkg_dir):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, f"{f} mentions the oracle"
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            assert "paper_2506_20818_b200" not in open(os.path.join(ROOT, "oracle", f)).read()
