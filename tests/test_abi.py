"""CPU-side checks of the C-ABI library: it builds, loads and exports every declared symbol."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2409_09099_b200 import build
    path = build.build()
    return ctypes.CDLL(str(path))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "sste.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sste_[a-z0-9_]+)\s*\(", text)))


def test_exports_every_declared_symbol(lib):
    names = _declared_symbols()
    assert len(names) >= 18
    for n in ("sste_beta_init", "sste_project_compress", "sste_linear_fwd", "sste_mvue_sparsify",
              "sste_linear_bwd_input", "sste_linear_bwd_weight"):
        assert n in names
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_names(lib):
    from paper_2409_09099_b200 import binding
    assert sorted(binding.EXPORTS) == _declared_symbols()
    for n in binding.EXPORTS[7:13]:
        assert hasattr(binding.Context, n[len("sste_"):])


def test_host_only_queries(lib):
    lib.sste_workspace_bytes.restype = ctypes.c_size_t
    lib.sste_vals_bytes.restype = ctypes.c_size_t
    lib.sste_meta_bytes.restype = ctypes.c_size_t
    lib.sste_status_string.restype = ctypes.c_char_p
    assert lib.sste_workspace_bytes() >= 256
    assert lib.sste_vals_bytes(256, 512, 0) == 256 * 256 * 2
    assert lib.sste_vals_bytes(256, 512, 2) == 256 * 256
    assert lib.sste_meta_bytes(256, 512) == 256 * 512 // 8
    assert lib.sste_status_string(0) == b"ok"
    assert b"128" in lib.sste_status_string(2)
    # argument validation that needs no device
    handle = ctypes.c_void_p()
    assert lib.sste_create(ctypes.byref(handle), 0, None, ctypes.c_size_t(0)) == 5       # workspace missing
    assert lib.sste_create(None, 0, None, ctypes.c_size_t(0)) == 1
    assert lib.sste_destroy(None) == 1
    assert lib.sste_beta_init(None, None, 128, 128, 0, None, None) == 1


def test_product_path_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2409_09099_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle|sste_oracle|libsste_oracle", src, flags=re.M), f
