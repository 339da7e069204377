"""The shared library loads without a GPU and exports every function include/fsharp.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__ as ge
    ge.build()
    from paper_2302_00787_b200 import binding
    return binding.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fsharp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fsharp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 16
    for n in names:
        assert hasattr(lib, n), n
    from paper_2302_00787_b200 import binding
    assert sorted(binding.EXPORTS) == names


def test_layout_queries_and_messages(lib):
    assert lib.fsharp_stats_doubles(64) == 2 * 64 * 64 + 2 * 64
    assert lib.fsharp_params_doubles(16) == 5 * 256 + 8
    assert lib.fsharp_strerror(0) == b"ok"
    assert b"shape" in lib.fsharp_strerror(-2)
    # argument checks that need no device
    assert lib.fsharp_create(None, 0, None) == -1
    assert lib.fsharp_destroy(None) == -1
    assert lib.fsharp_set_impl(None, 0) == -1


def test_no_gpu_means_an_error_not_a_fallback(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = ctypes.c_void_p()
    assert lib.fsharp_create(ctypes.byref(h), 0, None) == -9     # FSHARP_E_CUDA
    from paper_2302_00787_b200 import binding
    with pytest.raises(RuntimeError):
        binding.Context(0)


def test_product_never_imports_the_checker():
    pkg = os.path.join(ROOT, "paper_2302_00787_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, os.path.join(dirpath, f)
    src = open(os.path.join(ROOT, "oracle", "favor_sharp.py")).read()
    assert "paper_2302_00787_b200" not in src and "ctypes" not in src
