"""CPU-side checks of the boundary: the library builds, loads, and exports what the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2509_15235_b200 import build
    return ctypes.CDLL(build.build())


def _declared():
    text = open(os.path.join(ROOT, "include", "vispec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vispec_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert "vispec_tree_verify_attn" in names and "vispec_kv_compact" in names and len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} declared in vispec.h but not exported"


def test_binding_lists_the_same_entry_points():
    from paper_2509_15235_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_strerror_and_null_argument_handling_need_no_gpu(lib):
    lib.vispec_strerror.restype = ctypes.c_char_p
    assert lib.vispec_strerror(0) == b"ok"
    assert b"tree" in lib.vispec_strerror(-8)
    assert lib.vispec_ctx_create(None, None, 0) == -1          # VISPEC_E_NULL
    assert lib.vispec_ctx_destroy(None) == 0
    assert lib.vispec_workspace_bytes(None, None) == -1


def test_shape_validation_precedes_any_cuda_call(lib):
    from paper_2509_15235_b200.binding import VispecShape
    h = ctypes.c_void_p()
    for bad in (VispecShape(1, 129, 4, 4, 64, 512, 1), VispecShape(1, 8, 6, 4, 64, 512, 1),
                VispecShape(1, 8, 4, 4, 96, 512, 1), VispecShape(0, 8, 4, 4, 64, 512, 1),
                VispecShape(1, 8, 4, 4, 64, 4, 1)):
        assert lib.vispec_ctx_create(ctypes.byref(h), ctypes.byref(bad), 0) == -3   # VISPEC_E_SHAPE


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2509_15235_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src and "vispec_oracle" not in src
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            src = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2509_15235_b200" not in src and "vispec.h" not in src
