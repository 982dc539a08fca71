"""CPU-side checks of the C-ABI boundary: the library loads, exports every symbol the header declares,
the binding covers them, and argument validation that needs no device behaves as documented."""
import ctypes as C
import os
import re

import pytest

import paper_2510_02470_b200 as sage

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "sage.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sage_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = sage.lib()
    names = declared_symbols()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/sage.h but not exported"


def test_binding_covers_header():
    assert sorted(sage.SIGNATURES) == declared_symbols()


def test_no_torch_types_in_header():
    text = open(os.path.join(ROOT, "include", "sage.h")).read()
    assert "torch" not in text.lower() and "at::" not in text and 'extern "C"' in text


def test_select_count_matches_rule():
    assert sage.sage_select_count(4096, 0.1) == 410
    assert sage.sage_select_count(50000, 0.3) == 15000
    assert sage.sage_select_count(3, 0.5) == 2
    assert sage.sage_select_count(10, -1.0) == 0 and sage.sage_select_count(10, 7.0) == 10
    assert sage.sage_select_count(0, 0.5) == 0 and sage.sage_select_count(5, float("nan")) == 0


def test_argument_validation_without_device():
    lib = sage.lib()
    h = C.c_void_p()
    assert lib.sage_fd_create(None, 10, 4, 0, 0) == 1
    assert lib.sage_fd_create(C.byref(h), 0, 4, 0, 0) == 1
    assert lib.sage_fd_create(C.byref(h), 10, 1, 0, 0) == 1
    assert lib.sage_fd_create(C.byref(h), 10, 257, 0, 0) == 5
    assert lib.sage_fd_create(C.byref(h), 10, 4, 9, 0) == 1
    assert h.value is None                                   # out untouched on error
    assert b"ell" in lib.sage_last_error() or b"bad" in lib.sage_last_error()
    assert lib.sage_fd_update(None, None, 1, 1, None) == 1
    assert lib.sage_fd_finalize(None, None) == 1
    assert lib.sage_select(None, -1, 0.1, None, None, None) == 1
    assert lib.sage_select(None, 5, float("nan"), None, None, None) == 1
    assert lib.sage_select(None, 0, 0.5, None, None, None) == 0   # empty input is fine
    lib.sage_fd_destroy(None)                                # allowed
    for s in range(8):
        assert lib.sage_status_string(s)
    assert b"sm_100a" in lib.sage_version()


def test_fails_loudly_without_cuda_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(sage.SageError) as e:
        sage.sage_fd_create(64, 4, sage.SAGE_F32, 0)
    assert e.value.status == 4


def test_product_never_imports_oracle():
    pkg = os.path.join(ROOT, "paper_2510_02470_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh", ".cpp")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text and "oracle/" not in text, f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".cpp")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2510_02470_b200" not in text, f
