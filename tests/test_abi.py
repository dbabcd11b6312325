"""CPU-only checks of the C-ABI boundary: the library builds/loads, exports every declared symbol, and its
host-side logic answers without a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2502_05431_b200 import build as ape_build
from paper_2502_05431_b200 import libape

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ape_build.build()
    return libape.load()


def _declared():
    text = open(os.path.join(ROOT, "include", "ape.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ape_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/ape.h but not exported"
    assert sorted(libape.EXPORTS) == names


def test_status_strings(lib):
    assert libape.status_string(0) == "ok"
    seen = {libape.status_string(c) for c in range(-10, 1)}
    assert len(seen) == 11 and "unknown status" not in seen
    assert libape.status_string(-99) == "unknown status"


def test_null_arguments_are_rejected_without_a_device(lib):
    assert lib.ape_create(None, 0) == -1
    assert lib.ape_destroy(None) == -1
    assert lib.ape_plan_destroy(None) == -1
    n = C.c_size_t(0)
    assert lib.ape_plan_workspace_bytes(None, C.byref(n)) == -1
    assert lib.ape_attend(None, 1.0, 1.0, 0, None, 0, None) == -1
    assert lib.ape_encode_contexts(None, None, 0, None) == -1
    v = C.c_int32(0)
    assert lib.ape_get_status(None, C.byref(v)) == -1
    p = C.c_void_p()
    assert lib.ape_attend_plan(None, None, None, None, None, None, None, 0, 0, C.byref(p)) == -1


def test_create_fails_cleanly_without_gpu(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = C.c_void_p()
    rc = lib.ape_create(C.byref(h), 0)
    assert rc < 0 and not h.value


def test_binding_raises_when_library_is_missing(monkeypatch):
    monkeypatch.setattr(libape, "_lib", None)
    monkeypatch.setattr(libape, "LIB_PATH", "/nonexistent/libape.so")
    with pytest.raises(ImportError):
        libape.load()
