"""Host-only checks of the C-ABI library: it loads, exports every declared symbol, and rejects
bad arguments before touching CUDA.  No compute calls."""
import ctypes
import os
import re

import pytest

from paper_2608_15241_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "lora_mixed_linear.h")


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    names = re.findall(r"\b([A-Za-z_][A-Za-z0-9_]*)\s*\([^;{]*\)\s*;", src)
    return sorted(set(names))


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert "lora_mixed_linear" in names and "register_adapter" in names and "retire_version" in names
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), f"{n} declared in the header but not exported"
    assert set(binding.EXPORTS) <= set(names)


def test_status_strings(lib):
    assert binding.lml_status_string(0) == "ok"
    texts = {binding.lml_status_string(i) for i in range(10)}
    assert len(texts) == 10


def test_invalid_arguments_are_rejected_on_the_host(lib):
    h = ctypes.c_void_p()
    INVALID = 1
    assert lib.lml_table_create(None, 0, 64, 64, 4) == INVALID
    assert lib.lml_table_create(ctypes.byref(h), 0, 60, 64, 4) == INVALID      # d_in not a multiple of 8
    assert lib.lml_table_create(ctypes.byref(h), 0, 64, 0, 4) == INVALID
    assert lib.lml_table_create(ctypes.byref(h), 0, 64, 64, 0) == INVALID
    assert lib.lml_table_create(ctypes.byref(h), 0, 64, 64, 65) == INVALID
    assert lib.lml_table_create(ctypes.byref(h), -1, 64, 64, 4) == INVALID
    assert h.value is None
    slot = ctypes.c_int(-1)
    assert lib.register_adapter(None, 0, 0, None, None, 4, 1.0, None, ctypes.byref(slot)) == INVALID
    assert lib.retire_version(None, 0, 0) == INVALID
    assert lib.lml_lookup(None, 0, 0, ctypes.byref(slot)) == INVALID
    assert lib.lora_mixed_linear(None, None, None, 1, None, None, 0, None, None, None, 0, None) == INVALID
    assert lib.lml_segment_tokens(None, None, 0, None, None, None, None) == INVALID
    assert lib.lml_workspace_bytes(None, 1, 1) == 0
    assert lib.lml_table_destroy(None) == INVALID


def test_create_without_a_gpu_fails_cleanly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("has a GPU")
    h = ctypes.c_void_p()
    st = lib.lml_table_create(ctypes.byref(h), 0, 64, 64, 4)
    assert st != 0 and h.value is None


def test_binding_raises_on_error(lib):
    with pytest.raises(binding.LmlError):
        binding.lml_table_create(0, 60, 64, 4)
