"""Host-only checks of the C ABI: the library builds, loads without a GPU and
exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2511_16964_b200 import build, binding
    build.build()
    return binding.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "pike.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pike_[a-z_]+)\s*\(", text)))


def test_header_declares_the_three_chains():
    names = _declared()
    for n in ("pike_linear_epilogue", "pike_mlp_block", "pike_attention_chain", "pike_create", "pike_destroy"):
        assert n in names


def test_every_declared_symbol_is_exported(lib):
    raw = ctypes.CDLL(lib._name)
    for name in _declared():
        assert hasattr(raw, name), f"{name} declared in pike.h but not exported"


def test_binding_export_list_matches_header():
    from paper_2511_16964_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_status_strings(lib):
    from paper_2511_16964_b200 import pike_status_string
    assert pike_status_string(0) == "ok"
    seen = {pike_status_string(c) for c in range(0, 11)}
    assert len(seen) == 11 and "unknown status" not in seen
    assert pike_status_string(99) == "unknown status"


def test_struct_layouts_match_the_header():
    from paper_2511_16964_b200 import binding
    assert ctypes.sizeof(binding.pike_tensor_t) == 8 + 4 + 4 + 32 + 32
    assert ctypes.sizeof(binding.pike_epilogue_t) == 28


def test_null_arguments_are_rejected_without_a_gpu(lib):
    assert lib.pike_create(None, 0) == 1                      # PIKE_ERR_NULL
    assert lib.pike_destroy(None) == 1
    n = ctypes.c_size_t(0)
    assert lib.pike_linear_epilogue_workspace(None, None, None, None, ctypes.byref(n)) == 1


def test_create_without_a_device_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = ctypes.c_void_p()
    rc = lib.pike_create(ctypes.byref(h), 0)
    assert rc != 0 and not h.value
