"""The C-ABI library loads and exports every symbol include/milora.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "milora.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(milora_[a-z_0-9]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_2410_18035_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def test_header_declares_the_named_entry_points():
    names = _declared()
    for must in ("milora_route", "milora_apply_prefill", "milora_apply_decode", "milora_register_adapter",
                 "milora_register_router", "milora_group", "milora_create", "milora_destroy"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    for name in _declared():
        assert hasattr(lib, name), f"libmilora.so does not export {name}"


def test_binding_covers_every_declared_symbol():
    from paper_2410_18035_b200 import binding
    assert sorted(binding.SIGNATURES) == _declared()


def test_status_strings(lib):
    lib.milora_status_string.restype = ctypes.c_char_p
    seen = {lib.milora_status_string(i) for i in range(9)}
    assert len(seen) == 9 and lib.milora_status_string(0) == b"ok"
    # host-side argument validation needs no device
    assert lib.milora_create(None, None) == 1
    assert lib.milora_destroy(None) == 0
    lib.milora_set_decode_path.argtypes = [ctypes.c_void_p, ctypes.c_int]
    lib.milora_decode_path_for.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
    assert lib.milora_set_decode_path(None, 2) == 1
    assert lib.milora_decode_path_for(None, 1, 1, None) == 1
    lib.milora_apply_prefill_shared.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                                ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    assert lib.milora_apply_prefill_shared(None, 0, 1, None, None, None, None, None) == 1
    lib.milora_apply_decode_layers.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
    assert lib.milora_apply_decode_layers(None, None, 1, None) == 1


def test_product_path_does_not_touch_the_oracle():
    """Neither the package nor the synthetic-input module may import the oracle."""
    for sub in ("paper_2410_18035_b200", "synth"):
        for dirpath, _, files in os.walk(os.path.join(ROOT, sub)):
            for f in files:
                if f.endswith((".py", ".cu", ".h", ".cuh")):
                    src = open(os.path.join(dirpath, f)).read()
                    assert not re.search(r"^\s*(from|import)\s+oracle\b", src, flags=re.M), f
    for dirpath, _, files in os.walk(os.path.join(ROOT, "oracle")):
        for f in files:
            if f.endswith(".py"):
                src = open(os.path.join(dirpath, f)).read()
                assert "paper_2410_18035_b200" not in src, f
