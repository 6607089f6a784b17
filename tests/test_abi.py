"""The C-ABI library builds, loads without a GPU and exports every symbol the
public header declares (no compute calls here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2604_05650_b200 import build, binding
    build.build()
    return binding.load_library()


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(lvspec_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(lib):
    from paper_2604_05650_b200 import binding
    declared = _declared()
    assert {"lvspec_verify_attention", "lvspec_loose_accept"} <= declared
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert declared == set(binding.EXPORTS)


def test_struct_layouts_match_the_header():
    from paper_2604_05650_b200 import binding
    assert ctypes.sizeof(binding.AttnShape) == 32
    assert ctypes.sizeof(binding.Thresholds) == 16
    assert binding.Thresholds.n_loose.offset == 8


def test_status_strings_and_null_context(lib):
    assert lib.lvspec_status_string(0) == b"ok"
    assert lib.lvspec_status_string(5) != lib.lvspec_status_string(4)
    assert lib.lvspec_launch_count(None) == 0
    assert lib.lvspec_destroy(None) == 1
    assert lib.lvspec_set_stream(None, None) == 1


def test_create_fails_loudly_without_a_gpu(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2604_05650_b200 import binding
    with pytest.raises(binding.LvspecError):
        binding.Context(0)


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2604_05650_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".h", ".cuh")):
                text = open(os.path.join(dirpath, fn)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b", text, flags=re.M), fn
                assert "lvspec_oracle" not in text, fn
