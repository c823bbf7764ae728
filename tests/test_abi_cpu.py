"""CPU-side checks of the boundary: the library builds, loads and exports what include/meteora.h declares.
No compute call is made here (there is no GPU on this side of the test suite)."""
import ctypes
import os
import re

import pytest

from paper_2405_13053_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "meteora.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(meteora_[a-z_]+)\s*\(", text)))


def test_header_functions_are_exported(lib):
    names = declared_functions()
    assert "meteora_linear_forward" in names and "meteora_gate_topk" in names
    assert "meteora_route" in names and "meteora_lora_delta" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in meteora.h but not exported"
    assert set(names) == set(binding.EXPORTS)      # the binding mirrors the header, name for name


def test_status_strings(lib):
    assert binding.meteora_status_string(0) == "ok"
    for code in range(-6, 0):
        assert binding.meteora_status_string(code) not in ("ok", "unknown status")
    assert binding.meteora_status_string(-99) == "unknown status"


def test_shape_validation_needs_no_gpu(lib):
    good = binding.make_shape(64, 256, 256, 4, 8, 2, __import__("torch").float32)
    assert binding.meteora_workspace_bytes(good) > 0
    for field, value in (("k", 0), ("k", 5), ("N", 129), ("r", 65), ("d_in", 0), ("T", -1), ("temperature", 0.0)):
        bad = binding.make_shape(64, 256, 256, 4, 8, 2, __import__("torch").float32)
        setattr(bad, field, value)
        assert binding.meteora_workspace_bytes(bad) == 0, field
    # null pointers are rejected on the host before any launch
    rc = lib.meteora_linear_forward(None, None, None, None, None, ctypes.byref(good), None, None, 0, None)
    assert rc == -1
    assert lib.meteora_set_tuning(b"no_such_knob", 1) == -1
    assert lib.meteora_route(None, 4, 3, 2, None, None, None, None) == -1      # k > N


def test_workspace_size_grows_with_tokens(lib):
    import torch
    a = binding.meteora_workspace_bytes(binding.make_shape(16, 4096, 4096, 28, 8, 2, torch.bfloat16))
    b = binding.meteora_workspace_bytes(binding.make_shape(128, 4096, 4096, 28, 8, 2, torch.bfloat16))
    assert 0 < a < b
