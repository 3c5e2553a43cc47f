"""Host-only checks of the C-ABI library: it loads without a GPU, exports every symbol that
include/*.h declare, and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

from paper_1910_06188_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared_functions():
    names = set()
    for header in sorted(os.listdir(os.path.join(ROOT, "include"))):
        text = open(os.path.join(ROOT, "include", header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(q8_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_header_and_binding_agree(lib):
    declared = _declared_functions()
    assert declared, "no declarations found in include/"
    assert sorted(binding.SIGNATURES) == declared
    for name in declared:
        assert hasattr(lib, name), f"libq8.so does not export {name}"
        assert callable(getattr(binding, name, None)) or name in ("q8_status_string",), name


def test_status_strings(lib):
    seen = set()
    for code in range(0, 11):
        s = binding.status_string(code)
        assert s and s != "unknown status" and s not in seen
        seen.add(s)
    assert binding.status_string(99) == "unknown status"


def test_workspace_size_formula(lib):
    assert binding.q8_linear_workspace_bytes(128, 768, 768) == 256 + 128 * 768
    assert binding.q8_linear_workspace_bytes(1, 8, 17) == 256 + 256
    assert binding.q8_linear_workspace_bytes(0, 8, 17) == 256
    assert binding.q8_calibrate_state_bytes() == 32


def test_argument_errors_need_no_device(lib):
    """These all return before any CUDA call, so they run on a machine without a GPU."""
    fake = 0x1000  # never dereferenced
    L = lib
    # NULL checks
    assert L.q8_linear(None, fake, fake, None, None, 0, fake, 4, 4, 16, fake, 1 << 20, None, None, None) == binding.Q8_ERR_NULL
    assert L.q8_linear(fake, fake, fake, None, None, 0, fake, 4, 4, 16, None, 1 << 20, None, None, None) == binding.Q8_ERR_NULL
    assert L.q8_linear_q(None, fake, fake, fake, None, 0, fake, 4, 4, 16, None, None, None) == binding.Q8_ERR_NULL
    assert L.q8_quantize_weight(fake, 4, 4, fake, None, None, None) == binding.Q8_ERR_NULL
    assert L.q8_quantize_activation(fake, 4, None, fake, None, None, None) == binding.Q8_ERR_NULL
    assert L.q8_calibrate(fake, 4, 0.5, None, None) == binding.Q8_ERR_NULL
    assert L.q8_embedding(None, 4, fake, fake, 10, 16, fake, None, None, None) == binding.Q8_ERR_NULL
    assert L.q8_poll_status(None, None, None) == binding.Q8_ERR_NULL
    # shapes
    assert L.q8_linear(fake, fake, fake, None, None, 0, fake, -1, 4, 16, fake, 1 << 20, None, None, None) == binding.Q8_ERR_SHAPE
    assert L.q8_linear(fake, fake, fake, None, None, 0, fake, 4, 4, 0, fake, 1 << 20, None, None, None) == binding.Q8_ERR_SHAPE
    assert L.q8_linear(fake, fake, fake, None, None, 0, fake, 4, 4, binding.Q8_MAX_K + 1, fake, 1 << 30, None, None, None) == binding.Q8_ERR_OVERFLOW
    assert L.q8_linear(fake, fake, fake, None, None, 0, fake, 1 << 31, 4, 16, fake, 1 << 40, None, None, None) == binding.Q8_ERR_SHAPE
    assert L.q8_embedding(fake, -1, fake, fake, 10, 16, fake, None, None, None) == binding.Q8_ERR_SHAPE
    assert L.q8_quantize_activation(fake, -5, fake, fake, None, None, None) == binding.Q8_ERR_SHAPE
    # enum / parameter values
    assert L.q8_linear(fake, fake, fake, None, None, 7, fake, 4, 4, 16, fake, 1 << 20, None, None, None) == binding.Q8_ERR_ARG
    assert L.q8_calibrate(fake, 4, 1.0, fake, None) == binding.Q8_ERR_ARG
    assert L.q8_calibrate(fake, 4, -0.1, fake, None) == binding.Q8_ERR_ARG
    assert L.q8_calibrate(fake, 4, float("nan"), fake, None) == binding.Q8_ERR_ARG
    # alignment
    assert L.q8_linear(fake + 2, fake, fake, None, None, 0, fake, 4, 4, 16, fake, 1 << 20, None, None, None) == binding.Q8_ERR_ALIGN
    assert L.q8_linear(fake, fake, fake, None, None, 0, fake, 4, 4, 16, fake + 64, 1 << 20, None, None, None) == binding.Q8_ERR_ALIGN
    assert L.q8_calibrate(fake, 4, 0.5, fake + 4, None) == binding.Q8_ERR_ALIGN
    # workspace
    assert L.q8_linear(fake, fake, fake, None, None, 0, fake, 4, 4, 16, fake, 256, None, None, None) == binding.Q8_ERR_WORKSPACE
    # empty problems are no-ops that never reach the device
    assert L.q8_linear(fake, fake, fake, None, None, 0, fake, 0, 4, 16, fake, 256, None, None, None) == binding.Q8_OK
    assert L.q8_linear(fake, fake, fake, None, None, 0, fake, 4, 0, 16, fake, 512, None, None, None) == binding.Q8_OK
    assert L.q8_linear_q(fake, fake, fake, fake, None, 0, fake, 0, 4, 16, None, None, None) == binding.Q8_OK
    assert L.q8_embedding(fake, 0, fake, fake, 10, 16, fake, None, None, None) == binding.Q8_OK


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libq8.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load()


def test_product_code_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_1910_06188_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"
