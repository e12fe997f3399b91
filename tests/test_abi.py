"""The C-ABI library loads and exports what include/mxp.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2510_14557_b200 import build, binding
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "mxp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mxp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"mxp_quantize", "mxp_dequantize", "mxp_gemm"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    from paper_2510_14557_b200 import binding
    assert sorted(binding.EXPORTS) == names


def test_status_strings_and_version(lib):
    from paper_2510_14557_b200 import binding
    assert binding.status_string(0) == "ok"
    assert "invalid" in binding.status_string(1)
    assert "sm_100a" in binding.version()


def test_argument_validation_without_launch(lib):
    # every call below must be rejected before anything touches a device
    null = None
    fake = ctypes.c_void_p(4096)  # aligned, never dereferenced
    q = lib.mxp_quantize
    assert q(fake, 1, 4, 48, 48, 1, fake, fake, fake, null) == 1      # cols % 32
    assert q(fake, 1, 4, 64, 64, 1, fake, fake, null, null) == 1      # MX+ needs an index plane
    assert q(fake, 7, 4, 64, 64, 1, fake, fake, fake, null) == 1      # bad dtype
    assert q(fake, 1, 4, 64, 64, 9, fake, fake, fake, null) == 1      # bad mode
    assert q(fake, 1, 4, 64, 64, 6, fake, fake, null, null) == 1      # MXFP8+ needs an index plane
    assert q(fake, 1, 4, 64, 60, 1, fake, fake, fake, null) == 1      # ld < cols
    assert q(ctypes.c_void_p(4100), 1, 4, 64, 64, 1, fake, fake, fake, null) == 1  # misaligned
    assert q(null, 1, 0, 64, 64, 1, null, null, null, null) == 0      # empty is a no-op
    from paper_2510_14557_b200.binding import _Packed
    p = _Packed(4096, 4096, None, 4, 64, 1)
    assert lib.mxp_dequantize(ctypes.byref(p), fake, 0, 64, null) == 1  # MX+ without index
    p = _Packed(4096, 4096, 4096, 4, 64, 1)
    assert lib.mxp_dequantize(ctypes.byref(p), null, 0, 64, null) == 1
    b = _Packed(4096, 4096, 4096, 8, 128, 1)
    a = _Packed(4096, 4096, 4096, 4, 128, 1)
    g = lib.mxp_gemm
    assert g(4, 8, 128, fake, 128, ctypes.byref(a), ctypes.byref(b), fake, 1, 8, fake, 256, null) == 1  # both A forms
    assert g(4, 8, 128, null, 0, null, ctypes.byref(b), fake, 1, 8, fake, 256, null) == 1            # neither
    assert g(4, 9, 128, null, 0, ctypes.byref(a), ctypes.byref(b), fake, 1, 16, fake, 256, null) == 1  # N mismatch
    assert g(4, 8, 128, null, 0, ctypes.byref(a), ctypes.byref(b), fake, 1, 8, null, 0, null) == 3    # workspace
    assert lib.mxp_gemm_workspace_bytes(4, 8, 128, 0, 1, 1) >= 16
    assert lib.mxp_tensor_peak_probe(9, 1, None, None) == 1
