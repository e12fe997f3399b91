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


def test_argument_validation_of_the_later_entry_points(lib):
    # rejected before anything touches a device, like the calls above
    import numpy as np
    from paper_2510_14557_b200.binding import _Packed
    null = None
    fake = ctypes.c_void_p(4096)
    odd = ctypes.c_void_p(4100)
    qr = lib.mxp_quantize_reordered
    assert qr(fake, 1, 4, 64, 64, null, 1, fake, fake, fake, null) == 1     # no ordering
    assert qr(fake, 1, 4, 64, 64, odd, 1, fake, fake, fake, null) == 1      # ordering not 16-byte aligned
    assert qr(fake, 1, 4, 48, 48, fake, 1, fake, fake, fake, null) == 1     # cols % 32
    assert qr(fake, 1, 4, 64, 64, fake, 1, fake, fake, null, null) == 1     # MX+ needs an index plane
    assert qr(fake, 1, 4, 64, 64, fake, 4, fake, fake, fake, null) == 2     # 6-bit modes: unsupported
    assert qr(fake, 1, 0, 64, 64, null, 1, null, null, null, null) == 0     # empty is a no-op
    nq = lib.mxp_nvfp4_quantize
    assert nq(fake, 1, 4, 64, 64, 0.0, 1, fake, fake, fake, null) == 1      # tensor scale must be > 0
    assert nq(fake, 1, 4, 64, 64, float("nan"), 1, fake, fake, fake, null) == 1
    assert nq(fake, 1, 4, 48, 48, 1.0, 1, fake, fake, fake, null) == 1      # cols % 32
    assert nq(fake, 1, 4, 64, 64, 1.0, 1, fake, fake, null, null) == 1      # NVFP4+ needs an index plane
    assert nq(fake, 1, 4, 64, 64, 1.0, 0, fake, ctypes.c_void_p(4097), null, null) == 1  # scales 2-byte aligned
    nd = lib.mxp_nvfp4_dequantize
    assert nd(fake, fake, null, 4, 64, 1.0, 1, fake, 0, 64, null) == 1      # NVFP4+ without indices
    assert nd(fake, fake, null, 4, 64, 1.0, 0, fake, 0, 60, null) == 1      # ld < cols
    assert nd(fake, fake, null, 0, 64, 1.0, 0, null, 0, 64, null) == 0      # empty
    b = _Packed(4096, 4096, 4096, 32, 256, 1)
    ch = lib.mxp_gemm_decode_chained
    assert ch(1, 32, 256, null, 256, ctypes.byref(b), fake, 1, 32, null, null) == 1   # no activations
    assert ch(1, 32, 256, fake, 250, ctypes.byref(b), fake, 1, 32, null, null) == 1   # lda < K
    assert ch(1, 33, 256, fake, 256, ctypes.byref(b), fake, 1, 33, null, null) == 1   # N mismatch
    assert ch(1, 32, 256, fake, 256, ctypes.byref(b), fake, 1, 32, ctypes.c_void_p(4104), null) == 1  # status block alignment
    assert ch(100, 32, 256, fake, 256, ctypes.byref(b), fake, 1, 32, null, null) == 2  # M > 64
    b6 = _Packed(4096, 4096, None, 32, 256, 3)
    assert ch(1, 32, 256, fake, 256, ctypes.byref(b6), fake, 1, 32, null, null) == 1  # 6-bit weights
    dp = lib.mxp_gemm_dense_prepacked
    wide32 = lib.mxp_gemm_prepack_bytes(32, 256, 1)
    assert dp(70, 32, 256, null, 256, ctypes.byref(b), fake, wide32, fake, 1, 32, fake, 1 << 20, null) == 1  # no activations
    assert dp(70, 32, 256, fake, 256, ctypes.byref(b), null, wide32, fake, 1, 32, fake, 1 << 20, null) == 1  # no prepacked copy
    assert dp(70, 32, 256, fake, 256, ctypes.byref(b6), fake, wide32, fake, 1, 32, fake, 1 << 20, null) == 1  # 6-bit weights
    assert dp(70, 32, 256, fake, 256, ctypes.byref(b), fake, wide32, fake, 1, 32, fake, 16, null) == 3       # workspace
    assert dp(70, 32, 256, fake, 256, ctypes.byref(b), fake, wide32 - 1024, fake, 1, 32, fake, 1 << 20, null) == 1  # copy of another size
    assert lib.mxp_gemm_dense_prepacked_workspace_bytes(70, 256) > 70 * 256 * 2
    assert lib.mxp_gemm_dense_prepacked_workspace_bytes(70, 96) == 0
    # the ordering rule runs on the host
    cnt = np.arange(64, dtype=np.int64)
    out = np.zeros(64, np.int32)
    co = lib.mxp_channel_order
    assert co(cnt.ctypes.data, 64, out.ctypes.data) == 0
    assert sorted(out.tolist()) == list(range(64)) and out[0] == 63 and out[32] == 62
    assert co(cnt.ctypes.data, 48, out.ctypes.data) == 1
    assert co(null, 64, out.ctypes.data) == 1


def test_prepacked_copies_are_checked_against_the_call(lib):
    # A prepacked weight copy is a bare device pointer: the calls that read one take its size and
    # refuse, before any launch, a copy made for another shape or for another pairing of operand
    # modes (a plain copy under an MXFP4+ partner would otherwise be read far past its end).
    from paper_2510_14557_b200.binding import _Packed
    null = None
    fake = ctypes.c_void_p(4096)
    M, N, K = 512, 384, 256
    MX, MXP = 0, 1
    PLAIN, WIDE, SPLIT, WIDE8 = 0, 1, 2, 3
    form = lib.mxp_gemm_prepack_form
    assert (form(MX, MX), form(MXP, MX), form(MX, MXP), form(MXP, MXP)) == (PLAIN, PLAIN, SPLIT, WIDE)
    # MX++ is read widened: the partner as 6-bit E2M3 codes, the MX++ operand itself as E4M3 bytes
    assert form(2, MX) == WIDE and form(MX, 2) == WIDE8 and form(MXP, 5) == WIDE8 and form(MXP, 3) == WIDE
    size = {f: lib.mxp_gemm_prepack_bytes(N, K, f) for f in (PLAIN, WIDE, SPLIT, WIDE8)}
    assert 0 < size[PLAIN] < min(size[SPLIT], size[WIDE]) and size[WIDE] < size[WIDE8] and len(set(size.values())) == 4
    assert size[WIDE] - size[PLAIN] == N * K * 3 // 4 and size[WIDE8] - size[PLAIN] == N * K
    assert lib.mxp_gemm_prepack_bytes(N, K, 6) == 0 and lib.mxp_gemm_prepack_bytes(N, 96, WIDE) == 0
    # MXFP6+ / MXFP8+ weights: two planes of E2M3 codes, three planes of E4M3 bytes
    assert form(MX, 4) == 4 and form(MXP, 6) == 5
    assert lib.mxp_gemm_prepack_bytes(N, K, 4) - size[PLAIN] == 2 * N * K * 3 // 4
    assert lib.mxp_gemm_prepack_bytes(N, K, 5) - size[PLAIN] == 3 * N * K
    ws = 1 << 30
    gp = lib.mxp_gemm_prepacked

    def call(amode, bmode, nbytes, n=N):
        a = _Packed(4096, 4096, 4096, M, K, amode)
        b = _Packed(4096, 4096, 4096, n, K, bmode)
        return gp(M, n, K, ctypes.byref(a), ctypes.byref(b), fake, nbytes, fake, 1, n, fake, ws, null)

    for amode, bmode in ((MX, MX), (MXP, MX), (MX, MXP), (MXP, MXP)):
        right = form(amode, bmode)
        for f in (PLAIN, WIDE, SPLIT, WIDE8):
            if f != right:
                assert call(amode, bmode, size[f]) == 1, (amode, bmode, f)
        assert call(amode, bmode, lib.mxp_gemm_prepack_bytes(N + 128, K, right)) == 1  # another shape's copy
    gr = lib.mxp_gemm_ready
    a = _Packed(4096, 4096, 4096, M, K, MXP)
    b = _Packed(4096, 4096, 4096, N, K, MX)
    # an MXFP4+ A prepared by the quantizer against a plain B reads B's plain copy, nothing else
    assert gr(M, N, K, ctypes.byref(a), ctypes.byref(b), fake, size[WIDE], fake, 1, N, fake, ws, null) == 1
    assert gr(M, N, K, ctypes.byref(a), ctypes.byref(b), fake, size[SPLIT], fake, 1, N, fake, ws, null) == 1
    both = _Packed(4096, 4096, 4096, N, K, MXP)
    assert gr(M, N, K, ctypes.byref(a), ctypes.byref(both), fake, size[PLAIN], fake, 1, N, fake, ws, null) == 1
    # mxp_gemm_prepack: the form must fit the operand's mode
    pk = lib.mxp_gemm_prepack
    assert pk(ctypes.byref(a), PLAIN, fake, ws, null) == 1      # an MXFP4+ operand has no plain form
    assert pk(ctypes.byref(b), SPLIT, fake, ws, null) == 1      # a plain operand has nothing to split
    assert pk(ctypes.byref(a), 7, fake, ws, null) == 1
    assert pk(ctypes.byref(a), WIDE8, fake, ws, null) == 1      # E2M3 codes are this operand's widened form
    pp = _Packed(4096, 4096, 4096, N, K, 2)
    assert pk(ctypes.byref(pp), WIDE, fake, ws, null) == 1      # ... and E4M3 bytes an MX++ operand's
