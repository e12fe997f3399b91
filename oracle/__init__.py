"""MX+ CPU oracle: ctypes binding of ``mxp_oracle.c``.

TEST INFRASTRUCTURE ONLY.  Importable from ``tests/``, the smoke check and the
benchmark's CPU-baseline / reference legs.  The product package never imports it
and it never imports the product package.

The arithmetic lives in the C file (fp64, one block at a time, in the order the
paper gives it: Sec. 2 Eq. 1, Sec. 4.1-4.2, Sec. 5 Eq. 3 / Eq. 4).  This module only
marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

MODE_MXFP4 = 0
MODE_MXFP4_PLUS = 1
MODE_MXFP4_PP = 2  # MX++ (Sec. 4.3)
FMT_E2M3 = 6       # MXFP6 / MXFP6+ elements (Table "Concrete MX-compliant formats")
FMT_E4M3 = 8       # MXFP8 / MXFP8+ elements

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mxp_oracle.c")
_LIB = os.path.join(_HERE, "libmxp_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, -O2, OpenMP over rows)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            subprocess.check_call(
                ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                 "-fno-fast-math", "-ffp-contract=off", _SRC, "-o", tmp, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        # MXP_ORACLE_LIB: an already built alternative (the mutation test loads deliberately
        # broken copies of mxp_oracle.c through it to show that the pins notice)
        lib = ctypes.CDLL(os.environ.get("MXP_ORACLE_LIB") or build())
        i64, p, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        lib.oracle_quantize.argtypes = [p, ci, i64, i64, i64, ci, ci, p, p, p]
        lib.oracle_quantize.restype = ci
        lib.oracle_dequantize.argtypes = [p, p, p, i64, i64, ci, ci, p, i64]
        lib.oracle_dequantize.restype = ci
        lib.oracle_gemm_fp64.argtypes = [p, i64, p, i64, i64, i64, i64, p, i64]
        lib.oracle_gemm_fp64.restype = None
        lib.oracle_e2m1_value.argtypes = [ci]
        lib.oracle_e2m1_value.restype = ctypes.c_double
        lib.oracle_bm_split.argtypes = [ci, ctypes.POINTER(ci), ctypes.POINTER(ci)]
        lib.oracle_bm_split.restype = None
        lib.oracle_elem_value.argtypes = [ci, ci]
        lib.oracle_elem_value.restype = ctypes.c_double
        lib.oracle_quantize_wide.argtypes = [p, ci, i64, i64, i64, ci, ci, ci, p, p, p]
        lib.oracle_quantize_wide.restype = ci
        lib.oracle_dequantize_wide.argtypes = [p, p, p, i64, i64, ci, ci, ci, p, i64]
        lib.oracle_dequantize_wide.restype = ci
        lib.oracle_nvfp4_quantize.argtypes = [p, ci, i64, i64, ctypes.c_float, ci, p, p, p]
        lib.oracle_nvfp4_quantize.restype = ci
        lib.oracle_nvfp4_dequantize.argtypes = [p, p, p, i64, i64, ctypes.c_float, ci, p]
        lib.oracle_nvfp4_dequantize.restype = ci
        lib.oracle_e4m3_round.argtypes = [ctypes.c_double]
        lib.oracle_e4m3_round.restype = ci
        lib.oracle_pack6.argtypes = [p, i64, p]
        lib.oracle_pack6.restype = None
        lib.oracle_set_threads.argtypes = [ci]
        lib.oracle_max_threads.restype = ci
        lib.oracle_get_threads.restype = ci
        _lib = lib
    return _lib


def set_threads(n: int) -> None:
    _load().oracle_set_threads(int(n))


def get_threads() -> int:
    return int(_load().oracle_get_threads())


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def e2m1_value(code: int) -> float:
    return float(_load().oracle_e2m1_value(int(code)))


def bm_split(m: int):
    """Eq. 4: E2M1 magnitude codes of (BM_H, BM_L) for the 3-bit BM mantissa m."""
    h, l = ctypes.c_int(), ctypes.c_int()
    _load().oracle_bm_split(int(m), ctypes.byref(h), ctypes.byref(l))
    return h.value, l.value


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def quantize(x: np.ndarray, mode: int, k: int = 32, bf16_bits: bool = False):
    """Quantize a 2-D array along its rows in blocks of k.

    x: float32, float64, or (bf16_bits=True) uint16 holding bfloat16 bit patterns.
    Returns (nibbles[rows, cols/2], scales[rows, cols/k], bm_index[rows, cols/k]), uint8.
    """
    assert x.ndim == 2
    x = np.ascontiguousarray(x)
    if bf16_bits:
        assert x.dtype == np.uint16
        kind = 1
    elif x.dtype == np.float32:
        kind = 0
    elif x.dtype == np.float64:
        kind = 2
    else:
        raise TypeError(x.dtype)
    rows, cols = x.shape
    if cols % k or k % 2:
        raise ValueError("cols must be a multiple of the (even) block length")
    nib = np.zeros((rows, cols // 2), np.uint8)
    sc = np.zeros((rows, cols // k), np.uint8)
    idx = np.zeros((rows, cols // k), np.uint8)
    rc = _load().oracle_quantize(_ptr(x), kind, rows, cols, cols, k, mode,
                                 _ptr(nib), _ptr(sc), _ptr(idx))
    if rc != 0:
        raise ValueError("oracle_quantize rejected its arguments")
    return nib, sc, idx


def dequantize(nib: np.ndarray, sc: np.ndarray, idx, mode: int, k: int = 32) -> np.ndarray:
    """Eq. 3 decode to float64, shape [rows, cols]."""
    nib = np.ascontiguousarray(nib, np.uint8)
    sc = np.ascontiguousarray(sc, np.uint8)
    rows, half = nib.shape
    cols = half * 2
    if idx is None:
        idx = np.zeros_like(sc)
    idx = np.ascontiguousarray(idx, np.uint8)
    assert sc.shape == (rows, cols // k) and idx.shape == sc.shape
    out = np.empty((rows, cols), np.float64)
    rc = _load().oracle_dequantize(_ptr(nib), _ptr(sc), _ptr(idx), rows, cols, k, mode,
                                   _ptr(out), cols)
    if rc != 0:
        raise ValueError("oracle_dequantize rejected its arguments")
    return out


def elem_value(fmt: int, code: int) -> float:
    """Value of a magnitude code of the E2M3 (fmt 6) or E4M3 (fmt 8) element type."""
    return float(_load().oracle_elem_value(int(fmt), int(code)))


def quantize_wide(x: np.ndarray, fmt: int, plus: bool, k: int = 32, bf16_bits: bool = False):
    """MXFP6(+) / MXFP8(+): returns (codes[rows, cols] one per byte, scales, bm_index)."""
    assert x.ndim == 2
    x = np.ascontiguousarray(x)
    if bf16_bits:
        assert x.dtype == np.uint16
        kind = 1
    elif x.dtype == np.float32:
        kind = 0
    elif x.dtype == np.float64:
        kind = 2
    else:
        raise TypeError(x.dtype)
    rows, cols = x.shape
    if cols % k:
        raise ValueError("cols must be a multiple of the block length")
    codes = np.zeros((rows, cols), np.uint8)
    sc = np.zeros((rows, cols // k), np.uint8)
    idx = np.zeros((rows, cols // k), np.uint8)
    rc = _load().oracle_quantize_wide(_ptr(x), kind, rows, cols, cols, k, fmt, int(plus),
                                      _ptr(codes), _ptr(sc), _ptr(idx))
    if rc != 0:
        raise ValueError("oracle_quantize_wide rejected its arguments")
    return codes, sc, idx


def dequantize_wide(codes: np.ndarray, sc: np.ndarray, idx, fmt: int, plus: bool, k: int = 32) -> np.ndarray:
    codes = np.ascontiguousarray(codes, np.uint8)
    sc = np.ascontiguousarray(sc, np.uint8)
    rows, cols = codes.shape
    if idx is None:
        idx = np.zeros_like(sc)
    idx = np.ascontiguousarray(idx, np.uint8)
    out = np.empty((rows, cols), np.float64)
    rc = _load().oracle_dequantize_wide(_ptr(codes), _ptr(sc), _ptr(idx), rows, cols, k, fmt,
                                        int(plus), _ptr(out), cols)
    if rc != 0:
        raise ValueError("oracle_dequantize_wide rejected its arguments")
    return out


def pack6(codes: np.ndarray) -> np.ndarray:
    """6-bit storage of a [rows, cols] code array (cols % 4 == 0): [rows, 3 cols / 4] bytes."""
    codes = np.ascontiguousarray(codes, np.uint8)
    rows, cols = codes.shape
    assert cols % 4 == 0
    out = np.zeros((rows, cols // 4 * 3), np.uint8)
    _load().oracle_pack6(_ptr(codes), rows * cols, _ptr(out))
    return out


def gemm_fp64(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """D = A @ B.T in fp64 by a plain triple loop (A: M x K, B: N x K)."""
    a = np.ascontiguousarray(a, np.float64)
    b = np.ascontiguousarray(b, np.float64)
    m, k = a.shape
    n, k2 = b.shape
    assert k == k2
    d = np.empty((m, n), np.float64)
    _load().oracle_gemm_fp64(_ptr(a), k, _ptr(b), k, m, n, k, _ptr(d), n)
    return d


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float64."""
    u = bits.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def channel_order(outlier_count) -> np.ndarray:
    """Channel ordering that scatters outlier channels over the blocks (Sec. 8, "Scattering
    outliers with channel reordering"), as int32 [cols]: position p takes channel order[p].

    Channels are ranked by outlier count, most first (equal counts: lower channel first).
    The cols/32 highest-ranked channels go one to each block, at the block's first position.
    The other channels are cut into the half with more outliers and the half with fewer
    (the odd one out joins the latter); the positions still free are filled front to back,
    first with the half that has fewer outliers, then with the half that has more, each in
    ranked order.  (The passage leaves the direction of "remaining places" and the handling
    of ties and odd counts open; this is the reading the library documents.)"""
    cnt = [int(c) for c in np.asarray(outlier_count).reshape(-1)]
    cols = len(cnt)
    assert cols > 0 and cols % 32 == 0
    nblk = cols // 32
    ranked = sorted(range(cols), key=lambda c: (-cnt[c], c))
    order = [-1] * cols
    for j in range(nblk):
        order[32 * j] = ranked[j]
    rest = ranked[nblk:]
    more, fewer = rest[:len(rest) // 2], rest[len(rest) // 2:]
    free = [p for p in range(cols) if p % 32 != 0]
    for p, c in zip(free, fewer + more):
        order[p] = c
    return np.asarray(order, np.int32)


def quantize_reordered(x: np.ndarray, order: np.ndarray, mode: int, bf16_bits: bool = False):
    """Quantization of the rows with their channels taken in `order` (same passage): the
    definition is quantize(x[:, order])."""
    return quantize(np.ascontiguousarray(np.asarray(x)[:, np.asarray(order, np.int64)]), mode,
                    bf16_bits=bf16_bits)


def e4m3_round(q: float) -> int:
    """E4M3 byte (sign 0) nearest to q >= 0: ties to even, saturating at 448."""
    return int(_load().oracle_e4m3_round(float(q)))


def nvfp4_quantize(x: np.ndarray, tensor_scale: float, plus: bool, bf16_bits: bool = False):
    """NVFP4 / NVFP4+ (Sec. 8, "Applicability of MX+ to NVFP4"): blocks of 16, E4M3 block
    scale over the fp32 `tensor_scale`.  Returns (nibbles[rows, cols/2], scales[rows, cols/16],
    bm_index[rows, cols/32]: two 4-bit indices per byte, zero for plain NVFP4)."""
    assert x.ndim == 2
    x = np.ascontiguousarray(x)
    if bf16_bits:
        assert x.dtype == np.uint16
        kind = 1
    else:
        assert x.dtype == np.float32
        kind = 0
    rows, cols = x.shape
    if cols % 32:
        raise ValueError("cols must be a multiple of 32")
    nib = np.zeros((rows, cols // 2), np.uint8)
    sc = np.zeros((rows, cols // 16), np.uint8)
    idx = np.zeros((rows, cols // 32), np.uint8)
    rc = _load().oracle_nvfp4_quantize(_ptr(x), kind, rows, cols, float(tensor_scale), int(plus),
                                       _ptr(nib), _ptr(sc), _ptr(idx))
    if rc != 0:
        raise ValueError("oracle_nvfp4_quantize rejected its arguments")
    return nib, sc, idx


def nvfp4_dequantize(nib: np.ndarray, sc: np.ndarray, idx, tensor_scale: float, plus: bool) -> np.ndarray:
    """Decoded values as float64, exact (E * value(scale byte) * tensor_scale has at most 32
    significant bits); a consumer rounds once to its own output type."""
    nib = np.ascontiguousarray(nib, np.uint8)
    sc = np.ascontiguousarray(sc, np.uint8)
    rows, cols = nib.shape[0], nib.shape[1] * 2
    idx = np.zeros((rows, cols // 32), np.uint8) if idx is None else np.ascontiguousarray(idx, np.uint8)
    out = np.zeros((rows, cols), np.float64)
    rc = _load().oracle_nvfp4_dequantize(_ptr(nib), _ptr(sc), _ptr(idx), rows, cols,
                                         float(tensor_scale), int(plus), _ptr(out))
    if rc != 0:
        raise ValueError("oracle_nvfp4_dequantize rejected its arguments")
    return out
