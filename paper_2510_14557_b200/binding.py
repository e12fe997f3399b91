"""ctypes binding of libmxp.so: argument marshalling only.

Every function takes torch CUDA tensors (device memory owned by the caller), passes their
data pointers and the current CUDA stream through the C ABI declared in ``include/mxp.h``
and raises ``MxpError`` on a non-zero status.  There is no fallback: if the shared
library is missing or cannot be loaded, importing a symbol from here raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

MXP_OK = 0
MODE_MXFP4 = 0
MODE_MXFP4_PLUS = 1
MODE_MXFP4_PP = 2
MODE_MXFP6, MODE_MXFP6_PLUS, MODE_MXFP8, MODE_MXFP8_PLUS = 3, 4, 5, 6  # quantize / dequantize only
F32 = 0
BF16 = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmxp.so")

EXPORTS = ["mxp_quantize", "mxp_quantize_reordered", "mxp_channel_order", "mxp_nvfp4_quantize", "mxp_nvfp4_dequantize", "mxp_dequantize", "mxp_gemm", "mxp_gemm_noalloc", "mxp_gemm_decode_chained", "mxp_gemm_decode_prepack_bytes", "mxp_gemm_decode_workspace_bytes", "mxp_gemm_decode_prepack", "mxp_gemm_decode_prepacked", "mxp_gemm_decode_prepacked_next", "mxp_gemm_workspace_bytes", "mxp_gemm_min_workspace_bytes",
           "mxp_gemm_prepack_bytes", "mxp_gemm_prepack_form", "mxp_gemm_prepack", "mxp_gemm_prepacked",
           "mxp_gemm_dense_prepacked", "mxp_gemm_dense_prepacked_workspace_bytes",
           "mxp_quantize_gemm_ready", "mxp_gemm_ready",
           "mxp_debug_override", "mxp_gemm_status", "mxp_gemm_clock_stamp", "mxp_wait_selftest", "mxp_tensor_peak_probe", "mxp_status_string", "mxp_version"]


class MxpError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__("%s failed: %s (status %d)" % (fn, status_string(status), status))


class _Packed(ctypes.Structure):
    _fields_ = [("nibbles", ctypes.c_void_p), ("scales", ctypes.c_void_p),
                ("bm_index", ctypes.c_void_p), ("rows", ctypes.c_int64),
                ("cols", ctypes.c_int64), ("mode", ctypes.c_int)]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libmxp.so (built in-tree by ``build.py``); raises if it is not there."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libmxp.so is not built: run `python -m paper_2510_14557_b200.build`")
        l = ctypes.CDLL(LIB_PATH)
        i64, vp, ci, sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        l.mxp_quantize.argtypes = [vp, ci, i64, i64, i64, ci, vp, vp, vp, vp]
        l.mxp_quantize.restype = ci
        l.mxp_dequantize.argtypes = [ctypes.POINTER(_Packed), vp, ci, i64, vp]
        l.mxp_dequantize.restype = ci
        l.mxp_gemm.argtypes = [i64, i64, i64, vp, i64, ctypes.POINTER(_Packed),
                               ctypes.POINTER(_Packed), vp, ci, i64, vp, sz, vp]
        l.mxp_gemm.restype = ci
        l.mxp_gemm_noalloc.argtypes = [i64, i64, i64, ctypes.POINTER(_Packed), ctypes.POINTER(_Packed),
                                       vp, ci, i64, ctypes.POINTER(ci), vp]
        l.mxp_gemm_noalloc.restype = ci
        l.mxp_gemm_dense_prepacked_workspace_bytes.argtypes = [i64, i64]
        l.mxp_gemm_dense_prepacked_workspace_bytes.restype = sz
        l.mxp_gemm_dense_prepacked.argtypes = [i64, i64, i64, vp, i64, ctypes.POINTER(_Packed), vp, sz, vp, ci,
                                               i64, vp, sz, vp]
        l.mxp_gemm_dense_prepacked.restype = ci
        l.mxp_quantize_reordered.argtypes = [vp, ci, i64, i64, i64, vp, ci, vp, vp, vp, vp]
        l.mxp_quantize_reordered.restype = ci
        l.mxp_nvfp4_quantize.argtypes = [vp, ci, i64, i64, i64, ctypes.c_float, ci, vp, vp, vp, vp]
        l.mxp_nvfp4_quantize.restype = ci
        l.mxp_nvfp4_dequantize.argtypes = [vp, vp, vp, i64, i64, ctypes.c_float, ci, vp, ci, i64, vp]
        l.mxp_nvfp4_dequantize.restype = ci
        l.mxp_channel_order.argtypes = [vp, i64, vp]
        l.mxp_channel_order.restype = ci
        l.mxp_gemm_decode_chained.argtypes = [i64, i64, i64, vp, i64, ctypes.POINTER(_Packed), vp, ci,
                                              i64, vp, vp]
        l.mxp_gemm_decode_chained.restype = ci
        l.mxp_gemm_decode_prepack_bytes.argtypes = [i64, i64, ci]
        l.mxp_gemm_decode_prepack_bytes.restype = sz
        l.mxp_gemm_decode_workspace_bytes.argtypes = [i64, i64]
        l.mxp_gemm_decode_workspace_bytes.restype = sz
        l.mxp_gemm_decode_prepack.argtypes = [ctypes.POINTER(_Packed), vp, sz, vp]
        l.mxp_gemm_decode_prepack.restype = ci
        l.mxp_gemm_decode_prepacked.argtypes = [i64, i64, i64, vp, i64, ci, vp, sz, vp, ci, i64, vp, sz, ci, vp]
        l.mxp_gemm_decode_prepacked.restype = ci
        l.mxp_gemm_decode_prepacked_next.argtypes = [i64, i64, i64, vp, i64, ci, vp, sz, vp, ci, i64, vp, sz, ci, vp, sz, vp]
        l.mxp_gemm_decode_prepacked_next.restype = ci
        l.mxp_gemm_workspace_bytes.argtypes = [i64, i64, i64, ci, ci, ci]
        l.mxp_gemm_workspace_bytes.restype = sz
        l.mxp_gemm_min_workspace_bytes.argtypes = [i64, i64, i64, ci, ci, ci]
        l.mxp_gemm_min_workspace_bytes.restype = sz
        l.mxp_gemm_prepack_bytes.argtypes = [i64, i64, ci]
        l.mxp_gemm_prepack_bytes.restype = sz
        l.mxp_gemm_prepack.argtypes = [ctypes.POINTER(_Packed), ci, vp, sz, vp]
        l.mxp_gemm_prepack.restype = ci
        l.mxp_gemm_prepack_form.argtypes = [ci, ci]
        l.mxp_gemm_prepack_form.restype = ci
        l.mxp_gemm_prepacked.argtypes = [i64, i64, i64, ctypes.POINTER(_Packed), ctypes.POINTER(_Packed),
                                         vp, sz, vp, ci, i64, vp, sz, vp]
        l.mxp_gemm_prepacked.restype = ci
        l.mxp_gemm_ready.argtypes = l.mxp_gemm_prepacked.argtypes
        l.mxp_gemm_ready.restype = ci
        l.mxp_quantize_gemm_ready.argtypes = [vp, ci, i64, i64, i64, ci, ci, vp, vp, vp, vp, sz, vp]
        l.mxp_quantize_gemm_ready.restype = ci
        l.mxp_debug_override.argtypes = [ci, ci]
        l.mxp_debug_override.restype = ci
        l.mxp_wait_selftest.argtypes = [vp, sz, i64, vp]
        l.mxp_wait_selftest.restype = ci
        l.mxp_gemm_status.argtypes = [vp, vp]
        l.mxp_gemm_status.restype = ci
        l.mxp_gemm_clock_stamp.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint64)]
        l.mxp_gemm_clock_stamp.restype = ci
        l.mxp_tensor_peak_probe.argtypes = [ci, ci, ctypes.POINTER(ctypes.c_double),
                                            ctypes.POINTER(ctypes.c_double)]
        l.mxp_tensor_peak_probe.restype = ci
        l.mxp_status_string.argtypes = [ci]
        l.mxp_status_string.restype = ctypes.c_char_p
        l.mxp_version.restype = ctypes.c_char_p
        _lib = l
    return _lib


def status_string(status: int) -> str:
    return lib().mxp_status_string(int(status)).decode()


def version() -> str:
    return lib().mxp_version().decode()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("expected float32 or bfloat16, got %s" % t.dtype)


def _check(fn: str, status: int) -> None:
    if status != MXP_OK:
        raise MxpError(fn, status)


@dataclass
class Packed:
    """An MXFP4 / MXFP4+ operand: three uint8 device planes (see include/mxp.h)."""
    nibbles: torch.Tensor        # [rows, cols/2]
    scales: torch.Tensor         # [rows, cols/32]
    bm_index: Optional[torch.Tensor]  # [rows, cols/32] or None (MXFP4)
    rows: int
    cols: int
    mode: int

    def c_struct(self) -> _Packed:
        return _Packed(self.nibbles.data_ptr(), self.scales.data_ptr(),
                       self.bm_index.data_ptr() if self.bm_index is not None else None,
                       self.rows, self.cols, self.mode)


def element_bits(mode: int) -> int:
    return 6 if mode in (MODE_MXFP6, MODE_MXFP6_PLUS) else 8 if mode in (MODE_MXFP8, MODE_MXFP8_PLUS) else 4


def alloc_packed(rows: int, cols: int, mode: int, device="cuda", index_for_mxfp4=False) -> Packed:
    nib = torch.empty((rows, cols * element_bits(mode) // 8), dtype=torch.uint8, device=device)
    sc = torch.empty((rows, cols // 32), dtype=torch.uint8, device=device)
    idx = None
    if mode not in (MODE_MXFP4, MODE_MXFP6, MODE_MXFP8) or index_for_mxfp4:
        idx = torch.empty((rows, cols // 32), dtype=torch.uint8, device=device)
    return Packed(nib, sc, idx, rows, cols, mode)


def mxp_quantize(src: torch.Tensor, mode: int, out: Optional[Packed] = None) -> Packed:
    """Quantizes a 2-D CUDA tensor (float32 / bfloat16, unit inner stride) along its rows."""
    assert src.is_cuda and src.dim() == 2 and src.stride(1) == 1
    rows, cols = src.shape
    if out is None:
        out = alloc_packed(rows, cols, mode, src.device)
    st = lib().mxp_quantize(src.data_ptr(), _dt(src), rows, cols, src.stride(0), mode,
                            out.nibbles.data_ptr(), out.scales.data_ptr(),
                            out.bm_index.data_ptr() if out.bm_index is not None else None,
                            _stream())
    _check("mxp_quantize", st)
    return out


def mxp_quantize_reordered(src: torch.Tensor, order: torch.Tensor, mode: int,
                           out: Optional[Packed] = None) -> Packed:
    """quantize(src[:, order]) in one pass: `order` is an int32 CUDA tensor of src.shape[1]
    entries (position c of the quantized rows takes source channel order[c])."""
    assert src.is_cuda and src.dim() == 2 and src.stride(1) == 1
    assert order.is_cuda and order.dtype == torch.int32 and order.is_contiguous()
    rows, cols = src.shape
    assert order.numel() == cols
    if out is None:
        out = alloc_packed(rows, cols, mode, src.device)
    st = lib().mxp_quantize_reordered(src.data_ptr(), _dt(src), rows, cols, src.stride(0),
                                      order.data_ptr(), mode, out.nibbles.data_ptr(),
                                      out.scales.data_ptr(),
                                      out.bm_index.data_ptr() if out.bm_index is not None else None,
                                      _stream())
    _check("mxp_quantize_reordered", st)
    return out


def mxp_nvfp4_quantize(src: torch.Tensor, tensor_scale: float, plus: bool):
    """NVFP4 / NVFP4+ of a 2-D CUDA tensor: returns (nibbles, scales, bm_index or None) as uint8
    tensors [rows, cols/2], [rows, cols/16], [rows, cols/32]."""
    assert src.is_cuda and src.dim() == 2 and src.stride(1) == 1
    rows, cols = src.shape
    nib = torch.empty((rows, cols // 2), dtype=torch.uint8, device=src.device)
    sc = torch.empty((rows, cols // 16), dtype=torch.uint8, device=src.device)
    idx = torch.empty((rows, cols // 32), dtype=torch.uint8, device=src.device) if plus else None
    st = lib().mxp_nvfp4_quantize(src.data_ptr(), _dt(src), rows, cols, src.stride(0),
                                  float(tensor_scale), int(plus), nib.data_ptr(), sc.data_ptr(),
                                  idx.data_ptr() if plus else None, _stream())
    _check("mxp_nvfp4_quantize", st)
    return nib, sc, idx


def mxp_nvfp4_dequantize(nib: torch.Tensor, sc: torch.Tensor, idx: Optional[torch.Tensor],
                         tensor_scale: float, plus: bool, dtype=torch.float32) -> torch.Tensor:
    rows, cols = nib.shape[0], nib.shape[1] * 2
    out = torch.empty((rows, cols), dtype=dtype, device=nib.device)
    st = lib().mxp_nvfp4_dequantize(nib.data_ptr(), sc.data_ptr(),
                                    idx.data_ptr() if idx is not None else None, rows, cols,
                                    float(tensor_scale), int(plus), out.data_ptr(), _dt(out),
                                    out.stride(0), _stream())
    _check("mxp_nvfp4_dequantize", st)
    return out


def mxp_channel_order(outlier_count) -> torch.Tensor:
    """Channel ordering (int32 CPU tensor) from per-channel outlier counts, by the paper's
    rule; see the header for the exact placement."""
    cnt = torch.as_tensor(outlier_count, dtype=torch.int64).contiguous().cpu()
    order = torch.empty(cnt.numel(), dtype=torch.int32)
    st = lib().mxp_channel_order(cnt.data_ptr(), cnt.numel(), order.data_ptr())
    _check("mxp_channel_order", st)
    return order


def mxp_dequantize(p: Packed, dtype=torch.float32, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    if out is None:
        out = torch.empty((p.rows, p.cols), dtype=dtype, device=p.nibbles.device)
    cs = p.c_struct()
    st = lib().mxp_dequantize(ctypes.byref(cs), out.data_ptr(), _dt(out), out.stride(0), _stream())
    _check("mxp_dequantize", st)
    return out


def mxp_gemm_workspace_bytes(M: int, N: int, K: int, a_dense: bool, a_mode: int, b_mode: int) -> int:
    return int(lib().mxp_gemm_workspace_bytes(M, N, K, int(a_dense), a_mode, b_mode))


def mxp_gemm_min_workspace_bytes(M: int, N: int, K: int, a_dense: bool, a_mode: int, b_mode: int) -> int:
    return int(lib().mxp_gemm_min_workspace_bytes(M, N, K, int(a_dense), a_mode, b_mode))


def mxp_gemm(a, b: Packed, out_dtype=torch.bfloat16, out: Optional[torch.Tensor] = None,
             workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """D = dec(A) @ dec(B).T.  `a` is a bf16 CUDA tensor (weight-only form) or a Packed."""
    N, K = b.rows, b.cols
    dense = isinstance(a, torch.Tensor)
    M = a.shape[0] if dense else a.rows
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=b.nibbles.device)
    a_mode = MODE_MXFP4 if dense else a.mode
    need = mxp_gemm_workspace_bytes(M, N, K, dense, a_mode, b.mode)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=b.nibbles.device)
    ws_ptr = workspace.data_ptr() if workspace is not None else None
    ws_len = workspace.numel() if workspace is not None else 0
    bs = b.c_struct()
    if dense:
        assert a.dtype == torch.bfloat16 and a.is_cuda and a.stride(1) == 1
        st = lib().mxp_gemm(M, N, K, a.data_ptr(), a.stride(0), None, ctypes.byref(bs),
                            out.data_ptr(), _dt(out), out.stride(0), ws_ptr, ws_len, _stream())
    else:
        as_ = a.c_struct()
        st = lib().mxp_gemm(M, N, K, None, 0, ctypes.byref(as_), ctypes.byref(bs),
                            out.data_ptr(), _dt(out), out.stride(0), ws_ptr, ws_len, _stream())
    _check("mxp_gemm", st)
    return out


PREPACK_PLAIN, PREPACK_WIDE, PREPACK_SPLIT, PREPACK_WIDE8, PREPACK_WIDE_X2, PREPACK_WIDE8_X3 = 0, 1, 2, 3, 4, 5


def mxp_gemm_prepack_form(a_mode: int, b_mode: int) -> int:
    """The form of B's prepacked copy that mxp_gemm_prepacked reads for these modes."""
    return int(lib().mxp_gemm_prepack_form(a_mode, b_mode))


def mxp_gemm_prepack(p: Packed, wide, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Prepacked copy of an operand (normally the weights) for mxp_gemm_prepacked.  `wide`: a
    PREPACK_* form (True: the operand's widened form, False: PREPACK_PLAIN); take it from
    mxp_gemm_prepack_form(a_mode, b_mode) of the GEMMs the copy is for."""
    if wide is True:  # the operand's own widened form: E4M3 bytes for MX++ and MXFP8, E2M3 codes otherwise
        wide = {2: PREPACK_WIDE8, 5: PREPACK_WIDE8, 4: PREPACK_WIDE_X2, 6: PREPACK_WIDE8_X3}.get(p.mode, PREPACK_WIDE)
    need = int(lib().mxp_gemm_prepack_bytes(p.rows, p.cols, int(wide)))
    if need == 0:
        raise MxpError("mxp_gemm_prepack_bytes", 2)
    if out is None:
        out = torch.empty(need, dtype=torch.uint8, device=p.nibbles.device)
    cs = p.c_struct()
    st = lib().mxp_gemm_prepack(ctypes.byref(cs), int(wide), out.data_ptr(), out.numel(), _stream())
    _check("mxp_gemm_prepack", st)
    return out


def mxp_gemm_prepacked(a: Packed, b: Packed, b_prepacked: torch.Tensor, out_dtype=torch.bfloat16,
                       out: Optional[torch.Tensor] = None,
                       workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """D = dec(A) @ dec(B).T with B's prepacked copy from mxp_gemm_prepack."""
    M, N, K = a.rows, b.rows, b.cols
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=b.nibbles.device)
    if workspace is None:
        workspace = torch.empty(mxp_gemm_workspace_bytes(M, N, K, False, a.mode, b.mode),
                                dtype=torch.uint8, device=b.nibbles.device)
    as_, bs = a.c_struct(), b.c_struct()
    st = lib().mxp_gemm_prepacked(M, N, K, ctypes.byref(as_), ctypes.byref(bs), b_prepacked.data_ptr(),
                                  b_prepacked.numel(), out.data_ptr(), _dt(out), out.stride(0), workspace.data_ptr(),
                                  workspace.numel(), _stream())
    _check("mxp_gemm_prepacked", st)
    return out


def mxp_quantize_gemm_ready(src: torch.Tensor, mode: int, workspace: torch.Tensor,
                            out: Optional[Packed] = None, b_mode: Optional[int] = None) -> Packed:
    """mxp_quantize that also writes A's GEMM-ready form into `workspace` (see include/mxp.h).
    `b_mode`: the mode of the operand it will be multiplied with (default: the same mode)."""
    assert src.is_cuda and src.dim() == 2 and src.stride(1) == 1
    rows, cols = src.shape
    if out is None:
        out = alloc_packed(rows, cols, mode, src.device)
    st = lib().mxp_quantize_gemm_ready(src.data_ptr(), _dt(src), rows, cols, src.stride(0), mode,
                                       mode if b_mode is None else b_mode,
                                       out.nibbles.data_ptr(), out.scales.data_ptr(),
                                       out.bm_index.data_ptr() if out.bm_index is not None else None,
                                       workspace.data_ptr(), workspace.numel(), _stream())
    _check("mxp_quantize_gemm_ready", st)
    return out


def mxp_gemm_ready(a: Packed, b: Packed, b_prepacked: torch.Tensor, workspace: torch.Tensor,
                   out_dtype=torch.bfloat16, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """D = dec(A) @ dec(B).T, A prepared in `workspace` by mxp_quantize_gemm_ready."""
    M, N, K = a.rows, b.rows, b.cols
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=b.nibbles.device)
    as_, bs = a.c_struct(), b.c_struct()
    st = lib().mxp_gemm_ready(M, N, K, ctypes.byref(as_), ctypes.byref(bs), b_prepacked.data_ptr(),
                              b_prepacked.numel(), out.data_ptr(), _dt(out), out.stride(0), workspace.data_ptr(),
                              workspace.numel(), _stream())
    _check("mxp_gemm_ready", st)
    return out


def mxp_gemm_noalloc(a: Packed, b: Packed, out: torch.Tensor, read_status: bool = False):
    """Packed-operand GEMM that allocates nothing: for callers that may not call cudaMalloc
    (code living inside another framework's memory pool, plugins loaded once the pool owns
    the device).  `out` must be preallocated by the caller; the kernel's scratch sits in a
    4 KB array inside the library.  Returns the kernel status when `read_status` is set
    (that synchronises the stream), else None."""
    ks = ctypes.c_int(0)
    as_, bs = a.c_struct(), b.c_struct()
    st = lib().mxp_gemm_noalloc(a.rows, b.rows, b.cols, ctypes.byref(as_), ctypes.byref(bs),
                                out.data_ptr(), _dt(out), out.stride(0),
                                ctypes.byref(ks) if read_status else None, _stream())
    _check("mxp_gemm_noalloc", st)
    return ks.value if read_status else None


def mxp_gemm_decode_chained(a: torch.Tensor, b: Packed, out: torch.Tensor,
                            status_block: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Weight-only GEMM launched as a programmatic dependent of the preceding kernel on the
    stream (a chain of decode GEMMs).  `b` must not be written by that preceding kernel; `a`
    and `out` are ordered as usual.  `status_block`: 16 zeroed bytes on the device, or None."""
    assert a.dtype == torch.bfloat16 and a.is_cuda and a.stride(1) == 1
    bs = b.c_struct()
    st = lib().mxp_gemm_decode_chained(a.shape[0], b.rows, b.cols, a.data_ptr(), a.stride(0),
                                       ctypes.byref(bs), out.data_ptr(), _dt(out), out.stride(0),
                                       status_block.data_ptr() if status_block is not None else None,
                                       _stream())
    _check("mxp_gemm_decode_chained", st)
    return out


class DecodeWeights:
    """Weights re-tiled once for mxp_gemm_decode_prepacked: the device buffer plus the shape and
    mode it was made from (what the C call wants to see again)."""

    def __init__(self, buf: torch.Tensor, rows: int, cols: int, mode: int):
        self.buf, self.rows, self.cols, self.mode = buf, rows, cols, mode


def mxp_gemm_decode_prepack(b: Packed) -> DecodeWeights:
    """Re-tiles MXFP4 / MXFP4+ weights for the decode GEMM (once per weight matrix and device)."""
    need = int(lib().mxp_gemm_decode_prepack_bytes(b.rows, b.cols, b.mode))
    if need == 0:
        raise MxpError("mxp_gemm_decode_prepack_bytes", 2)
    out = torch.empty(need, dtype=torch.uint8, device=b.nibbles.device)
    bs = b.c_struct()
    _check("mxp_gemm_decode_prepack", lib().mxp_gemm_decode_prepack(ctypes.byref(bs), out.data_ptr(), out.numel(), _stream()))
    return DecodeWeights(out, b.rows, b.cols, b.mode)


def mxp_gemm_decode_workspace_bytes(M: int, K: int) -> int:
    return int(lib().mxp_gemm_decode_workspace_bytes(M, K))


def mxp_gemm_decode_prepacked(a: torch.Tensor, w: DecodeWeights, out_dtype=torch.bfloat16,
                              out: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                              chained: bool = False, next_w: Optional[DecodeWeights] = None) -> torch.Tensor:
    """D = a @ dec(W).T for 1..16 activation rows on the FP4 tensor path, weights re-tiled by
    mxp_gemm_decode_prepack.  `chained`, `next_w` (the weights of the call expected next: a
    prefetch hint, mxp_gemm_decode_prepacked_next): see include/mxp.h."""
    assert a.dtype == torch.bfloat16 and a.is_cuda and a.stride(1) == 1
    M, N, K = a.shape[0], w.rows, w.cols
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=a.device)
    if workspace is None:
        workspace = torch.zeros(max(256, mxp_gemm_decode_workspace_bytes(M, K)), dtype=torch.uint8, device=a.device)
    if next_w is None:
        st = lib().mxp_gemm_decode_prepacked(M, N, K, a.data_ptr(), a.stride(0), w.mode, w.buf.data_ptr(),
                                             w.buf.numel(), out.data_ptr(), _dt(out), out.stride(0),
                                             workspace.data_ptr(), workspace.numel(), int(chained), _stream())
        _check("mxp_gemm_decode_prepacked", st)
    else:
        st = lib().mxp_gemm_decode_prepacked_next(M, N, K, a.data_ptr(), a.stride(0), w.mode, w.buf.data_ptr(),
                                                  w.buf.numel(), out.data_ptr(), _dt(out), out.stride(0),
                                                  workspace.data_ptr(), workspace.numel(), int(chained),
                                                  next_w.buf.data_ptr(), next_w.buf.numel(), _stream())
        _check("mxp_gemm_decode_prepacked_next", st)
    return out


def mxp_gemm_dense_prepacked(a: torch.Tensor, b: Packed, b_prepacked: torch.Tensor,
                             out_dtype=torch.bfloat16, out: Optional[torch.Tensor] = None,
                             workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Weight-only GEMM on the tensor-core kernel with B's prepacked copy
    (mxp_gemm_prepack(b, True)); `a` is a bf16 CUDA tensor with any number of rows."""
    assert a.dtype == torch.bfloat16 and a.is_cuda and a.stride(1) == 1
    M, N, K = a.shape[0], b.rows, b.cols
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=a.device)
    need = int(lib().mxp_gemm_dense_prepacked_workspace_bytes(M, K))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=a.device)
    bs = b.c_struct()
    st = lib().mxp_gemm_dense_prepacked(M, N, K, a.data_ptr(), a.stride(0), ctypes.byref(bs),
                                        b_prepacked.data_ptr(), b_prepacked.numel(), out.data_ptr(), _dt(out),
                                        out.stride(0), workspace.data_ptr(), workspace.numel(),
                                        _stream())
    _check("mxp_gemm_dense_prepacked", st)
    return out


KNOB_INPLACE_KERNEL, KNOB_STREAM_HALVES, KNOB_WEIGHT_ONLY_KERNEL, KNOB_ONE_SIDED = 0, 1, 2, 3


def mxp_debug_override(knob: int, value: int) -> None:
    """Forces a kernel choice (tests and measurements; see include/mxp.h).  0 = automatic."""
    _check("mxp_debug_override", lib().mxp_debug_override(knob, value))


def mxp_wait_selftest(workspace: torch.Tensor, limit_cycles: int) -> None:
    """Launches the bounded-wait self-test; read the outcome with mxp_gemm_status(workspace)."""
    _check("mxp_wait_selftest", lib().mxp_wait_selftest(workspace.data_ptr(), workspace.numel(),
                                                        int(limit_cycles), _stream()))


def mxp_gemm_status(workspace: torch.Tensor) -> int:
    return int(lib().mxp_gemm_status(workspace.data_ptr(), _stream()))


def mxp_gemm_clock_stamp(workspace: torch.Tensor):
    """(sm_cycles, nanoseconds) of the last streamed tensor-core GEMM that used `workspace`."""
    clk, ns = ctypes.c_uint64(), ctypes.c_uint64()
    st = lib().mxp_gemm_clock_stamp(workspace.data_ptr(), _stream(), ctypes.byref(clk), ctypes.byref(ns))
    _check("mxp_gemm_clock_stamp", st)
    return clk.value, ns.value


def mxp_tensor_peak_probe(kind: int, iters: int):
    ms, fl = ctypes.c_double(), ctypes.c_double()
    st = lib().mxp_tensor_peak_probe(kind, iters, ctypes.byref(ms), ctypes.byref(fl))
    _check("mxp_tensor_peak_probe", st)
    return ms.value, fl.value
