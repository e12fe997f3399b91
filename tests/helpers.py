"""Shared helpers of the GPU parity tests (marshalling only; no method arithmetic)."""
import numpy as np
import torch

import oracle
from paper_2510_14557_b200 import synth


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)


def to_dev(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def packed_to_host(p):
    idx = p.bm_index.cpu().numpy() if p.bm_index is not None else None
    return p.nibbles.cpu().numpy(), p.scales.cpu().numpy(), idx


def host_to_packed(nib, sc, idx, mode):
    from paper_2510_14557_b200 import Packed
    rows, half = nib.shape
    return Packed(to_dev(nib), to_dev(sc), to_dev(idx) if idx is not None else None, rows, half * 2, mode)


def bf16_round(x: np.ndarray) -> np.ndarray:
    """float64 -> nearest bfloat16 (ties to even), returned as float64."""
    f = x.astype(np.float32)
    return synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(f)).astype(np.float64)


def gemm_bound(da: np.ndarray, db: np.ndarray) -> np.ndarray:
    """Per-entry tolerance 1e-3 * |a_m| * |b_n| on the decoded operands."""
    return 1e-3 * np.linalg.norm(da, axis=1)[:, None] * np.linalg.norm(db, axis=1)[None, :]


def check_gemm(d_gpu: torch.Tensor, da: np.ndarray, db: np.ndarray, ref: np.ndarray = None):
    """Compares a GPU result with the oracle's fp64 product of the decoded operands."""
    if ref is None:
        ref = oracle.gemm_fp64(da, db)
    tol = gemm_bound(da, db)
    got = d_gpu.float().cpu().numpy().astype(np.float64)
    if d_gpu.dtype == torch.bfloat16:
        # the output rounding itself may move the value by up to one bf16 ulp of the result
        tol = tol + np.abs(ref) * 2.0 ** -8
    err = np.abs(got - ref)
    bad = err > tol + 1e-300
    assert not bad.any(), "max err/tol = %g at %s" % (
        np.max(err / (tol + 1e-300)), np.unravel_index(np.argmax(err / (tol + 1e-300)), err.shape))
    return float(np.max(err / (tol + 1e-300)))
