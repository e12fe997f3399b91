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


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float64 -> nearest bfloat16 bit patterns, ONE rounding (ties to even), subnormals kept."""
    x = np.asarray(x, np.float64)
    mag = np.abs(x)
    _, ex = np.frexp(mag)                                  # mag = f * 2^ex, f in [0.5, 1)
    q = np.maximum(ex - 8, -133).astype(np.int64)          # quantum: 8 significant bits; 2^-133 below 2^-126
    r = np.ldexp(np.rint(np.ldexp(mag, -q)), q)            # rint: ties to even; both ldexp exact
    bits = r.astype(np.float32).view(np.uint32) >> 16      # exact: r is a bfloat16 value
    return (bits | (np.signbit(x).astype(np.uint32) << 15)).astype(np.uint16)


def nvfp4_boundary_blocks(ts, seed):
    """Blocks of 16 whose elements sit exactly on, one binary32 step above and one step below
    a rounding boundary of the element cast, the BM cast or the scale cast, for scales of every
    mantissa -- the inputs on which a reciprocal-and-multiply recipe and the definition part."""
    g = synth.rng(seed)
    ts32 = np.float32(ts)
    rows = []
    for _ in range(160):
        sb = int(g.integers(3, 0x7E))
        d = np.float64(oracle.elem_value(oracle.FMT_E4M3, sb)) * np.float64(ts32)
        blk = np.empty(16, np.float64)
        blk[0] = d * g.choice([5.5, 5.75, 6.0, 6.25, 5.25, 6.75, 5.9])          # the BM
        # the boundaries, and other values with few significant bits that are none
        ties = g.choice([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0,
                         0.375, 0.875, 0.4375, 0.3125, 0.625, 1.0, 3.0, 0.1875], 15)
        blk[1:] = ties * d * g.choice([-1.0, 1.0], 15)
        b32 = blk.astype(np.float32)
        step = g.integers(-1, 2, 16).astype(np.int32)                          # -1, 0, +1 ulp
        b32 = (b32.view(np.int32) + step).view(np.float32)
        rows.append(np.roll(b32, int(g.integers(0, 16))))
    # scale-cast boundaries: amax = 6 ts * (midpoint of two neighbouring oracle.FMT_E4M3 values) +- 1 ulp
    for sb in list(range(0, 0x7D, 3)):
        mid = 0.5 * (oracle.elem_value(oracle.FMT_E4M3, sb) + oracle.elem_value(oracle.FMT_E4M3, sb + 1))
        for step in (-1, 0, 1):
            a = np.float32(np.float64(6.0) * mid * np.float64(ts32))
            a = (a.view(np.int32) + np.int32(step)).view(np.float32)
            blk = np.full(16, a * np.float32(0.3), np.float32)
            blk[int(g.integers(0, 16))] = -a
            rows.append(blk)
    x = np.stack(rows)
    x = np.concatenate([x, np.zeros(((-x.shape[0]) % 2, 16), np.float32)])
    return x.reshape(-1, 32)
