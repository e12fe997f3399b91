"""Pins for the oracle's fp64 GEMM of decoded operands (no GPU)."""
import numpy as np

import oracle
from oracle import MODE_MXFP4 as MX, MODE_MXFP4_PLUS as MXP
from paper_2510_14557_b200 import synth


def test_single_block_by_hand():
    # A = [13 at k=8, 3 at k=2], B = [2 at k=8, -1 at k=2]: MX+ decodes 13 exactly -> 26 - 3
    a = np.zeros((1, 32), np.float32)
    b = np.zeros((1, 32), np.float32)
    a[0, 8], a[0, 2] = 13.0, 3.0
    b[0, 8], b[0, 2] = 2.0, -1.0
    da = oracle.dequantize(*oracle.quantize(a, MXP), MXP)
    db = oracle.dequantize(*oracle.quantize(b, MXP), MXP)
    assert oracle.gemm_fp64(da, db)[0, 0] == 13.0 * 2.0 - 3.0
    da4 = oracle.dequantize(*oracle.quantize(a, MX), MX)  # MXFP4 sees 12 instead of 13
    assert oracle.gemm_fp64(da4, db)[0, 0] == 12.0 * 2.0 - 3.0


def test_one_hot_b_returns_decoded_a():
    a, _ = synth.config1()
    qa = oracle.quantize(a, MXP)
    da = oracle.dequantize(*qa, MXP)
    k = a.shape[1]
    b = np.eye(k, dtype=np.float32)  # row n of B (N x K) is 1.0 at k = n
    qb = oracle.quantize(b, MXP)
    db = oracle.dequantize(*qb, MXP)
    assert np.array_equal(db, b.astype(np.float64))  # 1.0 is an exactly representable BM
    d = oracle.gemm_fp64(da, db)
    assert np.array_equal(d, da)


def test_matches_library_matmul_on_decoded_operands():
    a, b = synth.config1()
    for mode in (MX, MXP):
        da = oracle.dequantize(*oracle.quantize(a, mode), mode)
        db = oracle.dequantize(*oracle.quantize(b, mode), mode)
        d = oracle.gemm_fp64(da, db)
        ref = da @ db.T
        scale = np.linalg.norm(da, axis=1)[:, None] * np.linalg.norm(db, axis=1)[None, :]
        assert np.max(np.abs(d - ref) / scale) < 1e-14
    # orientation: B is N x K (not symmetric shapes)
    da = np.arange(6, dtype=np.float64).reshape(2, 3)
    db = np.arange(12, dtype=np.float64).reshape(4, 3) - 5
    assert np.array_equal(oracle.gemm_fp64(da, db), da @ db.T)


def test_missing_bm_residual_exceeds_the_parity_bound():
    # the tolerance used for GPU parity (1e-3 * |a_m| * |b_n|) must be able to see a
    # dropped BM correction: compare MX+ and MXFP4 decodes of the same activations
    a, b = synth.config1()
    dap = oracle.dequantize(*oracle.quantize(a, MXP), MXP)
    dam = oracle.dequantize(*oracle.quantize(a, MX), MX)
    db = oracle.dequantize(*oracle.quantize(b, MXP), MXP)
    dp, dm = oracle.gemm_fp64(dap, db), oracle.gemm_fp64(dam, db)
    scale = np.linalg.norm(dap, axis=1)[:, None] * np.linalg.norm(db, axis=1)[None, :]
    assert np.max(np.abs(dp - dm) / scale) > 1e-2
