"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times,
whole-matrix encodings bit for bit and sampled GEMM outputs the oracle computes one by one
(configs 2, 4 and 5; config 3 is covered in test_gpu_gemm.py)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_gemm, to_dev_bf16
from paper_2510_14557_b200 import synth

pytestmark = pytest.mark.gpu
MX, MXP, MXPP = 0, 1, 2


def mxp():
    import paper_2510_14557_b200 as m
    return m


def sample(n, step, extra):
    return np.unique(np.concatenate([np.arange(0, n, step), np.asarray(extra)]))


def planes_equal(p, ref, with_index):
    """Whole planes, bit for bit (compared on the host in one piece)."""
    assert np.array_equal(p.nibbles.cpu().numpy(), ref[0]), "codes differ"
    assert np.array_equal(p.scales.cpu().numpy(), ref[1]), "scales differ"
    if with_index:
        assert np.array_equal(p.bm_index.cpu().numpy(), ref[2]), "BM indices differ"


@pytest.fixture
def oracle_all_cores():
    oracle.set_threads(oracle.max_threads())
    yield
    oracle.set_threads(1)


@pytest.mark.parametrize("mode", [MX, MXP, MXPP])
def test_quantize_config2_whole_matrix_bit_exact(mode, oracle_all_cores):
    # 8192 x 8192 bf16 through the one-lane-per-block kernel: every byte of every plane, and
    # the decode of the whole matrix (exact in fp32), 1024 rows at a time
    bits = synth.config2()
    p = mxp().mxp_quantize(to_dev_bf16(bits), mode)
    ref = oracle.quantize(bits, mode, bf16_bits=True)
    planes_equal(p, ref, mode != MX)
    d = mxp().mxp_dequantize(p, torch.float32)
    for r0 in range(0, 8192, 1024):
        r1 = r0 + 1024
        want = oracle.dequantize(ref[0][r0:r1], ref[1][r0:r1], ref[2][r0:r1], mode)
        assert np.array_equal(d[r0:r1].cpu().numpy().astype(np.float64), want)


def _bench_step_parity(a_bits, w_bits, row_step, col_step):
    """The benchmark's step: weights quantized and prepacked once; activations through the fused
    quantizer (packed planes + GEMM-ready planes), then the GEMM on the prepared operands."""
    m = mxp()
    M, K = a_bits.shape
    N = w_bits.shape[0]
    w = to_dev_bf16(w_bits)
    pw = m.mxp_quantize(w, MXP)
    pre = m.mxp_gemm_prepack(pw, True)
    del w
    ws = torch.zeros(max(4096, m.mxp_gemm_workspace_bytes(M, N, K, False, MXP, MXP)),
                     dtype=torch.uint8, device="cuda")
    a = to_dev_bf16(a_bits)
    pa = m.mxp_quantize_gemm_ready(a, MXP, ws)
    d = m.mxp_gemm_ready(pa, pw, pre, ws, out_dtype=torch.bfloat16)
    torch.cuda.synchronize()
    assert m.mxp_gemm_status(ws) == 0
    # the encodings the GEMM consumed are the oracle's, bit for bit, over the whole of A and W
    oracle.set_threads(oracle.max_threads())
    try:
        planes_equal(pa, oracle.quantize(a_bits, MXP, bf16_bits=True), True)
        planes_equal(pw, oracle.quantize(w_bits, MXP, bf16_bits=True), True)
    finally:
        oracle.set_threads(1)
    # the output on sampled rows and columns (the fp64 product is O(M N K))
    rows = sample(M, row_step, [M - 1, M - 2, 255, 256, 257])
    cols = sample(N, col_step, [N - 1, N - 2, 239, 240, 479, 480, 481])
    qa = oracle.quantize(a_bits[rows], MXP, bf16_bits=True)
    qw = oracle.quantize(w_bits[cols], MXP, bf16_bits=True)
    rsel, csel = torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()
    da = oracle.dequantize(qa[0], qa[1], qa[2], MXP)
    dw = oracle.dequantize(qw[0], qw[1], qw[2], MXP)
    check_gemm(d[rsel][:, csel], da, dw)
    # the same operands through plain mxp_gemm (prepack inside the call): identical output
    d2 = m.mxp_gemm(pa, pw, out_dtype=torch.bfloat16, workspace=ws)
    assert torch.equal(d2[rsel][:, csel], d[rsel][:, csel])


def test_prefill_config4_bench_step_sampled():
    a_bits, w_bits = synth.config4()
    _bench_step_parity(a_bits, w_bits, row_step=97, col_step=61)


def test_prefill_config5_bench_step_sampled():
    # the headline workload: 8192 x 8192 activations, 28672 x 8192 weights
    a_bits, w_bits = synth.config5()
    _bench_step_parity(a_bits, w_bits, row_step=409, col_step=449)


def test_weight_only_4096_cubed_sampled():
    # the largest shape of the paper's matmul table (M = N = K = 4096), weight-only form: the
    # tensor-core path as mxp_gemm takes it and with the weights prepacked once
    m = mxp()
    M = N = K = 4096
    a_bits, w_bits = synth.config3(M, N, K, seed=7)
    pw = m.mxp_quantize(to_dev_bf16(w_bits), MXP)
    a = to_dev_bf16(a_bits)
    ws = torch.zeros(m.mxp_gemm_workspace_bytes(M, N, K, True, 0, MXP), dtype=torch.uint8, device="cuda")
    d = m.mxp_gemm(a, pw, out_dtype=torch.bfloat16, workspace=ws)
    assert m.mxp_gemm_status(ws) == 0
    d2 = m.mxp_gemm_dense_prepacked(a, pw, m.mxp_gemm_prepack(pw, True), out_dtype=torch.bfloat16)
    rows = sample(M, 211, [M - 1, 255, 256])
    cols = sample(N, 173, [N - 1, 239, 240, 479, 480])
    qw = oracle.quantize(w_bits[cols], MXP, bf16_bits=True)
    dw = oracle.dequantize(qw[0], qw[1], qw[2], MXP)
    da = oracle.bf16_bits_to_f64(a_bits[rows])
    rsel, csel = torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()
    check_gemm(d[rsel][:, csel], da, dw)
    assert torch.equal(d, d2)
