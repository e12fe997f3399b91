"""No GEMM kernel writes outside its M x N output.

D is a view into a larger buffer filled with a NaN bit pattern: ldd > N (padding columns after
every row) and rows before and after the M the call is given.  Ragged M and N drive the
partial-tile paths of every kernel family -- the streamed CTA-pair kernel, the in-place
Eq. 4 kernels, the weight-only decode kernels and the weight-only tensor-core path -- and
afterwards every sentinel must still hold its pattern while the inside matches the oracle."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_gemm, host_to_packed, to_dev_bf16
from paper_2510_14557_b200 import synth

pytestmark = pytest.mark.gpu
MX, MXP, MXPP = 0, 1, 2
PAD_ROWS, PAD_COLS = 3, 40
SENTINEL = {torch.float32: 0x7FC5A5A5, torch.bfloat16: 0x7FC5}


def mxp():
    import paper_2510_14557_b200 as m
    return m


def guarded(M, N, dt):
    """(whole buffer as integers, D view of M x N inside it)."""
    it = torch.int32 if dt == torch.float32 else torch.int16
    buf = torch.full((M + 2 * PAD_ROWS, N + PAD_COLS), SENTINEL[dt], dtype=it, device="cuda")
    return buf, buf.view(dt)[PAD_ROWS:PAD_ROWS + M, :N]


def sentinels_intact(buf, M, N, dt):
    want = SENTINEL[dt]
    b = buf.cpu().numpy()
    ok = (b[:PAD_ROWS] == want).all() and (b[PAD_ROWS + M:] == want).all() and (b[:, N:] == want).all()
    inside = b[PAD_ROWS:PAD_ROWS + M, :N]
    return bool(ok), int((inside == want).sum())


def raw(rows, K, mode, seed):
    g = synth.rng(seed)
    nib = g.integers(0, 256, (rows, K // 2), dtype=np.uint8)
    sc = g.integers(122, 132, (rows, K // 32), dtype=np.uint8)
    idx = None if mode == MX else g.integers(0, 32 if mode == MXP else 256, (rows, K // 32), dtype=np.uint8)
    return host_to_packed(nib, sc, idx, mode), oracle.dequantize(nib, sc, idx, mode)


@pytest.mark.parametrize("small_workspace", [False, True])
@pytest.mark.parametrize("amode,bmode", [(MX, MX), (MXP, MX), (MX, MXP), (MXP, MXP)])
@pytest.mark.parametrize("M,N,K", [(257, 481, 256), (300, 250, 128), (129, 959, 384), (513, 130, 128),
                                   (100, 300, 256), (131, 77, 128)])
def test_packed_gemm_leaves_sentinels(M, N, K, amode, bmode, small_workspace):
    m = mxp()
    ap, da = raw(M, K, amode, M + K)
    bp, db = raw(N, K, bmode, N + K + 1)
    need = (m.mxp_gemm_min_workspace_bytes if small_workspace else m.mxp_gemm_workspace_bytes)(
        M, N, K, False, amode, bmode)
    ws = torch.zeros(max(need, 256), dtype=torch.uint8, device="cuda")[:max(need, 16)]
    for dt in (torch.float32, torch.bfloat16):
        buf, d = guarded(M, N, dt)
        m.mxp_gemm(ap, bp, out=d, workspace=ws)
        assert m.mxp_gemm_status(ws) == 0
        ok, untouched = sentinels_intact(buf, M, N, dt)
        assert ok, "a kernel wrote outside D"
        assert untouched == 0, "%d outputs never written" % untouched
        check_gemm(d.contiguous(), da, db)


@pytest.mark.parametrize("wmode", [MX, MXP, MXPP])
@pytest.mark.parametrize("M,N,K", [(1, 48, 256), (3, 2384, 512), (16, 304, 1024), (5, 77, 96), (16, 33, 32),
                                   (40, 64, 768), (64, 1000, 256), (65, 300, 256), (200, 481, 384)])
def test_weight_only_gemm_leaves_sentinels(M, N, K, wmode):
    # M <= 64: the streamed decode kernel (N % 16 == 0, K % 256 == 0) or the general one;
    # M > 64 with the full workspace: the tensor-core path
    m = mxp()
    a_bits, _ = synth.config3(M, 32, K, seed=M + N)
    bp, db = raw(N, K, wmode, N + K + 2)
    da = oracle.bf16_bits_to_f64(a_bits)
    need = m.mxp_gemm_workspace_bytes(M, N, K, True, MX, wmode)
    ws = torch.zeros(max(need, 256), dtype=torch.uint8, device="cuda")
    for dt in (torch.float32, torch.bfloat16):
        buf, d = guarded(M, N, dt)
        m.mxp_gemm(to_dev_bf16(a_bits), bp, out=d, workspace=ws)
        torch.cuda.synchronize()
        ok, untouched = sentinels_intact(buf, M, N, dt)
        assert ok, "a kernel wrote outside D"
        assert untouched == 0, "%d outputs never written" % untouched
        check_gemm(d.contiguous(), da, db)


def test_prepacked_and_ready_paths_leave_sentinels():
    # the benchmark's step on a ragged shape: fused quantizer, weights prepacked once
    m = mxp()
    M, N, K = 300, 730, 512
    a_bits, w_bits = synth.config3(M, N, K, seed=3)
    pw = m.mxp_quantize(to_dev_bf16(w_bits), MXP)
    pre = m.mxp_gemm_prepack(pw, True)
    ws = torch.zeros(m.mxp_gemm_workspace_bytes(M, N, K, False, MXP, MXP), dtype=torch.uint8, device="cuda")
    pa = m.mxp_quantize_gemm_ready(to_dev_bf16(a_bits), MXP, ws)
    qa = oracle.quantize(a_bits, MXP, bf16_bits=True)
    qw = oracle.quantize(w_bits, MXP, bf16_bits=True)
    da, dw = oracle.dequantize(*qa, MXP), oracle.dequantize(*qw, MXP)
    for dt in (torch.float32, torch.bfloat16):
        buf, d = guarded(M, N, dt)
        m.mxp_gemm_ready(pa, pw, pre, ws, out=d)
        assert m.mxp_gemm_status(ws) == 0
        ok, untouched = sentinels_intact(buf, M, N, dt)
        assert ok and untouched == 0
        check_gemm(d.contiguous(), da, dw)
        buf, d = guarded(M, N, dt)
        m.mxp_gemm_prepacked(pa, pw, pre, out=d, workspace=ws)
        ok, untouched = sentinels_intact(buf, M, N, dt)
        assert ok and untouched == 0
