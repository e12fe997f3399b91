"""GPU parity of the one-sided MX+ GEMM: FP4 main pass on BM_H plus Eq. 4's BM_L residual as a
sparse tensor-core instruction (Sec. 5.1 Eq. 4, Sec. 5.2 Algorithm 1), in both directions --
MXFP4+ activations x MXFP4 weights, and MXFP4 activations x MXFP4+ weights (computed as
D^T = W A^T and stored transposed) -- against the oracle's fp64 product of the decoded operands."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_gemm, host_to_packed
from paper_2510_14557_b200 import synth

pytestmark = pytest.mark.gpu
MX, MXP = 0, 1
ONE_SIDED = [(MXP, MX), (MX, MXP)]


def mxp():
    import paper_2510_14557_b200 as m
    return m


@pytest.fixture
def knob():
    m = mxp()
    used = []

    def set_(k, v):
        used.append(k)
        m.mxp_debug_override(k, v)
    yield set_
    for k in used:
        m.mxp_debug_override(k, 0)


def raw(rows, K, mode, seed, lo=120, hi=134):
    """Planes filled directly: every code, BM position and BM mantissa occurs."""
    g = synth.rng(seed)
    nib = g.integers(0, 256, (rows, K // 2), dtype=np.uint8)
    sc = g.integers(lo, hi, (rows, K // 32), dtype=np.uint8)
    idx = g.integers(0, 32, (rows, K // 32), dtype=np.uint8) if mode == MXP else None
    return host_to_packed(nib, sc, idx, mode), oracle.dequantize(nib, sc, idx, mode)


def identity(K, mode):
    eye = np.eye(K, dtype=np.float32)
    q = oracle.quantize(eye, mode)
    assert np.array_equal(oracle.dequantize(q[0], q[1], q[2], mode), eye.astype(np.float64))
    return host_to_packed(q[0], q[1], q[2] if mode != MX else None, mode)


@pytest.mark.parametrize("halves", [0, 1, 2])
@pytest.mark.parametrize("K", [128, 256, 384, 1024])
def test_identity_partner_returns_the_decode_bit_for_bit(K, halves, knob):
    # the MX+ operand's planes are random bytes: every code, BM position (all 32: every group of
    # eight, every pair, both elements), sign and mantissa, so every metadata nibble and every
    # compressed slot the split writes is used; the partner is the identity, so each output is
    # one decoded element: BM_H from the main pass plus BM_L from the sparse pass, exactly.
    # K = 128 and 384 end in a stage with a single K group.
    m = mxp()
    if halves:
        knob(m.KNOB_STREAM_HALVES, halves)
    rows = 300
    # MXFP4+ activations (A slot as given) x identity weights
    ap, da = raw(rows, K, MXP, seed=K + 1)
    d = m.mxp_gemm(ap, identity(K, MX), out_dtype=torch.float32)
    assert np.array_equal(d.cpu().numpy().astype(np.float64), da)
    # identity activations x MXFP4+ weights: D = dec(W)^T through the transposed store
    wp, dw = raw(rows, K, MXP, seed=K + 2)
    d = m.mxp_gemm(identity(K, MX), wp, out_dtype=torch.float32)
    assert np.array_equal(d.cpu().numpy().astype(np.float64), dw.T)


def test_every_bm_position_and_mantissa_one_by_one():
    # block b of row r has its BM at position (r + b) % 32 with code r % 16 (sign and three
    # mantissa bits), all other codes zero: what comes out is BM_H + BM_L alone
    m = mxp()
    rows, K = 512, 256
    nib = np.zeros((rows, K // 2), np.uint8)
    idx = np.zeros((rows, K // 32), np.uint8)
    sc = np.full((rows, K // 32), 127, np.uint8)
    for r in range(rows):
        for b in range(K // 32):
            p = (r + b) % 32
            idx[r, b] = p
            nib[r, b * 16 + p // 2] = (r % 16) << (4 * (p % 2))
    dec = oracle.dequantize(nib, sc, idx, MXP)
    assert set(np.unique(np.abs(dec))) == {0.0, 4.0, 4.5, 5.0, 5.5, 6.0, 6.5, 7.0, 7.5}
    p = host_to_packed(nib, sc, idx, MXP)
    d = m.mxp_gemm(p, identity(K, MX), out_dtype=torch.float32)
    assert np.array_equal(d.cpu().numpy().astype(np.float64), dec)
    d = m.mxp_gemm(identity(K, MX), p, out_dtype=torch.float32)
    assert np.array_equal(d.cpu().numpy().astype(np.float64), dec.T)


@pytest.mark.parametrize("amode,bmode", ONE_SIDED)
@pytest.mark.parametrize("M,N,K", [(300, 520, 1024), (257, 129, 2176), (512, 512, 128), (129, 959, 384),
                                   (1000, 300, 256), (513, 481, 640)])
def test_parity_prepacked_and_widened_paths_agree(M, N, K, amode, bmode, knob):
    # ragged M and N on both sides of the tile shapes; the same call through mxp_gemm (operands
    # prepared inside), with the weights prepacked once, and on the single widened pass
    m = mxp()
    ap, da = raw(M, K, amode, seed=M + 1)
    bp, db = raw(N, K, bmode, seed=N + 2)
    ref = oracle.gemm_fp64(da, db)
    form = m.mxp_gemm_prepack_form(amode, bmode)
    assert form == (m.PREPACK_SPLIT if bmode == MXP else m.PREPACK_PLAIN)
    pre = m.mxp_gemm_prepack(bp, form)
    ws = torch.zeros(m.mxp_gemm_workspace_bytes(M, N, K, False, amode, bmode), dtype=torch.uint8, device="cuda")
    for dt in (torch.float32, torch.bfloat16):
        d0 = m.mxp_gemm(ap, bp, out_dtype=dt, workspace=ws)
        assert m.mxp_gemm_status(ws) == 0
        check_gemm(d0, da, db, ref)
        d1 = m.mxp_gemm_prepacked(ap, bp, pre, out_dtype=dt, workspace=ws)
        assert m.mxp_gemm_status(ws) == 0
        assert torch.equal(d0, d1)
    knob(m.KNOB_ONE_SIDED, 1)
    assert m.mxp_gemm_prepack_form(amode, bmode) == m.PREPACK_WIDE
    d2 = m.mxp_gemm(ap, bp, out_dtype=torch.float32, workspace=ws)
    check_gemm(d2, da, db, ref)
    with pytest.raises(m.MxpError):   # the copy made for the sparse path is not the one this path reads
        m.mxp_gemm_prepacked(ap, bp, pre, workspace=ws)


@pytest.mark.parametrize("amode,bmode", ONE_SIDED)
def test_quantized_operands_and_special_blocks(amode, bmode):
    # operands quantized by the library from the benchmark's distributions (outlier channels on
    # the activation side), plus flushed blocks (scale byte 0 with codes behind it: zeros), BMs
    # at the first and last position and blocks whose BM_L is zero
    m = mxp()
    M, N, K = 384, 640, 512
    a_bits, w_bits = synth.config3(M, N, K, seed=11)
    qa = list(oracle.quantize(a_bits, amode, bf16_bits=True))
    qw = list(oracle.quantize(w_bits, bmode, bf16_bits=True))
    x = qa if amode == MXP else qw
    x[1][::7, 1] = 0                       # flushed blocks, codes left in place
    x[2][::5, 2] = 0
    x[2][::3, 3] = 31
    x[0][::3, 3 * 16 + 15] &= 0x4F         # BM at position 31: mantissa bits m1 m0 cleared (BM_L = 0)
    da, dw = oracle.dequantize(qa[0], qa[1], qa[2], amode), oracle.dequantize(qw[0], qw[1], qw[2], bmode)
    ap = host_to_packed(qa[0], qa[1], qa[2] if amode == MXP else None, amode)
    wp = host_to_packed(qw[0], qw[1], qw[2] if bmode == MXP else None, bmode)
    for dt in (torch.float32, torch.bfloat16):
        check_gemm(m.mxp_gemm(ap, wp, out_dtype=dt), da, dw)


def test_integer_valued_operands_are_exact():
    # small integers times powers of two: every partial sum is exact in fp32, so the main pass,
    # the residual pass and the widened pass must all give the oracle's sum to the bit
    m = mxp()
    M, N, K = 256 + 64, 448 + 32, 512
    g = synth.rng(5)
    a = g.integers(-3, 4, (M, K)).astype(np.float32) * 2.0
    a[:, ::32] = g.choice([9.0, -11.0, 13.0, 15.0, -10.0], (M, K // 32))   # BMs with all three mantissa bits
    w = g.integers(-2, 3, (N, K)).astype(np.float32)
    w[:, 5::32] = g.choice([4.0, -6.0], (N, K // 32))
    for amode, bmode, aa, ww in ((MXP, MX, a, w), (MX, MXP, w[:M], np.resize(a, (N, K)))):
        qa, qw = oracle.quantize(aa, amode), oracle.quantize(ww, bmode)
        da, dw = oracle.dequantize(qa[0], qa[1], qa[2], amode), oracle.dequantize(qw[0], qw[1], qw[2], bmode)
        ap = host_to_packed(qa[0], qa[1], qa[2] if amode == MXP else None, amode)
        wp = host_to_packed(qw[0], qw[1], qw[2] if bmode == MXP else None, bmode)
        d = m.mxp_gemm(ap, wp, out_dtype=torch.float32)
        assert np.array_equal(d.cpu().numpy().astype(np.float64), oracle.gemm_fp64(da, dw))


@pytest.mark.parametrize("M,N,K", [(512, 640, 512), (300, 481, 1024), (129, 200, 256), (1000, 300, 768)])
def test_quantizer_emits_the_split_form_for_the_gemm(M, N, K):
    # the paper's main scenario as two launches: activations quantized to MXFP4+ and split per
    # Eq. 4 by the same kernel, straight into the GEMM's workspace, then the sparse-residual GEMM
    # against MXFP4 weights prepared once.  Same packed planes as mxp_quantize (bit-exact against
    # the oracle), same product as mxp_gemm on those planes (bit-identical: same kernel, same
    # operands).  M not a multiple of 256: the last row groups' metadata is filled for rows the
    # activations do not have.
    from helpers import packed_to_host, to_dev_bf16
    m = mxp()
    a_bits, w_bits = synth.config3(M, N, K, seed=M + K)
    a = to_dev_bf16(a_bits)
    pw = m.mxp_quantize(to_dev_bf16(w_bits), MX)
    pre = m.mxp_gemm_prepack(pw, m.mxp_gemm_prepack_form(MXP, MX))
    ws = torch.full((m.mxp_gemm_workspace_bytes(M, N, K, False, MXP, MX),), 0xEE, dtype=torch.uint8, device="cuda")
    pa = m.mxp_quantize_gemm_ready(a, MXP, ws, b_mode=MX)
    qa = oracle.quantize(a_bits, MXP, bf16_bits=True)
    for got, want in zip(packed_to_host(pa), qa):
        assert np.array_equal(got, want)
    ws2 = torch.zeros_like(ws)
    for dt in (torch.float32, torch.bfloat16):
        d = m.mxp_gemm_ready(pa, pw, pre, ws, out_dtype=dt)
        assert m.mxp_gemm_status(ws) == 0
        assert torch.equal(d, m.mxp_gemm(pa, pw, out_dtype=dt, workspace=ws2))
    qw = oracle.quantize(w_bits, MX, bf16_bits=True)
    check_gemm(d, oracle.dequantize(qa[0], qa[1], qa[2], MXP), oracle.dequantize(qw[0], qw[1], qw[2], MX))
    # K with half a stage at its end is not taken by the fused form
    if K == 768:
        with pytest.raises(m.MxpError):
            m.mxp_quantize_gemm_ready(a[:, :640].contiguous(), MXP, ws, b_mode=MX)
