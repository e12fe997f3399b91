"""GPU parity of the streamed tensor-core GEMM at the wider element formats (MXFP6 / MXFP6+ /
MXFP8 / MXFP8+ operands: Table of MX formats, Sec. 4.1-4.2), of the quantizer that writes the
GEMM-ready form (Sec. 5: quantization right before the matrix multiply), of MX++ weights in the
weight-only kernels (Sec. 4.3), and of the bounded device-side waits."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_gemm, host_to_packed, to_dev, to_dev_bf16
from paper_2510_14557_b200 import synth

pytestmark = pytest.mark.gpu
MX, MXP, MXPP = 0, 1, 2


def mxp():
    import paper_2510_14557_b200 as m
    return m


@pytest.fixture
def force():
    """Forces a kernel choice for the duration of a test (mxp_debug_override)."""
    m = mxp()
    knobs = {"weight_only": m.KNOB_WEIGHT_ONLY_KERNEL, "one_sided": m.KNOB_ONE_SIDED}
    names = {"old": 1, "stream": 2, "wide": 1}
    used = []

    def set_(knob, value):
        used.append(knobs[knob])
        m.mxp_debug_override(knobs[knob], names[value])
    yield set_
    for k in used:
        m.mxp_debug_override(k, 0)


def quantized(x_bits_or_f32, mode, bf16=False):
    q = oracle.quantize(x_bits_or_f32, mode, bf16_bits=bf16)
    dec = oracle.dequantize(q[0], q[1], q[2], mode)
    return host_to_packed(q[0], q[1], q[2] if mode != MX else None, mode), dec


def _raw_operand(rows, K, mode, seed, scale_lo=120, scale_hi=134):
    """Planes filled directly: every code, BM position, BM mantissa (and MX++ delta) occurs."""
    g = synth.rng(seed)
    nib = g.integers(0, 256, (rows, K // 2), dtype=np.uint8)
    sc = g.integers(scale_lo, scale_hi, (rows, K // 32), dtype=np.uint8)
    idx = None
    if mode == MXP:
        idx = g.integers(0, 32, (rows, K // 32), dtype=np.uint8)
    elif mode == MXPP:
        idx = g.integers(0, 256, (rows, K // 32), dtype=np.uint8)
    return host_to_packed(nib, sc, idx, mode), oracle.dequantize(nib, sc, idx, mode)


@pytest.mark.parametrize("kernel", ["old", "stream"])
def test_weight_only_mxpp_raw_planes_one_hot(kernel, force):
    # one-hot activations return single decoded weights exactly (fp32 output): random raw MX++
    # planes, i.e. every code, BM position, BM mantissa and delta
    force("weight_only", kernel)
    K, N = 512, 64
    wp, dw = _raw_operand(N, K, MXPP, seed=51, scale_lo=100, scale_hi=150)
    a = np.zeros((16, K), np.float32)
    cols = [(m * 37 + 5) % K for m in range(16)]
    for m, c in enumerate(cols):
        a[m, c] = 2.0 ** (m - 8)
    d = mxp().mxp_gemm(to_dev_bf16(synth.f32_to_bf16_bits(a)), wp, out_dtype=torch.float32)
    got = d.cpu().numpy().astype(np.float64)
    for m, c in enumerate(cols):
        want = (dw[:, c] * 2.0 ** (m - 8)).astype(np.float32).astype(np.float64)
        assert np.array_equal(got[m], want)


# ------------------------------------------------------------------ bounded waits
def test_bounded_wait_reports_timeout_and_leaves_the_device_usable():
    # a wait that nothing satisfies comes back after its cycle limit, the kernel reports
    # MXP_ERR_TIMEOUT through the status block and exits normally (no trap, no hang)
    m = mxp()
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    m.mxp_wait_selftest(ws, 2_000_000)            # about a millisecond
    assert m.mxp_gemm_status(ws) == 5             # MXP_ERR_TIMEOUT
    torch.cuda.synchronize()
    # the context is intact: a GEMM right after gives a correct result and a clean status
    ap, da = _raw_operand(192, 256, MXP, seed=61)
    bp, db = _raw_operand(320, 256, MXP, seed=62)
    need = m.mxp_gemm_workspace_bytes(192, 320, 256, False, 1, 1)
    ws2 = torch.zeros(need, dtype=torch.uint8, device="cuda")
    d = m.mxp_gemm(ap, bp, out_dtype=torch.float32, workspace=ws2)
    check_gemm(d, da, db)
    assert m.mxp_gemm_status(ws2) == 0
    with pytest.raises(Exception):
        m.mxp_wait_selftest(ws, 0)                # limit out of range: rejected, nothing launched


# ------------------------------------------------------------------ MXFP6 / MXFP6+ operands
MX6, MX6P = 3, 4


def _raw_operand6(rows, K, plus, seed, scale_lo=118, scale_hi=136):
    """MXFP6(+) planes filled directly: every E2M3 code, BM position and five-bit BM mantissa."""
    g = synth.rng(seed)
    codes = g.integers(0, 64, (rows, K), dtype=np.uint8)
    sc = g.integers(scale_lo, scale_hi, (rows, K // 32), dtype=np.uint8)
    idx = g.integers(0, 32, (rows, K // 32), dtype=np.uint8) if plus else None
    dec = oracle.dequantize_wide(codes, sc, idx, oracle.FMT_E2M3, plus)
    from paper_2510_14557_b200 import Packed
    p = Packed(to_dev(oracle.pack6(codes)), to_dev(sc), to_dev(idx) if plus else None, rows, K,
               MX6P if plus else MX6)
    return p, dec


def _any_operand(rows, K, mode, seed):
    if mode in (MX6, MX6P):
        return _raw_operand6(rows, K, mode == MX6P, seed)
    return _raw_operand(rows, K, mode, seed)


@pytest.mark.parametrize("amode,bmode", [(MX6, MX6), (MX6P, MX6), (MX6, MX6P), (MX6P, MX6P),
                                         (MX6P, MX), (MX6P, MXP), (MXP, MX6P), (MX6P, MXPP), (MX, MX6)])
@pytest.mark.parametrize("M,N,K", [(300, 520, 1024), (257, 129, 384), (64, 100, 256), (513, 1000, 128)])
def test_tc_mxfp6_operands(M, N, K, amode, bmode):
    # E2M3 elements go to the tensor core as they are; the BM of an MXFP6+ block enters as the
    # sum of two E2M3 values in two planes, and the K loop runs once per pair of planes
    ap, da = _any_operand(M, K, amode, seed=M + 3)
    bp, db = _any_operand(N, K, bmode, seed=N + 4)
    m = mxp()
    ws = torch.zeros(m.mxp_gemm_workspace_bytes(M, N, K, False, amode, bmode), dtype=torch.uint8, device="cuda")
    for dt in (torch.float32, torch.bfloat16):
        d = m.mxp_gemm(ap, bp, out_dtype=dt, workspace=ws)
        assert m.mxp_gemm_status(ws) == 0
        check_gemm(d, da, db)


@pytest.mark.parametrize("amode", [MX6, MX6P])
def test_tc_mxfp6_identity_partner_returns_the_decode(amode):
    # B = identity: D must equal the oracle's decode of A bit for bit, for every E2M3 code, BM
    # position and BM mantissa (the two planes of a BM add up exactly)
    M, K = 384, 256
    ap, da = _raw_operand6(M, K, amode == MX6P, seed=23)
    eye = np.eye(K, dtype=np.float32)
    for bmode in (MX, MX6P):
        if bmode == MX:
            bp, db = quantized(eye, MX)
        else:
            codes, sc, idx = oracle.quantize_wide(eye, oracle.FMT_E2M3, True)
            db = oracle.dequantize_wide(codes, sc, idx, oracle.FMT_E2M3, True)
            from paper_2510_14557_b200 import Packed
            bp = Packed(to_dev(oracle.pack6(codes)), to_dev(sc), to_dev(idx), K, K, MX6P)
        assert np.array_equal(db, eye.astype(np.float64))
        d = mxp().mxp_gemm(ap, bp, out_dtype=torch.float32)
        assert np.array_equal(d.cpu().numpy().astype(np.float64), da)


def test_tc_mxfp6_quantized_end_to_end_and_rejections():
    from paper_2510_14557_b200 import MxpError
    m = mxp()
    a = synth.activations_normal(320, 512, seed=31, outlier_frac=0.02)
    w = synth.weights(384, 512, seed=32)
    pa = m.mxp_quantize(to_dev(a), MX6P)
    pw = m.mxp_quantize(to_dev(w), MX6)
    ca, sa, ia = oracle.quantize_wide(a, oracle.FMT_E2M3, True)
    cw, sw, iw = oracle.quantize_wide(w, oracle.FMT_E2M3, False)
    da = oracle.dequantize_wide(ca, sa, ia, oracle.FMT_E2M3, True)
    dw = oracle.dequantize_wide(cw, sw, None, oracle.FMT_E2M3, False)
    check_gemm(m.mxp_gemm(pa, pw, out_dtype=torch.float32), da, dw)
    with pytest.raises(MxpError):   # the in-place kernels (minimum workspace) are 4-bit only
        m.mxp_gemm(pa, pw, workspace=torch.zeros(4096, dtype=torch.uint8, device="cuda"))
    # weight-only with 6-bit weights: the same kernel, bf16 activations as two E4M3 planes
    a_bits = synth.f32_to_bf16_bits(a)
    check_gemm(m.mxp_gemm(to_dev_bf16(a_bits), pw, out_dtype=torch.float32), oracle.bf16_bits_to_f64(a_bits), dw)
    with pytest.raises(MxpError):   # the copy's form is the operand's own: one plane is not an MXFP6+ operand's
        m.mxp_gemm_prepack(pa, m.PREPACK_WIDE)


# ------------------------------------------------------------------ MXFP8 operands
MX8 = 5


MX8P = 6


def _raw_operand8(rows, K, seed, scale_lo=112, scale_hi=130, plus=False):
    """MXFP8(+) planes filled directly: every E4M3 code except the NaN pattern and, for MXFP8+,
    every BM position and seven-bit BM mantissa."""
    g = synth.rng(seed)
    codes = g.integers(0, 256, (rows, K), dtype=np.uint8)
    codes[(codes & 0x7F) == 0x7F] = 0x7E
    sc = g.integers(scale_lo, scale_hi, (rows, K // 32), dtype=np.uint8)
    sc[g.random((rows, K // 32)) < 0.02] = 0          # flushed blocks hold zero codes
    idx = None
    if plus:
        idx = g.integers(0, 32, (rows, K // 32), dtype=np.uint8)
        bm_code = g.integers(0, 256, (rows, K // 32), dtype=np.uint8)       # sign + E0M7, 0x7F included
        cols = (np.arange(K // 32) * 32)[None, :] + idx
        np.put_along_axis(codes, cols, bm_code, axis=1)
    codes[np.repeat(sc == 0, 32, axis=1)] = 0
    dec = oracle.dequantize_wide(codes, sc, idx, oracle.FMT_E4M3, plus)
    from paper_2510_14557_b200 import Packed
    return Packed(to_dev(codes), to_dev(sc), to_dev(idx) if plus else None, rows, K,
                  MX8P if plus else MX8), dec


def _operand_of(rows, K, mode, seed):
    if mode in (MX8, MX8P):
        return _raw_operand8(rows, K, seed, plus=mode == MX8P)
    return _any_operand(rows, K, mode, seed)


@pytest.mark.parametrize("amode,bmode", [(MX8, MX8), (MX8, MXP), (MX, MX8), (MX6P, MX8), (MX8, MXPP),
                                         (MX8P, MX8), (MX8, MX8P), (MX8P, MX8P), (MX8P, MXP), (MX6P, MX8P)])
@pytest.mark.parametrize("M,N,K", [(300, 520, 1024), (257, 129, 384), (64, 100, 256), (513, 1000, 128)])
def test_tc_mxfp8_operands(M, N, K, amode, bmode):
    # E4M3 elements are an operand format of the same instruction: the codes go in as stored,
    # next to 4- and 6-bit partners on the other side
    # (an MXFP8+ operand: three planes, the BM being the sum of three E4M3 values)
    ap, da = _operand_of(M, K, amode, seed=M + 5)
    bp, db = _operand_of(N, K, bmode, seed=N + 6)
    m = mxp()
    ws = torch.zeros(m.mxp_gemm_workspace_bytes(M, N, K, False, amode, bmode), dtype=torch.uint8, device="cuda")
    for dt in (torch.float32, torch.bfloat16):
        d = m.mxp_gemm(ap, bp, out_dtype=dt, workspace=ws)
        assert m.mxp_gemm_status(ws) == 0
        check_gemm(d, da, db)


def test_tc_mxfp8_identity_and_quantized_end_to_end():
    m = mxp()
    # B = identity: D is the decode of A bit for bit, for every E4M3 code
    M, K = 384, 256
    ap, da = _raw_operand8(M, K, seed=41)
    bp, db = quantized(np.eye(K, dtype=np.float32), MX)
    d = m.mxp_gemm(ap, bp, out_dtype=torch.float32)
    assert np.array_equal(d.cpu().numpy().astype(np.float64), da)
    # ... and for every BM position and seven-bit BM mantissa of MXFP8+ (three planes add up exactly)
    ap, da = _raw_operand8(M, K, seed=42, plus=True)
    d = m.mxp_gemm(ap, bp, out_dtype=torch.float32)
    assert np.array_equal(d.cpu().numpy().astype(np.float64), da)
    # quantized by the library, against the oracle's encode + decode + fp64 product
    a = synth.activations_normal(320, 512, seed=43, outlier_frac=0.02)
    w = synth.weights(384, 512, seed=44)
    pa, pw = m.mxp_quantize(to_dev(a), MX8), m.mxp_quantize(to_dev(w), MX8)
    ca, sa, _ = oracle.quantize_wide(a, oracle.FMT_E4M3, False)
    cw, sw, _ = oracle.quantize_wide(w, oracle.FMT_E4M3, False)
    check_gemm(m.mxp_gemm(pa, pw, out_dtype=torch.float32),
               oracle.dequantize_wide(ca, sa, None, oracle.FMT_E4M3, False),
               oracle.dequantize_wide(cw, sw, None, oracle.FMT_E4M3, False))
    # prepacked weights
    pre = m.mxp_gemm_prepack(pw, True)
    check_gemm(m.mxp_gemm_prepacked(pa, pw, pre, out_dtype=torch.float32),
               oracle.dequantize_wide(ca, sa, None, oracle.FMT_E4M3, False),
               oracle.dequantize_wide(cw, sw, None, oracle.FMT_E4M3, False))


# ------------------------------------------------------------------ fused quantize -> GEMM
@pytest.mark.parametrize("amode,bmode", [(MXP, MXP), (MX, MXP)])
@pytest.mark.parametrize("M,N,K", [(300, 520, 1024), (257, 1000, 384), (512, 512, 128)])
def test_quantize_gemm_ready_matches_the_two_step_path(M, N, K, amode, bmode, force):
    # the quantizer writes the packed planes (bit-exact, as mxp_quantize) and A's GEMM-ready
    # form (widened E2M3 codes; the split form of an MXFP4+ A against MXFP4 weights has its own
    # tests); the GEMM then needs no prepack launch and returns what mxp_gemm returns on the
    # widened pass
    m = mxp()
    force("one_sided", "wide")
    a_bits = synth.f32_to_bf16_bits(synth.activations_normal(M, K, seed=M + K, outlier_frac=0.02))
    a_bits[3, 32:64] = 0                       # a zero block
    a_bits[5, 64:96] = 0x0001                  # a flushed block
    bp, db = _raw_operand(N, K, bmode, seed=N)
    pre = m.mxp_gemm_prepack(bp, True)
    ws = torch.full((m.mxp_gemm_workspace_bytes(M, N, K, False, amode, bmode),), 0xA5, dtype=torch.uint8, device="cuda")
    pa = m.mxp_quantize_gemm_ready(to_dev_bf16(a_bits), amode, ws, b_mode=bmode)
    ref = oracle.quantize(a_bits, amode, bf16_bits=True)
    assert np.array_equal(pa.nibbles.cpu().numpy(), ref[0])
    assert np.array_equal(pa.scales.cpu().numpy(), ref[1])
    if amode != MX:
        assert np.array_equal(pa.bm_index.cpu().numpy(), ref[2])
    da = oracle.dequantize(*ref, amode)
    for dt in (torch.float32, torch.bfloat16):
        d = m.mxp_gemm_ready(pa, bp, pre, ws, out_dtype=dt)
        assert m.mxp_gemm_status(ws) == 0
        check_gemm(d, da, db)
        assert torch.equal(d, m.mxp_gemm(pa, bp, out_dtype=dt))


def test_quantize_gemm_ready_rejections():
    from paper_2510_14557_b200 import MxpError
    m = mxp()
    ws = torch.zeros(1 << 22, dtype=torch.uint8, device="cuda")
    x = torch.randn(256, 256, device="cuda")
    with pytest.raises(MxpError):   # fp32 source: not the fused kernel's case
        m.mxp_quantize_gemm_ready(x, MXP, ws)
    with pytest.raises(MxpError):   # MX++ keeps its own prepack
        m.mxp_quantize_gemm_ready(x.bfloat16(), MXPP, ws)
    with pytest.raises(MxpError):   # M <= 128: no streamed kernel
        m.mxp_quantize_gemm_ready(x.bfloat16()[:64].contiguous(), MXP, ws)
    with pytest.raises(MxpError):   # workspace too small
        m.mxp_quantize_gemm_ready(x.bfloat16(), MXP, ws[:4096])


@pytest.mark.parametrize("bmode", [3, 4, 5, 6])
@pytest.mark.parametrize("amode", [MXP, 4])
def test_tc_prepacked_weights_at_the_wider_formats(amode, bmode):
    # weights prepared once, all planes of an MXFP6+ (two) or MXFP8+ (three) operand included:
    # the same result as mxp_gemm on the same operands, to the bit
    m = mxp()
    M, N, K = 300, 520, 512
    ap, da = _operand_of(M, K, amode, seed=81)
    bp, db = _operand_of(N, K, bmode, seed=82)
    form = m.mxp_gemm_prepack_form(amode, bmode)
    assert form == {3: m.PREPACK_WIDE, 4: m.PREPACK_WIDE_X2, 5: m.PREPACK_WIDE8, 6: m.PREPACK_WIDE8_X3}[bmode]
    pre = m.mxp_gemm_prepack(bp, form)
    assert pre.numel() == m.mxp_gemm_prepack(bp, True).numel()
    for dt in (torch.float32, torch.bfloat16):
        d0 = m.mxp_gemm(ap, bp, out_dtype=dt)
        d1 = m.mxp_gemm_prepacked(ap, bp, pre, out_dtype=dt)
        check_gemm(d1, da, db)
        assert torch.equal(d0, d1)
