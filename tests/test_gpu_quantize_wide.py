"""GPU parity: MXFP6(+) / MXFP8(+) quantize and dequantize through the C ABI vs the CPU oracle
(bit-exact codes, scales, indices and decoded values)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import to_dev, to_dev_bf16
from paper_2510_14557_b200 import synth

pytestmark = pytest.mark.gpu
# mode -> (element format, plus)
MODES = {3: (oracle.FMT_E2M3, False), 4: (oracle.FMT_E2M3, True),
         5: (oracle.FMT_E4M3, False), 6: (oracle.FMT_E4M3, True)}


def mxp():
    import paper_2510_14557_b200 as m
    return m


def reference_planes(x, mode, bf16_bits=False):
    fmt, plus = MODES[mode]
    codes, sc, idx = oracle.quantize_wide(x, fmt, plus, bf16_bits=bf16_bits)
    stored = oracle.pack6(codes) if fmt == oracle.FMT_E2M3 else codes
    return stored, sc, idx, codes


def assert_equal(p, ref, mode, what=""):
    stored, sc, idx, _ = ref
    assert np.array_equal(p.scales.cpu().numpy(), sc), "scales differ " + what
    got = p.nibbles.cpu().numpy()
    assert got.shape == stored.shape
    assert np.array_equal(got, stored), "codes differ %s (%d bytes)" % (what, int((got != stored).sum()))
    if MODES[mode][1]:
        assert np.array_equal(p.bm_index.cpu().numpy(), idx), "indices differ " + what


def adversarial(emax):
    """Ties on both element grids, saturation, BM rounding and clamp, flush boundary, signed
    zeros, subnormals, equal maxima."""
    rows = []
    top = 2.0 ** emax
    ties = [1.0625, 1.1875, 1.3125, 0.0625, 0.1875, 2.125, 3.625, 2.0 ** -10, 3 * 2.0 ** -11,
            top * 1.03125, top * 1.09375, top * 1.00390625, top * 1.01171875, top * 1.9, top * 1.99]
    for sh in (0, -9, 25, -110, 110):
        for pos in (0, 1, 14, 15, 16, 30, 31):
            b = np.zeros(32, np.float32)
            b[pos] = top * 1.99609375
            for i, v in enumerate(ties):
                if i != pos:
                    b[(pos + 1 + i) % 32] = v * (-1) ** i
            rows.append(b * np.float32(2.0 ** sh))
    for bm in [1.0, 1.0078125, 1.01171875, 1.015625, 1.5, 1.984375, 1.9921875, 1.99609375, 1.998046875]:
        for pos in (2, 13, 31):
            b = np.full(32, 0.37, np.float32)
            b[pos] = -bm * top
            rows.append(b)
    b = np.zeros(32, np.float32); rows.append(b.copy())
    b[5] = 2.0 ** (-127 + emax); rows.append(b.copy())                       # flushed
    b[5] = 2.0 ** (-126 + emax); b[6] = 2.0 ** -135; rows.append(b.copy())   # smallest kept
    b = np.zeros(32, np.float32); b[3] = 5.0; b[4] = -5.0; b[31] = 5.0; rows.append(b.copy())
    b = np.full(32, -0.0, np.float32); b[9] = 1e-3; rows.append(b.copy())    # signed zeros
    b = np.full(32, 1e-41, np.float32); rows.append(b.copy())                # fp32 subnormals
    b = np.full(32, 3.0e38, np.float32); b[4] = np.finfo(np.float32).max; rows.append(b.copy())
    x = np.stack(rows)
    pad = (-x.shape[0]) % 4
    x = np.concatenate([x, np.zeros((pad, 32), np.float32)])
    return x.reshape(-1, 128)


@pytest.mark.parametrize("mode", sorted(MODES))
def test_adversarial_blocks_fp32_and_bf16(mode):
    x = adversarial(2 if mode in (3, 4) else 8)
    p = mxp().mxp_quantize(to_dev(x), mode)
    assert_equal(p, reference_planes(x, mode), mode, "fp32")
    bits = synth.f32_to_bf16_bits(x)
    p = mxp().mxp_quantize(to_dev_bf16(bits), mode)
    assert_equal(p, reference_planes(bits, mode, bf16_bits=True), mode, "bf16")


@pytest.mark.parametrize("mode", sorted(MODES))
def test_every_finite_bf16_pattern_as_block_max_and_as_element(mode):
    # all bf16 bit patterns, each once as the first element of a block, with NBMs that exercise
    # small codes; non-finite patterns are replaced (blocks holding them are not pinned)
    allp = np.arange(65536, dtype=np.uint16)
    allp[(allp & 0x7F80) == 0x7F80] = 0x3F80
    bits = np.zeros((2048, 32 * 32), np.uint16)
    bits[:, ::32] = allp.reshape(2048, 32)
    bits[:, 1::32] = 0x3E80   # 0.25
    bits[:, 5::32] = 0xBF40   # -0.75
    bits[:, 9::32] = np.roll(allp, 7).reshape(2048, 32) & 0xBFFF  # assorted smaller magnitudes
    p = mxp().mxp_quantize(to_dev_bf16(bits), mode)
    assert_equal(p, reference_planes(bits, mode, bf16_bits=True), mode)


@pytest.mark.parametrize("shape", [(1, 32), (3, 96), (5, 8192), (257, 2080), (1000, 32)])
@pytest.mark.parametrize("mode", sorted(MODES))
def test_ragged_sizes_bf16_and_fp32(shape, mode):
    bits = synth.config2(shape[0], shape[1], seed=shape[0] + shape[1])
    p = mxp().mxp_quantize(to_dev_bf16(bits), mode)
    assert_equal(p, reference_planes(bits, mode, bf16_bits=True), mode, str(shape))
    x = synth.activations_normal(shape[0], shape[1], seed=shape[1], outlier_frac=0.01)
    p = mxp().mxp_quantize(to_dev(x), mode)
    assert_equal(p, reference_planes(x, mode), mode, str(shape) + " fp32")


def test_strided_source_and_guard_bytes():
    m = mxp()
    x = synth.activations_normal(37, 256, seed=9)
    wide = torch.zeros((37, 384), dtype=torch.float32, device="cuda")
    wide[:, :256] = to_dev(x)
    for mode in (4, 6):
        out = m.alloc_packed(37 + 1, 256, mode)  # one spare row as a canary
        for t in (out.nibbles, out.scales, out.bm_index):
            t.fill_(0xA5)
        view = m.Packed(out.nibbles[:37], out.scales[:37], out.bm_index[:37], 37, 256, mode)
        m.mxp_quantize(wide[:, :256], mode, out=view)
        assert_equal(view, reference_planes(x, mode), mode)
        for t in (out.nibbles, out.scales, out.bm_index):
            assert bool((t[37] == 0xA5).all())


@pytest.mark.parametrize("mode", sorted(MODES))
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_dequantize_bit_exact(mode, dtype):
    m = mxp()
    fmt, plus = MODES[mode]
    x = np.concatenate([adversarial(2 if fmt == oracle.FMT_E2M3 else 8),
                        synth.activations_normal(64, 128, seed=5)])
    stored, sc, idx, codes = reference_planes(x, mode)
    ref = oracle.dequantize_wide(codes, sc, idx, fmt, plus)
    p = m.Packed(to_dev(stored), to_dev(sc), to_dev(idx) if plus else None, x.shape[0], x.shape[1], mode)
    got = m.mxp_dequantize(p, dtype).float().cpu().numpy().astype(np.float64)
    # at most 8 significant bits: exact in fp32; in bf16 too, except below its subnormal grid,
    # where the store rounds to nearest even
    if dtype == torch.bfloat16:
        from helpers import bf16_round
        ref = bf16_round(ref)
    assert np.array_equal(got, ref)
    assert np.array_equal(np.signbit(got), np.signbit(ref))


def test_unsupported_uses_of_the_wide_modes_are_rejected():
    from paper_2510_14557_b200 import MxpError
    m = mxp()
    a = torch.randn(256, 256, device="cuda", dtype=torch.bfloat16)
    p6 = m.mxp_quantize(a, 4)
    p8 = m.mxp_quantize(a, 6)
    tiny = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(MxpError):  # weight-only form at these widths: the tensor-core kernel and its workspace only
        m.mxp_gemm(a, p6, workspace=tiny)
    with pytest.raises(MxpError):
        m.mxp_gemm(a, p8, workspace=tiny)
    with pytest.raises(MxpError):  # an MXFP8+ operand's prepacked copy has three planes, not one
        m.mxp_gemm_prepack(p8, m.PREPACK_WIDE8)
    with pytest.raises(MxpError):  # the + modes need the index plane
        m.mxp_quantize(a, 6, out=m.Packed(p8.nibbles, p8.scales, None, 256, 256, 6))


@pytest.mark.parametrize("mode", [3, 4, 5, 6])
@pytest.mark.parametrize("M,N,K", [(1, 300, 256), (16, 129, 512), (70, 520, 384), (300, 1000, 1024)])
def test_weight_only_with_the_wider_weight_formats(M, N, K, mode):
    # bf16 activations x MXFP6 / MXFP6+ / MXFP8 / MXFP8+ weights (Sec. 4.2 lists these widths beside
    # MXFP4+): the block-scaled tensor-core kernel at any M, the activations as two E4M3 planes,
    # the weights' BM as the sum of two (MXFP6+) or three (MXFP8+) planes; against the oracle's
    # fp64 product of the decoded operands
    from helpers import check_gemm
    m = mxp()
    a_bits, w_bits = synth.config3(M, N, K, seed=M + N + K + mode)
    fmt, plus = MODES[mode]
    codes, sc, idx = oracle.quantize_wide(w_bits, fmt, plus, bf16_bits=True)
    dw = oracle.dequantize_wide(codes, sc, idx, fmt, plus)
    da = oracle.bf16_bits_to_f64(a_bits)
    wp = m.mxp_quantize(to_dev_bf16(w_bits), mode)
    assert_equal(wp, reference_planes(w_bits, mode, bf16_bits=True), mode)
    need = m.mxp_gemm_workspace_bytes(M, N, K, True, 0, mode)
    assert need > 4096
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    for dt in (torch.float32, torch.bfloat16):
        d = m.mxp_gemm(to_dev_bf16(a_bits), wp, out_dtype=dt, workspace=ws)
        assert m.mxp_gemm_status(ws) == 0
        check_gemm(d, da, dw)
