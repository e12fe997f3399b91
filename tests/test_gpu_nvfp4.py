"""GPU parity: mxp_nvfp4_quantize / mxp_nvfp4_dequantize through the C ABI vs the CPU oracle,
bit-exact (Sec. 8, "Applicability of MX+ to NVFP4")."""
import numpy as np
import pytest
import torch

import oracle
from helpers import f64_to_bf16_bits, nvfp4_boundary_blocks, to_dev, to_dev_bf16
from paper_2510_14557_b200 import synth

pytestmark = pytest.mark.gpu


def mxp():
    import paper_2510_14557_b200 as m
    return m


def check_planes(got, ref, plus):
    nib, sc, idx = got
    assert np.array_equal(sc.cpu().numpy(), ref[1]), "scales differ"
    d = nib.cpu().numpy() != ref[0]
    assert not d.any(), "nibbles differ in %d bytes" % int(d.sum())
    if plus:
        assert np.array_equal(idx.cpu().numpy(), ref[2]), "indices differ"


def tensor_scale(x):
    return float(np.abs(x).max() / (6.0 * 448.0))


@pytest.mark.parametrize("plus", [False, True])
@pytest.mark.parametrize("rows,cols", [(1, 32), (5, 96), (64, 4096), (33, 1056), (257, 8192)])
def test_bf16_bit_exact(rows, cols, plus):
    bits = synth.f32_to_bf16_bits(synth.activations_normal(rows, cols, rows + cols, 0.01, 30.0))
    x = oracle.bf16_bits_to_f64(bits)
    for ts in (tensor_scale(x), 1.0, 2.0 ** -20, 0.37):
        ref = oracle.nvfp4_quantize(bits, ts, plus, bf16_bits=True)
        got = mxp().mxp_nvfp4_quantize(to_dev_bf16(bits), ts, plus)
        check_planes(got, ref, plus)


@pytest.mark.parametrize("plus", [False, True])
def test_fp32_strided_bit_exact_with_wide_exponent_spread(plus):
    rows, cols, ld = 45, 320, 352
    g = synth.rng(8)
    blk_exp = np.repeat(g.integers(-26, 3, (rows, ld // 16)), 16, axis=1)      # per block of 16
    full = (g.standard_normal((rows, ld)) * np.exp2(blk_exp)).astype(np.float32)
    x = np.ascontiguousarray(full[:, :cols])
    for ts in (tensor_scale(x), 2.0 ** -12):
        ref = oracle.nvfp4_quantize(x, ts, plus)
        got = mxp().mxp_nvfp4_quantize(to_dev(full)[:, :cols], ts, plus)
        check_planes(got, ref, plus)
        # the spread reaches the coarse-scale fallback and flushed blocks as well
        assert (ref[1] <= 2).any() and (ref[1] == 0).any() and (ref[1] > 8).any()


def adversarial_blocks():
    """Ties of the element cast, of the BM cast and of the scale cast; equal maxima; signed
    zeros; saturating scale; scale bytes 0..4."""
    rows = []
    ties = [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 0.125, 5.9, 0.24, 0.26]
    for amax, sh in ((6.0, 0), (6.0, -5), (6.0, 7), (5.75, 0), (6.25, 0), (5.5, 0), (6.5, 0),
                     (6.375, 0), (5.65, 0), (7.0, 0), (4.5, 3)):
        for pos in (0, 7, 8, 15):
            b = np.zeros(16, np.float32)
            for i, v in enumerate(ties):
                b[(pos + 1 + i) % 16] = v * (-1) ** i
            b[pos] = -amax if pos & 1 else amax
            rows.append(b * np.float32(2.0 ** sh))
    b = np.zeros(16, np.float32); rows.append(b.copy())
    b[3] = 6.0; b[9] = -6.0; b[15] = 6.0; rows.append(b.copy())              # equal maxima
    b = np.full(16, -0.0, np.float32); b[4] = 1e-3; rows.append(b.copy())     # signed zeros
    for k in (0.4, 0.6, 1, 1.5, 2, 2.5, 3, 3.5, 4, 4.5):                      # scale bytes 0..4 and ties
        b = np.full(16, 2.0 ** -12, np.float32); b[5] = np.float32(6 * k * 2.0 ** -9); rows.append(b.copy())
    b = np.full(16, 100.0, np.float32); b[2] = 6 * 448.0; rows.append(b.copy())      # largest scale
    b = np.full(16, 100.0, np.float32); b[2] = 6 * 1000.0; rows.append(b.copy())     # saturating scale
    b = np.full(16, 100.0, np.float32); b[11] = -6 * 460.0; rows.append(b.copy())
    x = np.stack(rows)
    pad = (-x.shape[0]) % 4
    x = np.concatenate([x, np.zeros((pad, 16), np.float32)])
    return x.reshape(-1, 64)


@pytest.mark.parametrize("plus", [False, True])
def test_adversarial_blocks_bit_exact(plus):
    x = adversarial_blocks()
    for ts in (1.0, 0.75, 1.0 / 3.0):
        ref = oracle.nvfp4_quantize(x, ts, plus)
        got = mxp().mxp_nvfp4_quantize(to_dev(x), ts, plus)
        check_planes(got, ref, plus)


@pytest.mark.parametrize("plus", [False, True])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_decode_bit_exact(plus, dtype):
    rows, cols = 37, 512
    g = synth.rng(5)
    x = (g.standard_normal((rows, cols)) * np.exp2(g.integers(-10, 4, (rows, cols)))).astype(np.float32)
    ts = tensor_scale(x)
    nib, sc, idx = oracle.nvfp4_quantize(x, ts, plus)
    want = oracle.nvfp4_dequantize(nib, sc, idx, ts, plus)
    got = mxp().mxp_nvfp4_dequantize(to_dev(nib), to_dev(sc), to_dev(idx) if plus else None, ts, plus, dtype)
    # the oracle's decode is exact (float64); the library rounds it once to the output type
    if dtype == torch.float32:
        assert np.array_equal(got.cpu().numpy().view(np.uint32), want.astype(np.float32).view(np.uint32))
    else:
        assert np.array_equal(got.cpu().view(torch.int16).numpy().view(np.uint16), f64_to_bf16_bits(want))
    # every possible (code, scale byte) pair, BM in every position
    codes = np.arange(256, dtype=np.uint8).reshape(1, 256).repeat(128, axis=0)     # all byte values
    scb = (np.arange(128) % 127).astype(np.uint8).reshape(128, 1).repeat(32, axis=1)   # 0x7F is the NaN pattern
    rng_idx = g.integers(0, 256, (128, 16)).astype(np.uint8)
    # a tensor scale with 24 significant bits: products need the single rounding
    for ts in (0.5, 0.7330000996589661, 1.0 / 3.0):
        want = oracle.nvfp4_dequantize(codes, scb, rng_idx, ts, plus)
        got = mxp().mxp_nvfp4_dequantize(to_dev(codes), to_dev(scb), to_dev(rng_idx) if plus else None, ts, plus, dtype)
        if dtype == torch.float32:
            assert np.array_equal(got.cpu().numpy().view(np.uint32), want.astype(np.float32).view(np.uint32))
        else:
            assert np.array_equal(got.cpu().view(torch.int16).numpy().view(np.uint16), f64_to_bf16_bits(want))


@pytest.mark.parametrize("plus", [False, True])
def test_rounding_boundaries_bit_exact(plus):
    # elements, BMs and block maxima exactly on, one binary32 step above and one step below a
    # rounding boundary of the element, BM and scale casts: the codes must be those of exact
    # arithmetic, whatever a reciprocal in binary32 would make of them
    for ts, seed in ((1.0, 1), (0.37, 2), (2.0 ** -8, 3), (1.0 / 3.0, 4), (0.6458333134651184, 5)):
        x = nvfp4_boundary_blocks(ts, seed)
        ref = oracle.nvfp4_quantize(x, ts, plus)
        got = mxp().mxp_nvfp4_quantize(to_dev(x), ts, plus)
        check_planes(got, ref, plus)
    # bf16 sources: boundaries t * d that bf16 holds.  Tensor scales of up to 12 significant bits
    # take the kernel's short-operand form (quotient by a Newton step, no per-element settling),
    # longer ones the general form; signed zeros and tiny elements keep their sign in both.
    for ts, seed in ((2.0 ** -3, 9), (0.75, 10), (2867.0 / 4096.0, 11), (1.0 + 2.0 ** -11, 12),
                     (1.0 + 2.0 ** -12, 13), (3.0 * 2.0 ** -40, 14)):
        x = nvfp4_boundary_blocks(ts, seed)
        x[::7, 3] = -0.0
        x[::5, 11] = np.float32(-2.0 ** -120)
        x[::9, 17] = np.float32(3.0e38)       # the scale saturates and quotients overflow binary32
        x[1::9, 5] = np.float32(-2.0e30)
        bits = synth.f32_to_bf16_bits(x)
        ref = oracle.nvfp4_quantize(bits, ts, plus, bf16_bits=True)
        got = mxp().mxp_nvfp4_quantize(to_dev_bf16(bits), ts, plus)
        check_planes(got, ref, plus)


def test_config2_whole_matrix_and_argument_checks():
    m = mxp()
    bits = synth.config2()
    oracle.set_threads(oracle.max_threads())
    try:
        # a power-of-two tensor scale (exact ties are frequent) and the usual amax / (6 * 448)
        for ts in (2.0 ** -8, float(np.float32(np.abs(oracle.bf16_bits_to_f64(bits)).max() / (6 * 448)))):
            got = m.mxp_nvfp4_quantize(to_dev_bf16(bits), ts, True)
            ref = oracle.nvfp4_quantize(bits, ts, True, bf16_bits=True)
            check_planes(got, ref, True)
    finally:
        oracle.set_threads(1)
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    for bad in (0.0, -1.0, float("inf"), float("nan"), 2.0 ** -101, 2.0 ** 101):
        with pytest.raises(m.MxpError) as e:
            m.mxp_nvfp4_quantize(x, bad, True)
        assert e.value.status == 1
    with pytest.raises(m.MxpError):
        m.mxp_nvfp4_quantize(torch.zeros((4, 48), dtype=torch.bfloat16, device="cuda"), 1.0, False)
