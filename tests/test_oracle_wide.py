"""Pins for the oracle's MXFP6 / MXFP6+ (E2M3) and MXFP8 / MXFP8+ (E4M3) functions.

The paper prints no worked example at these widths (Table "Concrete MX-compliant formats",
Sec. 4.1, Sec. 4.2 give the types, the BM re-encoding and the layout), so the pins are the
types' definitions typed out, a library cast, a closed form, invariants and brute force."""
import numpy as np
import pytest

import oracle

E2M3, E4M3 = oracle.FMT_E2M3, oracle.FMT_E4M3
EMAX = {E2M3: 2, E4M3: 8}
MAXV = {E2M3: 7.5, E4M3: 448.0}


def test_element_tables_match_the_types_definitions():
    # E2M3: bias 1, subnormal step 1/8, largest 2^2 * 1.875; E4M3 (OCP FP8): bias 7, smallest
    # subnormal 2^-9, largest finite 2^8 * 1.75 (the all-ones code is NaN and is not a value)
    v6 = [oracle.elem_value(E2M3, c) for c in range(32)]
    assert v6[:9] == [0.0, 0.125, 0.25, 0.375, 0.5, 0.625, 0.75, 0.875, 1.0]
    assert v6[16] == 2.0 and v6[24] == 4.0 and v6[31] == 7.5 and v6[9] == 1.125
    assert all(b > a for a, b in zip(v6, v6[1:]))
    v8 = [oracle.elem_value(E4M3, c) for c in range(127)]
    assert v8[1] == 2.0 ** -9 and v8[8] == 2.0 ** -6 and v8[0x38] == 1.0 and v8[126] == 448.0
    assert v8[0x78] == 256.0 and v8[0x40] == 2.0 and v8[0x39] == 1.125
    assert all(b > a for a, b in zip(v8, v8[1:]))


def _scaled_case(fmt, seed, n=4096):
    # blocks whose first element fixes the scale at 2^0 * 2^emax (BM = 2^emax exactly), so the
    # other 31 elements are cast at scale 1 and can be compared with an independent cast
    g = np.random.default_rng(seed)
    x = np.zeros((n, 32), np.float64)
    x[:, 0] = 2.0 ** EMAX[fmt]
    mag = np.exp2(g.uniform(-12, EMAX[fmt], (n, 31))) * g.choice([-1.0, 1.0], (n, 31))
    x[:, 1:] = np.where(np.abs(mag) < 2.0 ** EMAX[fmt], mag, 1.0)
    return x


def test_e4m3_cast_matches_the_library_cast():
    torch = pytest.importorskip("torch")
    if not hasattr(torch, "float8_e4m3fn"):
        pytest.skip("no float8_e4m3fn in this torch")
    x = _scaled_case(E4M3, 1).astype(np.float32)
    codes, sc, _ = oracle.quantize_wide(x, E4M3, False)
    assert np.all(sc == 127)
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(codes, want)


@pytest.mark.parametrize("fmt", [E2M3, E4M3])
def test_cast_matches_round_half_even_on_the_types_grid(fmt):
    # closed form: the grid step at |x| is 2^(max(floor(log2|x|), emin) - 3); numpy's rint
    # rounds half to even, and an even multiple of the step is an even code
    x = _scaled_case(fmt, 2)
    codes, sc, _ = oracle.quantize_wide(x, fmt, False)
    dec = oracle.dequantize_wide(codes, sc, None, fmt, False)
    emin = 0 if fmt == E2M3 else -6
    a = np.abs(x)
    ex = np.floor(np.log2(np.maximum(a, 1e-300)))
    step = np.exp2(np.maximum(ex, emin) - 3)
    want = np.minimum(np.rint(a / step) * step, MAXV[fmt]) * np.sign(x)
    assert np.array_equal(dec, want)


@pytest.mark.parametrize("fmt", [E2M3, E4M3])
def test_saturation_and_ties(fmt):
    top = 2.0 ** EMAX[fmt]
    x = np.zeros((1, 32))
    x[0, 0] = top * 1.99          # BM near the top of its binade: plain format saturates
    x[0, 1] = -top * 1.99 * 0.999
    x[0, 2] = 1.0625              # midway between 1.0 (even code) and 1.125: ties to even
    x[0, 3] = 1.1875              # midway between 1.125 and 1.25 (even code)
    codes, sc, idx = oracle.quantize_wide(x, fmt, False)
    dec = oracle.dequantize_wide(codes, sc, idx, fmt, False)
    assert dec[0, 0] == MAXV[fmt] and dec[0, 1] == -MAXV[fmt]
    assert dec[0, 2] == 1.0 and dec[0, 3] == 1.25


@pytest.mark.parametrize("fmt", [E2M3, E4M3])
def test_bm_grid_error_bound_and_clamp(fmt):
    # the BM keeps its sign bit and spends the rest on mantissa: 2^emax * (1 + m / 2^(bits-1)),
    # so its relative error is at most half a grid step, except for the clamp at the top
    mb = fmt - 1
    g = np.random.default_rng(3)
    x = g.standard_normal((512, 32)) * np.exp2(g.integers(-20, 20, (512, 1)))
    codes, sc, idx = oracle.quantize_wide(x, fmt, True)
    dec = oracle.dequantize_wide(codes, sc, idx, fmt, True)
    codes0, sc0, _ = oracle.quantize_wide(x, fmt, False)
    assert np.array_equal(sc, sc0)                       # MX+ does not alter the shared scale
    rows = np.arange(512)
    bm = np.argmax(np.abs(x), axis=1)
    assert np.array_equal(idx[:, 0], bm)
    others = np.ones_like(x, bool)
    others[rows, bm] = False
    assert np.array_equal(codes[others], codes0[others])  # NBMs are the plain format's
    t, d = x[rows, bm], dec[rows, bm]
    scale = np.exp2(sc[:, 0].astype(np.float64) - 127)
    grid = scale * 2.0 ** EMAX[fmt] / 2 ** mb
    clamp = np.abs(t) > scale * 2.0 ** (EMAX[fmt] + 1) - grid
    assert np.all(np.abs(d - t)[~clamp] <= grid[~clamp] / 2 * (1 + 1e-12))
    assert np.all(np.abs(d[clamp]) == (scale * 2.0 ** (EMAX[fmt] + 1) - grid)[clamp])
    # and it is never worse than the plain cast of the same element
    dec0 = oracle.dequantize_wide(codes0, sc0, None, fmt, False)
    assert np.all(np.abs(d - t) <= np.abs(dec0[rows, bm] - t) + 1e-300)


@pytest.mark.parametrize("fmt", [E2M3, E4M3])
def test_every_code_round_trips(fmt):
    # a block holding the BM 2^emax and 31 representable values decodes to itself
    n = 32 if fmt == E2M3 else 127
    vals = np.array([oracle.elem_value(fmt, c) for c in range(n)])
    vals = vals[vals < 2.0 ** EMAX[fmt]]
    x = np.zeros((len(vals) // 31 + 1, 32))
    x[:, 0] = 2.0 ** EMAX[fmt]
    flat = np.resize(vals, x.shape[0] * 31) * np.resize([1.0, -1.0], x.shape[0] * 31)
    x[:, 1:] = flat.reshape(-1, 31)
    for plus in (False, True):
        codes, sc, idx = oracle.quantize_wide(x, fmt, plus)
        assert np.array_equal(oracle.dequantize_wide(codes, sc, idx, fmt, plus), x)


@pytest.mark.parametrize("fmt", [E2M3, E4M3])
def test_scale_and_flush_thresholds(fmt):
    # Eq. 1 with the format's emax; floor(log2 BM) <= -127 + emax flushes the block
    e = EMAX[fmt]
    x = np.zeros((4, 32), np.float64)
    x[0, 5] = 2.0 ** (-127 + e + 1)        # smallest exponent that survives: scale byte 1
    x[1, 5] = 2.0 ** (-127 + e) * 1.99     # flushed
    x[2, 7] = -3.0 * 2.0 ** 10             # floor(log2) = 11
    x[3, :] = 0.0
    codes, sc, idx = oracle.quantize_wide(x, fmt, True)
    assert sc[:, 0].tolist() == [1, 0, 11 - e + 127, 0]
    assert not codes[1].any() and not codes[3].any() and idx[1, 0] == 0
    assert idx[2, 0] == 7 and codes[2, 7] >> (fmt - 1) == 1   # sign kept on the BM
    dec = oracle.dequantize_wide(codes, sc, idx, fmt, True)
    assert dec[0, 5] == x[0, 5] and dec[2, 7] == x[2, 7] and not dec[1].any()


def test_six_bit_packing_order():
    # code i in bits 6i..6i+5 of the little-endian bit stream: four codes in three bytes
    codes = np.array([[0x01, 0x02, 0x03, 0x3F, 0x20, 0x00, 0x15, 0x2A]], np.uint8)
    want = 0
    for i, c in enumerate(codes[0]):
        want |= int(c) << (6 * i)
    assert oracle.pack6(codes)[0].tolist() == list(want.to_bytes(6, "little"))
    assert oracle.pack6(codes)[0, :3].tolist() == [0x81, 0x30, 0xFC]
