"""Pins for the CPU oracle's encoder / decoder (no GPU).

Each test checks the oracle against something other than itself: values the paper
prints, closed forms from the format definition, invariants the paper states, special
cases, and brute-force search on tiny blocks.
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import MODE_MXFP4 as MX, MODE_MXFP4_PLUS as MXP

GOLD = os.path.join(os.path.dirname(__file__), "golden")

# E2M1 magnitudes from the definition: 2-bit exponent with bias 1, 1 mantissa bit,
# implicit leading one, IEEE-like subnormals (Sec. 2 / Sec. 3.1).
E2M1 = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


def block(vals: dict, k=32):
    x = np.zeros((1, k), np.float32)
    for i, v in vals.items():
        x[0, i] = v
    return x


def nibble_list(nib_row):
    out = []
    for b in nib_row:
        out += [int(b) & 15, int(b) >> 4]
    return out


# ---------------------------------------------------------------- element table
def test_e2m1_table_matches_definition():
    for code in range(8):
        e, m = code >> 1, code & 1
        # (-1)^s * 2^(max(e,1)-bias) * (min(e,1) + m/2)
        want = 2.0 ** (max(e, 1) - 1) * (min(e, 1) + m / 2)
        assert oracle.e2m1_value(code) == want == E2M1[code]
    # emax = 11b - bias = 2, largest magnitude 1.5 * 2^2
    assert max(E2M1) == 1.5 * 2 ** 2


def test_decode_all_codes_both_modes():
    # one block, element 0 carries each of the 16 nibbles in turn; scale byte 127 (2^0)
    for nib in range(16):
        n = np.zeros((1, 16), np.uint8)
        n[0, 0] = nib
        sc = np.full((1, 1), 127, np.uint8)
        idx = np.zeros((1, 1), np.uint8)
        s, code = nib >> 3, nib & 7
        d_mx = oracle.dequantize(n, sc, None, MX)[0, 0]
        d_mxp = oracle.dequantize(n, sc, idx, MXP)[0, 0]
        assert d_mx == (-1) ** s * E2M1[code]
        assert math.copysign(1, d_mx) == (-1) ** s or code == 0
        # BM is "effectively E2M3" with exponent field 11b (Sec. 4.2): 2^(3-1) * (1 + m/8)
        assert d_mxp == (-1) ** s * 2.0 ** (3 - 1) * (1 + code / 8)
        # and equals Eq. 3's BM branch 2^emax * m_i with 3 mantissa bits
        assert abs(d_mxp) == 4 + code / 2


def test_scale_byte_applies_as_power_of_two():
    n = np.zeros((1, 16), np.uint8)
    n[0, 0] = 0x2 | (0x7 << 4)  # 1.0 and 6.0
    for byte in (1, 2, 100, 127, 128, 200, 254):
        sc = np.full((1, 1), byte, np.uint8)
        d = oracle.dequantize(n, sc, None, MX)
        assert d[0, 0] == 2.0 ** (byte - 127)
        assert d[0, 1] == 6 * 2.0 ** (byte - 127)
    d = oracle.dequantize(n, np.zeros((1, 1), np.uint8), None, MX)
    assert np.all(d == 0)  # reserved byte 0: all elements are zero (Sec. 4.1)


# ---------------------------------------------------------------- paper's numbers
def read_rows(name):
    rows = []
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            rows.append([c.strip() for c in line.split("|")])
    return rows


def test_paper_worked_numbers():
    for label, bm, se, elem, scaled, q in read_rows("paper_worked_numbers.txt"):
        bm, se, elem, scaled, q = float(bm), int(se), float(elem), float(scaled), float(q)
        x = block({0: bm, 1: elem})
        for mode in (MX, MXP):
            nib, sc, idx = oracle.quantize(x, mode)
            assert int(sc[0, 0]) - 127 == se, label
            assert abs(np.float32(elem) / 2.0 ** se - scaled) < 1e-6
            dec = oracle.dequantize(nib, sc, idx, mode)
            got = dec[0, 1] / 2.0 ** se
            assert got == q and math.copysign(1, got) == math.copysign(1, q), label


def test_exponent_of_running_example():
    # "0.99 has exponent -1"; BM in [8, 16) -> shared_exp 1 -> byte 128
    x = block({3: 0.99})
    _, sc, _ = oracle.quantize(x, MXP)
    assert int(sc[0, 0]) - 127 == -1 - 2
    for bm in (8.0, 13.0, 15.99):
        _, sc, _ = oracle.quantize(block({7: bm}), MX)
        assert sc[0, 0] == 128


def parse_kv(s):
    return {int(a.split(":")[0]): float(a.split(":")[1]) for a in s.split(",")}


def test_block_vectors():
    for name, inp, sb, ib, nib_p, nib_m, dec_p, dec_bm_m in read_rows("block_vectors.txt"):
        x = block(parse_kv(inp))
        want_p = bytes.fromhex(nib_p).ljust(16, b"\0")
        want_m = bytes.fromhex(nib_m).ljust(16, b"\0")
        nib, sc, idx = oracle.quantize(x, MXP)
        assert sc[0, 0] == int(sb, 16), name
        assert idx[0, 0] == int(ib, 16), name
        assert bytes(nib[0]) == want_p, (name, bytes(nib[0]).hex())
        dec = oracle.dequantize(nib, sc, idx, MXP)[0]
        want = np.zeros(32)
        for i, v in parse_kv(dec_p).items():
            want[i] = v
        assert np.array_equal(dec, want), name
        nib2, sc2, idx2 = oracle.quantize(x, MX)
        assert sc2[0, 0] == sc[0, 0] and idx2[0, 0] == 0
        assert bytes(nib2[0]) == want_m, (name, bytes(nib2[0]).hex())
        bm = int(ib, 16)
        assert oracle.dequantize(nib2, sc2, None, MX)[0, bm] == float(dec_bm_m)


# ---------------------------------------------------------------- flush rule
def test_flush_rule():
    # floor(log2 BM) <= -127 + emax = -125 -> whole block zero with biased scale 0
    for v in (2.0 ** -125, np.nextafter(np.float32(2.0 ** -124), np.float32(0)), 1e-45, 0.0, -0.0):
        x = block({5: v, 9: -(abs(v) / 2)})
        for mode in (MX, MXP):
            nib, sc, idx = oracle.quantize(x, mode)
            assert sc[0, 0] == 0 and idx[0, 0] == 0 and not nib.any()
            assert np.all(oracle.dequantize(nib, sc, idx, mode) == 0)
    for v in (2.0 ** -124, np.nextafter(np.float32(2.0 ** -124), np.float32(1))):
        nib, sc, idx = oracle.quantize(block({5: v}), MXP)
        assert sc[0, 0] == 1 and idx[0, 0] == 5
    # largest finite fp32: exponent 127 -> byte 127 - 2 + 127 = 252
    _, sc, _ = oracle.quantize(block({0: np.finfo(np.float32).max}), MXP)
    assert sc[0, 0] == 252


def test_scale_is_exponent_field_minus_emax():
    g = np.random.Generator(np.random.PCG64(7))
    x = (g.standard_normal((64, 64)) * np.exp(g.uniform(-60, 60, (64, 1)))).astype(np.float32)
    _, sc, _ = oracle.quantize(x, MXP)
    amax = np.abs(x).reshape(64, 2, 32).max(-1)
    field = (amax.view(np.uint32) >> 23) & 0xFF  # biased exponent of the block max
    assert np.array_equal(sc.astype(np.int64), field.astype(np.int64) - 2)


# ---------------------------------------------------------------- rounding
def all_bf16_upto(limit_bits):
    bits = np.arange(0, limit_bits + 1, dtype=np.uint32)
    return (bits << 16).view(np.float32)


def test_nbm_rounding_every_bf16_value_up_to_8():
    # scale 2^0: put a BM of 4.0 .. wait for values above the BM they would be the BM, so
    # use MXFP4 mode where every element (BM included) takes the plain E2M1 cast.
    vals = all_bf16_upto(0x4100)  # 0 .. 8.0
    vals = vals[vals < 8.0]
    for v in vals:
        x = block({0: 4.0 if v < 4 else float(v), 1: float(v)})
        nib, sc, _ = oracle.quantize(x, MX)
        assert sc[0, 0] == 127
        code = nibble_list(nib[0])[1]
        # independent arithmetic rounding: IEEE round-half-even on the binade's quantum
        q = 0.5 if v < 2 else (1.0 if v < 4 else 2.0)
        r = float(np.rint(np.float64(v) / q) * q)  # numpy rint = ties to even multiple
        r = min(r, 6.0)
        assert E2M1[code & 7] == r, (v, code)
        # nearest-value property, by exact rational search
        dist = [abs(Fraction(float(v)) - Fraction(t)) for t in E2M1]
        assert dist[code & 7] == min(dist)


def test_nbm_tie_points_go_to_even_code():
    ties = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0}
    for v, want in ties.items():
        for sgn in (1, -1):
            x = block({0: 7.5, 1: sgn * v})
            nib, sc, idx = oracle.quantize(x, MXP)
            d = oracle.dequantize(nib, sc, idx, MXP)
            assert d[0, 1] == sgn * want
    # above 5 everything saturates at 6 (7.92 -> 6.0 in the paper's example)
    for v in (5.01, 6.0, 7.0, 7.49):
        x = block({0: 7.5, 1: v})
        nib, sc, idx = oracle.quantize(x, MXP)
        assert oracle.dequantize(nib, sc, idx, MXP)[0, 1] == 6.0


def test_bm_code_every_bf16_and_grid():
    # every bf16 value in [4, 8) at scale 2^0 and at another scale
    bits = np.arange(0x4080, 0x4100, dtype=np.uint32)
    vals = (bits << 16).view(np.float32)
    grid = [4 + m / 2 for m in range(8)]
    for v in vals:
        for sh in (0, -9, 17):
            x = block({11: float(v) * 2.0 ** sh})
            nib, sc, idx = oracle.quantize(x, MXP)
            assert idx[0, 0] == 11 and sc[0, 0] == 127 + sh
            m = nibble_list(nib[0])[11] & 7
            dist = [abs(Fraction(float(v)) - Fraction(t)) for t in grid]
            assert dist[m] == min(dist)
            if dist.count(min(dist)) == 2:  # tie: even mantissa
                assert m % 2 == 0
            # error bounds: quarter step unless clamped at the top
            if v <= 7.75:
                assert abs(grid[m] - float(v)) <= 0.25
            # MX+ never represents the BM worse than MXFP4
            nib4, sc4, _ = oracle.quantize(x, MX)
            d4 = oracle.dequantize(nib4, sc4, None, MX)[0, 11]
            dp = oracle.dequantize(nib, sc, idx, MXP)[0, 11]
            xv = float(x[0, 11])
            assert abs(dp - xv) <= abs(d4 - xv)


def test_bm_representable_values_round_trip_exactly():
    for e in (-100, -3, 0, 5, 90):
        for j in range(8):
            for sgn in (1.0, -1.0):
                v = sgn * 2.0 ** e * (1 + j / 8)
                x = block({17: v, 2: v / 64})
                nib, sc, idx = oracle.quantize(x, MXP)
                assert oracle.dequantize(nib, sc, idx, MXP)[0, 17] == v


def test_bm_tie_points_and_clamp():
    for v, want in {4.25: 4.0, 4.75: 5.0, 5.25: 5.0, 5.75: 6.0, 6.25: 6.0, 6.75: 7.0,
                    7.25: 7.0, 7.75: 7.5, 7.9: 7.5, 7.99: 7.5}.items():
        nib, sc, idx = oracle.quantize(block({0: v}), MXP)
        assert sc[0, 0] == 127  # the scale is never bumped (Sec. 4.1)
        assert oracle.dequantize(nib, sc, idx, MXP)[0, 0] == want


# ---------------------------------------------------------------- invariants
def random_blocks(seed, rows=256, cols=256):
    g = np.random.Generator(np.random.PCG64(seed))
    x = g.standard_normal((rows, cols)).astype(np.float32)
    x *= np.exp(g.uniform(-8, 8, (rows, 1))).astype(np.float32)
    x[:, ::37] *= 30
    x[g.random((rows, cols)) < 0.05] = 0
    return x


def test_mode_relation_and_mxfp4_bm_exponent():
    x = random_blocks(3)
    x[5, 32:64] = 0  # one all-zero block
    nib_m, sc_m, idx_m = oracle.quantize(x, MX)
    nib_p, sc_p, idx_p = oracle.quantize(x, MXP)
    assert np.array_equal(sc_m, sc_p)  # "MX+ does not alter the shared scale"
    assert not idx_m.any() and idx_p.max() < 32  # 5 index bits, 3 reserved zero
    rows, cols = x.shape
    for r in range(rows):
        nm, np_ = nibble_list(nib_m[r]), nibble_list(nib_p[r])
        for b in range(cols // 32):
            bm = int(idx_p[r, b])
            blk = np.abs(x[r, b * 32:(b + 1) * 32])
            if sc_p[r, b] == 0:
                assert not any(nm[b * 32:(b + 1) * 32]) and not any(np_[b * 32:(b + 1) * 32])
                continue
            assert blk[bm] == blk.max() and bm == int(np.argmax(blk))  # first maximum
            for i in range(32):
                if i != bm:  # NBMs are plain E2M1 in both modes
                    assert nm[b * 32 + i] == np_[b * 32 + i]
            # in MXFP4 the BM's exponent field is always 11b (Sec. 4.1)
            assert (nm[b * 32 + bm] & 7) in (6, 7)
            assert nm[b * 32 + bm] >> 3 == np_[b * 32 + bm] >> 3


def test_layout_bits_per_element():
    x = random_blocks(4, 8, 64)
    nib, sc, idx = oracle.quantize(x, MXP)
    n = x.size
    assert 8 * (nib.nbytes + sc.nbytes) / n == 4.25
    assert 8 * (nib.nbytes + sc.nbytes + idx.nbytes) / n == 4.5


def test_nibble_order_and_sign_of_zero():
    x = block({0: 1.0, 1: 2.0, 2: -0.0, 3: -0.01, 31: -6.0})
    nib, sc, idx = oracle.quantize(x, MX)
    assert sc[0, 0] == 127
    assert nib[0, 0] == (0x2 | (0x4 << 4))  # element 0 low nibble, element 1 high nibble
    assert nib[0, 1] == (0x8 | (0x8 << 4))  # -0.0 and a value rounding to zero keep the sign
    assert nib[0, 15] == 0xF0


def test_round_trip_of_representable_blocks():
    g = np.random.Generator(np.random.PCG64(11))
    for _ in range(200):
        se = int(g.integers(-20, 20))
        codes = g.integers(0, 6, 32)  # NBMs strictly below 4 so the BM stays the maximum
        signs = g.choice([-1.0, 1.0], 32)
        y = np.array([E2M1[c] for c in codes]) * signs
        bm = int(g.integers(0, 32))
        y[bm] = (4 + int(g.integers(0, 8)) / 2) * signs[bm]
        y = (y * 2.0 ** se).astype(np.float32)[None, :]
        nib, sc, idx = oracle.quantize(y, MXP)
        assert idx[0, 0] == bm
        assert np.array_equal(oracle.dequantize(nib, sc, idx, MXP), y.astype(np.float64))


def test_eq4_split_exhaustive():
    for m in range(8):
        h, l = oracle.bm_split(m)
        assert E2M1[h] in (4.0, 6.0) and l <= 3
        assert E2M1[h] + E2M1[l] == 4 + m / 2  # BM = BM_H + BM_L, both valid FP4
        assert E2M1[h] == 4 * (1 + (m >> 2) / 2) and E2M1[l] == (m >> 1 & 1) + (m & 1) / 2


# ---------------------------------------------------------------- brute force
PROBE = sorted(set(
    [s * v * sc for v in E2M1 for s in (1, -1) for sc in (1.0, 0.25)]
    + [s * v for v in (0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 7.0) for s in (1, -1)]
    + [4 + m / 2 for m in range(8)] + [4.25, 4.75, 5.25, 6.75, 7.25, 7.75, 7.9, -7.6, -4.4]
    + [0.3, -0.39, 0.99, 2.2, -3.1, 2.0 ** -125, 2.0 ** -124]))


def search_quantize(xs, mode):
    """Second quantizer, by exhaustive search: with the scale and BM fixed by the format
    rules, try every code for every element and keep the nearest decode."""
    k = len(xs)
    a = [abs(Fraction(v)) for v in xs]
    amax = max(a)
    if amax == 0:
        return None
    e = 0  # find e with 2^e <= amax < 2^(e+1) by stepping
    while Fraction(2) ** e > amax:
        e -= 1
    while Fraction(2) ** (e + 1) <= amax:
        e += 1
    if e <= -125:
        return None
    se = e - 2
    bm = a.index(amax)
    dec = []
    for i in range(k):
        grid = [Fraction(4) + Fraction(m, 2) for m in range(8)] if (mode == MXP and i == bm) \
            else [Fraction(t) for t in E2M1]
        r = a[i] / Fraction(2) ** se
        best = min(abs(r - t) for t in grid)
        dec.append((best, [t * Fraction(2) ** se for t in grid if abs(r - t) == best]))
    return se, bm, dec


@pytest.mark.parametrize("k", [2, 4])
def test_tiny_blocks_against_search(k):
    vals = PROBE if k == 2 else PROBE[::5]
    combos = itertools.product(vals, repeat=k) if k == 2 else itertools.islice(
        itertools.product(vals, repeat=k), 0, None, 7)
    xs = np.array(list(combos), np.float32)
    for mode in (MX, MXP):
        nib, sc, idx = oracle.quantize(xs, mode, k=k)
        dec = oracle.dequantize(nib, sc, idx, mode, k=k)
        for r in range(xs.shape[0]):
            ref = search_quantize([float(v) for v in xs[r]], mode)
            if ref is None:
                assert sc[r, 0] == 0 and not nib[r].any()
                continue
            se, bm, cand = ref
            assert sc[r, 0] == se + 127
            if mode == MXP:
                assert idx[r, 0] == bm
            for i in range(k):
                err, allowed = cand[i]
                got = Fraction(float(dec[r, i]))
                assert abs(got) in allowed, (xs[r], i, float(got))
                assert math.copysign(1, dec[r, i]) == math.copysign(1, xs[r, i])


def test_nonfinite_block_is_marked():
    # not defined by the paper (parity unpinned); only the marker is checked
    x = block({3: np.inf})
    nib, sc, idx = oracle.quantize(x, MXP)
    assert sc[0, 0] == 0xFF and not nib.any()
