"""Pins for the oracle's MX++ variant (Sec. 4.3): NBMs get their own shared exponent, its
distance delta from the BM's stored in the three reserved bits of the index byte (no GPU).

Checked against the paper's worked numbers, a search restatement of "smallest exponent that
cannot saturate", invariants that follow from the definition, and special cases that reduce
to the (separately pinned) MX+ encoder.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import MODE_MXFP4_PLUS as MXP, MODE_MXFP4_PP as MXPP

GOLD = os.path.join(os.path.dirname(__file__), "golden")
E2M1 = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


def block(vals: dict, k=32):
    x = np.zeros((1, k), np.float32)
    for i, v in vals.items():
        x[0, i] = v
    return x


def delta_of(q):
    return int(q[2][0, 0]) >> 5


def test_paper_worked_numbers():
    rows = [l.split("|") for l in open(os.path.join(GOLD, "paper_mxpp_worked_numbers.txt"))
            if l.strip() and not l.startswith("#")]
    # the running example: BM with shared_exp 1 (a value in [8, 16)), NBMs 0.99 and -0.39
    x = block({0: 13.0, 1: 0.99, 2: -0.39})
    q = oracle.quantize(x, MXPP)
    assert int(q[1][0, 0]) - 127 == 1            # the scale byte keeps the BM's shared_exp
    se_new = 1 - delta_of(q)
    dec = oracle.dequantize(*q, MXPP)[0]
    for label, se, se_nbm, elem, scaled, quant in rows:
        label = label.strip()
        se, se_nbm, elem, scaled, quant = int(se), int(se_nbm), float(elem), float(scaled), float(quant)
        assert se == 1
        assert math.isclose(elem / 2.0 ** se_nbm, scaled, rel_tol=1e-9)
        if label == "no_offset_saturates":
            # what the offset of 1 prevents: at exponent -3 the value would exceed 6
            assert se_nbm == se_new - 1 and scaled > 6.0 and quant == 6.0
        else:
            assert se_nbm == se_new
            got = dec[1] if elem > 0 else dec[2]
            assert got == quant * 2.0 ** se_nbm
    assert dec[0] == 13.0                         # the BM is decoded with its own shared_exp


def test_delta_is_smallest_exponent_that_cannot_saturate():
    # Sec. 4.3 calls e "the smallest feasible shared exponent for NBMs to avoid saturation".
    # Search restatement: the smallest e' for which every value of the largest NBM's binade,
    # divided by 2^e', stays within the largest E2M1 magnitude (6); then clip to [se - 7, se].
    g = np.random.default_rng(0)
    for _ in range(400):
        bm_exp = int(g.integers(-20, 20))
        nbm_exp = bm_exp - int(g.integers(0, 12))
        bm = float(np.float32(2.0 ** bm_exp * g.uniform(1.0, 1.99)))
        nbm = float(np.float32(2.0 ** nbm_exp * g.uniform(1.0, 1.99)))
        if nbm >= bm:
            continue
        x = block({3: bm, 7: -nbm, 9: nbm / 3})
        q = oracle.quantize(x, MXPP)
        se = int(q[1][0, 0]) - 127
        binade_top = Fraction(2) ** (math.floor(math.log2(nbm)) + 1)
        e = None
        for cand in range(se - 40, se + 3):       # ascending: first feasible is the smallest
            if binade_top / Fraction(2) ** cand <= 6:
                e = cand
                break
        want = min(max(e, se - 7), se)
        assert se - delta_of(q) == want
        assert (int(q[2][0, 0]) & 31) == 3


@pytest.mark.parametrize("seed", range(4))
def test_invariants_against_mx_plus(seed):
    g = np.random.default_rng(seed)
    x = (g.standard_normal((64, 128)) * np.exp2(g.integers(-6, 6, (64, 1)))).astype(np.float32)
    x[:, ::17] *= 40.0                                   # outliers: large delta in many blocks
    qp = oracle.quantize(x, MXP)
    qq = oracle.quantize(x, MXPP)
    # scale plane and BM position are those of MX+ ("MX++ decouples the NBMs' scale")
    assert np.array_equal(qp[1], qq[1])
    assert np.array_equal(qp[2], qq[2] & 31)
    delta = qq[2] >> 5
    assert delta.min() >= 0 and delta.max() <= 7 and delta.max() >= 3
    dp = oracle.dequantize(*qp, MXP)
    dq = oracle.dequantize(*qq, MXPP)
    xd = x.astype(np.float64)
    # the BM decodes as in MX+; every NBM is at least as close as in MX+ (finer grid that
    # contains the coarse grid's points below its own maximum, and no saturation)
    rows, cols = x.shape
    bmcol = (np.arange(cols // 32)[None, :] * 32 + (qq[2] & 31)).astype(np.int64)
    r = np.arange(rows)[:, None]
    assert np.array_equal(dp[r, bmcol], dq[r, bmcol])
    assert np.all(np.abs(dq - xd) <= np.abs(dp - xd) + 1e-300)
    assert np.abs(dq - xd).sum() < 0.9 * np.abs(dp - xd).sum()   # and clearly closer overall
    # blocks with delta == 0 are encoded exactly as in MX+
    same = np.repeat(delta == 0, 16, axis=1)
    assert np.array_equal(qp[0][same], qq[0][same])


def test_no_nbm_saturates_unless_clipped_at_the_top():
    g = np.random.default_rng(5)
    x = (g.standard_normal((32, 256)) * 3).astype(np.float32)
    q = oracle.quantize(x, MXPP)
    delta = (q[2] >> 5).astype(np.int64)
    dec = oracle.dequantize(*q, MXPP)
    se_nbm = q[1].astype(np.int64) - 127 - delta
    scaled = np.abs(dec) / np.exp2(np.repeat(se_nbm, 32, axis=1))
    bm = np.zeros_like(dec, dtype=bool)
    rows, cols = x.shape
    bm[np.arange(rows)[:, None], np.arange(cols // 32)[None, :] * 32 + (q[2] & 31)] = True
    nbm_max = np.where(bm, 0, scaled).reshape(rows, cols // 32, 32).max(axis=2)
    # with the offset of 1 the largest NBM lands in [2, 4] on its grid (4 by rounding up)
    assert np.all(nbm_max[delta > 0] <= 4.0)
    assert np.all(nbm_max[(delta > 0) & (delta < 7)] >= 2.0)


def test_special_cases():
    # largest NBM in the BM's binade: e exceeds shared_exp, the upper clip gives delta 0
    q = oracle.quantize(block({0: 13.0, 1: 11.0, 2: 0.3}), MXPP)
    assert delta_of(q) == 0
    assert np.array_equal(q[0], oracle.quantize(block({0: 13.0, 1: 11.0, 2: 0.3}), MXP)[0])
    # nothing but zeros beside the BM: lower clip
    q = oracle.quantize(block({4: -5.0}), MXPP)
    assert delta_of(q) == 7 and (int(q[2][0, 0]) & 31) == 4
    assert oracle.dequantize(*q, MXPP)[0, 4] == -5.0
    # NBMs more than 7 binades below what the BM's scale gives: lower clip, delta 7
    q = oracle.quantize(block({0: 1024.0, 1: 2.0 ** -9}), MXPP)
    assert delta_of(q) == 7
    # representable blocks round-trip: BM 2^3 * 1.625, NBMs on the grid of exponent se - 4
    se = 3 - 2
    vals = {0: 13.0}
    for i, c in enumerate([0.5, 1.0, 1.5, 2.0, 3.0, -3.5]):
        vals[i + 1] = c * 2.0 ** (se - 4)
    vals[6] = -3.0 * 2.0 ** (se - 4)                    # replace the unrepresentable -3.5
    x = block(vals)
    q = oracle.quantize(x, MXPP)
    assert delta_of(q) == 4                             # largest NBM 3 * 2^-3: exponent -2, e = -3
    assert np.array_equal(oracle.dequantize(*q, MXPP), x.astype(np.float64))
    # flushed block: all-zero bytes, delta bits included
    q = oracle.quantize(block({5: 2.0 ** -125, 6: 2.0 ** -140}), MXPP)
    assert int(q[1][0, 0]) == 0 and int(q[2][0, 0]) == 0 and not q[0].any()
