"""Pins for the channel-reordering oracle (Sec. 8, "Scattering outliers with channel
reordering") and the host-side ordering the library builds; no GPU needed."""
import ctypes

import numpy as np
import pytest

import oracle
from paper_2510_14557_b200 import synth

MX, MXP = 0, 1


def test_order_is_a_permutation_with_heads_first():
    g = synth.rng(3)
    for cols in (32, 64, 96, 4096):
        cnt = g.integers(0, 50, cols)
        order = oracle.channel_order(cnt)
        assert sorted(order.tolist()) == list(range(cols))
        nblk = cols // 32
        heads = order[0::32]
        # the block heads are the nblk channels with the most outliers, in rank order
        ranked = sorted(range(cols), key=lambda c: (-int(cnt[c]), c))
        assert heads.tolist() == ranked[:nblk]
        assert all(cnt[h] >= cnt[c] for h in heads for c in order if c not in set(heads.tolist()))


def test_order_hand_example():
    # 64 channels, two blocks.  Channel 40 has the most outliers, then 3; the 62 others have
    # counts that fall with the channel number except for a tie between 10 and 11.
    cnt = np.zeros(64, np.int64)
    others = [c for c in range(64) if c not in (40, 3)]
    for r, c in enumerate(others):
        cnt[c] = 100 - r
    cnt[11] = cnt[10]                 # tie: 10 stays ahead of 11
    cnt[40], cnt[3] = 1000, 900
    order = oracle.channel_order(cnt)
    assert order[0] == 40 and order[32] == 3
    ranked = [c for c in sorted(others, key=lambda c: (-int(cnt[c]), c))]
    assert ranked.index(10) + 1 == ranked.index(11)
    more, fewer = ranked[:31], ranked[31:]
    assert order[1:32].tolist() == fewer
    assert order[33:64].tolist() == more
    # block 0 (the strongest head) is filled from the quieter half
    assert max(cnt[order[1:32]]) <= min(cnt[order[33:64]])


def test_clustered_outlier_channels_are_scattered():
    # outlier channels all inside the first block: after reordering every block has one
    cols, nblk = 256, 8
    cnt = np.zeros(cols, np.int64)
    cnt[4:4 + nblk] = np.arange(nblk, 0, -1) * 10
    order = oracle.channel_order(cnt)
    hot = set(range(4, 4 + nblk))
    per_block = [sum(1 for c in order[32 * j:32 * j + 32] if c in hot) for j in range(nblk)]
    assert per_block == [1] * nblk


def test_reordering_both_operands_keeps_the_product():
    # integer-valued operands: every partial sum is exact, so the products agree bit for bit
    g = synth.rng(9)
    a = g.integers(-8, 9, (5, 96)).astype(np.float64)
    b = g.integers(-8, 9, (7, 96)).astype(np.float64)
    order = oracle.channel_order(g.integers(0, 9, 96))
    assert np.array_equal(oracle.gemm_fp64(a, b), oracle.gemm_fp64(a[:, order], b[:, order]))


def test_quantize_reordered_is_quantize_of_the_gathered_rows():
    # with the identity ordering nothing changes; with a block-internal reversal the nibbles
    # of a block come out reversed, the scale stays and the BM index mirrors
    g = synth.rng(4)
    x = (g.standard_normal((3, 64)) * np.exp2(g.integers(-3, 4, (3, 64)))).astype(np.float32)
    ident = np.arange(64, dtype=np.int32)
    q0 = oracle.quantize(x, MXP)
    q1 = oracle.quantize_reordered(x, ident, MXP)
    assert all(np.array_equal(u, v) for u, v in zip(q0, q1))
    rev = np.concatenate([np.arange(31, -1, -1), np.arange(63, 31, -1)]).astype(np.int32)
    q2 = oracle.quantize_reordered(x, rev, MXP)
    assert np.array_equal(q2[1], q0[1])
    d0 = oracle.dequantize(q0[0], q0[1], q0[2], MXP)
    d2 = oracle.dequantize(q2[0], q2[1], q2[2], MXP)
    # unique maxima (continuous data): the same element is the BM, so values just move
    assert np.array_equal(d2, d0[:, rev])
    assert np.array_equal(q2[2] & 31, 31 - (q0[2] & 31))


def test_library_order_matches_the_oracle():
    from paper_2510_14557_b200 import binding
    g = synth.rng(12)
    for cols in (32, 64, 160, 4096):
        for hi in (2, 40):   # many ties / few ties
            cnt = g.integers(0, hi, cols)
            got = binding.mxp_channel_order(cnt).numpy()
            assert np.array_equal(got, oracle.channel_order(cnt))
    with pytest.raises(binding.MxpError):
        binding.mxp_channel_order(np.zeros(48, np.int64))
