"""GPU parity: mxp_quantize_reordered through the C ABI vs the oracle's definition
quantize(x[:, order]) (bit-exact) (Sec. 8, "Scattering outliers with channel reordering")."""
import numpy as np
import pytest
import torch

import oracle
from helpers import packed_to_host, to_dev, to_dev_bf16
from paper_2510_14557_b200 import synth

pytestmark = pytest.mark.gpu
MX, MXP, MXPP = 0, 1, 2


def mxp():
    import paper_2510_14557_b200 as m
    return m


def check(p, ref, mode):
    nib, sc, idx = packed_to_host(p)
    assert np.array_equal(sc, ref[1])
    assert np.array_equal(nib, ref[0])
    if mode != MX:
        assert np.array_equal(idx, ref[2])


def outlier_order(x_f32):
    """Ordering from the data the way the passage describes: outliers counted per channel."""
    thr = 3.0 * x_f32.std()
    return oracle.channel_order((np.abs(x_f32) > thr).sum(axis=0))


@pytest.mark.parametrize("mode", [MX, MXP, MXPP])
@pytest.mark.parametrize("rows,cols", [(1, 32), (3, 96), (64, 4096), (33, 1056), (129, 8192)])
def test_reordered_bf16_bit_exact(rows, cols, mode):
    bits = synth.f32_to_bf16_bits(synth.activations_normal(rows, cols, rows + cols, 0.01, 30.0))
    x = oracle.bf16_bits_to_f64(bits).astype(np.float32)
    for order in (outlier_order(x), synth.rng(cols).permutation(cols).astype(np.int32)):
        ref = oracle.quantize_reordered(bits, order, mode, bf16_bits=True)
        p = mxp().mxp_quantize_reordered(to_dev_bf16(bits), torch.from_numpy(order).cuda(), mode)
        check(p, ref, mode)


@pytest.mark.parametrize("mode", [MX, MXP, MXPP])
def test_reordered_fp32_strided_bit_exact(mode):
    rows, cols, ld = 37, 320, 352
    g = synth.rng(8)
    full = (g.standard_normal((rows, ld)) * np.exp2(g.integers(-20, 20, (rows, ld)))).astype(np.float32)
    full[:, 7] *= 64.0      # an outlier channel
    x = full[:, :cols]
    order = outlier_order(x)
    ref = oracle.quantize_reordered(x, order, mode)
    p = mxp().mxp_quantize_reordered(to_dev(full)[:, :cols], torch.from_numpy(order).cuda(), mode)
    check(p, ref, mode)


@pytest.mark.parametrize("mode", [MX, MXP])
def test_reordered_rows_that_are_only_element_aligned(mode):
    # a view that starts one element into the rows: no 16-byte row loads, channels are
    # fetched one by one from global memory
    rows, cols = 19, 224
    bits = synth.f32_to_bf16_bits(synth.activations_normal(rows, cols + 8, 77, 0.02, 30.0))
    order = synth.rng(1).permutation(cols).astype(np.int32)
    ref = oracle.quantize_reordered(bits[:, 1:1 + cols], order, mode, bf16_bits=True)
    p = mxp().mxp_quantize_reordered(to_dev_bf16(bits)[:, 1:1 + cols], torch.from_numpy(order).cuda(), mode)
    check(p, ref, mode)


def test_identity_order_equals_plain_quantize_and_bad_entries_are_clamped():
    m = mxp()
    bits = synth.f32_to_bf16_bits(synth.activations_normal(16, 256, 5, 0.01, 30.0))
    xd = to_dev_bf16(bits)
    ident = torch.arange(256, dtype=torch.int32, device="cuda")
    a, b = m.mxp_quantize(xd, MXP), m.mxp_quantize_reordered(xd, ident, MXP)
    assert torch.equal(a.nibbles, b.nibbles) and torch.equal(a.scales, b.scales)
    assert torch.equal(a.bm_index, b.bm_index)
    bad = ident.clone()
    bad[5], bad[200] = 100000, -1          # read as unsigned: both clamp to the last channel
    want = np.arange(256)
    want[5] = want[200] = 255
    ref = oracle.quantize_reordered(bits, want, MXP, bf16_bits=True)
    check(m.mxp_quantize_reordered(xd, bad, MXP), ref, MXP)


def test_reordered_rejects_wide_modes_and_misaligned_order():
    m = mxp()
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    order = torch.arange(68, dtype=torch.int32, device="cuda")
    with pytest.raises(m.MxpError) as e:
        m.mxp_quantize_reordered(x, order[:64], m.MODE_MXFP6_PLUS)
    assert e.value.status == 2
    with pytest.raises(m.MxpError) as e:
        m.mxp_quantize_reordered(x, order[1:65], MXP)   # 4 bytes off a 16-byte boundary
    assert e.value.status == 1


def test_reordering_raises_the_share_of_outliers_kept_as_bm():
    # what the reordering is for: with outliers concentrated in a few channels of one block,
    # more of them become a block's BM (and are kept at 3 mantissa bits) after reordering
    rows, cols = 64, 1024
    g = synth.rng(21)
    x = g.standard_normal((rows, cols)).astype(np.float32)
    hot = np.arange(8, 24)
    x[:, hot] *= 40.0
    bits = synth.f32_to_bf16_bits(x)
    xb = oracle.bf16_bits_to_f64(bits)
    order = outlier_order(x)
    m = mxp()
    plain = m.mxp_dequantize(m.mxp_quantize(to_dev_bf16(bits), MXP)).cpu().numpy().astype(np.float64)
    reo = m.mxp_dequantize(m.mxp_quantize_reordered(to_dev_bf16(bits), torch.from_numpy(order).cuda(), MXP))
    reo = reo.cpu().numpy().astype(np.float64)
    err_plain = np.abs(plain - xb)[:, hot].mean()
    err_reo = np.abs(reo - xb[:, order])[:, np.isin(order, hot)].mean()
    assert err_reo < 0.7 * err_plain
