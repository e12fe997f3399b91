"""GPU parity: mxp_quantize / mxp_dequantize through the C ABI vs the CPU oracle (bit-exact)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import bf16_round, packed_to_host, host_to_packed, to_dev, to_dev_bf16
from paper_2510_14557_b200 import synth

pytestmark = pytest.mark.gpu
MX, MXP, MXPP = 0, 1, 2   # MXPP: MX++ (Sec. 4.3)


def mxp():
    import paper_2510_14557_b200 as m
    return m


def assert_planes_equal(p, ref, mode, what=""):
    nib, sc, idx = packed_to_host(p)
    rn, rs, ri = ref
    assert np.array_equal(sc, rs), "scales differ " + what
    assert np.array_equal(nib, rn), "nibbles differ %s (%d bytes)" % (what, int((nib != rn).sum()))
    if mode != MX:
        assert np.array_equal(idx, ri), "indices differ " + what


def adversarial_f32():
    """Blocks that hit every branch: ties, saturation, flush boundary, equal maxima, zeros."""
    rows = []
    ties = [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 7.0, 4.25, 4.75, 5.25, 5.75, 6.25, 6.75, 7.25, 7.75]
    for sh in (0, -7, 30, -120, 120):
        for pos in (0, 1, 7, 8, 15, 16, 30, 31):
            b = np.zeros(32, np.float32)
            b[pos] = 7.5
            for i, v in enumerate(ties):
                b[(pos + 1 + i) % 32] = v * (-1) ** i
            rows.append(b * np.float32(2.0 ** sh))
    for bm in ties + [4.0, 6.0, 7.9, 7.99, 3.999, 15.9, 8.5, 9.5]:
        for pos in (3, 12, 29):
            b = np.full(32, 0.3, np.float32)
            b[pos] = -bm
            rows.append(b)
    b = np.zeros(32, np.float32); rows.append(b.copy())                      # all zero
    b[5] = 2.0 ** -125; rows.append(b.copy())                                # flushed
    b[5] = 2.0 ** -124; b[6] = 2.0 ** -126; rows.append(b.copy())            # smallest kept
    b = np.zeros(32, np.float32); b[0] = 6.0; b[1] = -6.0; b[31] = 6.0; rows.append(b.copy())
    b = np.full(32, -0.0, np.float32); b[9] = 1e-3; rows.append(b.copy())    # signed zeros
    b = np.full(32, 1e-41, np.float32); rows.append(b.copy())                # subnormals
    b = np.full(32, 3.0e38, np.float32); b[4] = np.finfo(np.float32).max; rows.append(b.copy())
    b = np.ones(32, np.float32); b[17] = np.inf; rows.append(b.copy())       # marker only
    b = np.ones(32, np.float32); b[2] = np.nan; rows.append(b.copy())
    x = np.stack(rows)
    pad = (-x.shape[0]) % 4
    x = np.concatenate([x, np.zeros((pad, 32), np.float32)])
    return x.reshape(-1, 128)  # four blocks per row


@pytest.mark.parametrize("mode", [MX, MXP, MXPP])
def test_config1_fp32_bit_exact(mode):
    a, b = synth.config1()
    for x in (a, b):
        p = mxp().mxp_quantize(to_dev(x), mode)
        assert_planes_equal(p, oracle.quantize(x, mode), mode)


@pytest.mark.parametrize("mode", [MX, MXP, MXPP])
def test_adversarial_blocks_fp32_and_bf16(mode):
    x = adversarial_f32()
    p = mxp().mxp_quantize(to_dev(x), mode)
    assert_planes_equal(p, oracle.quantize(x, mode), mode, "fp32")
    bits = synth.f32_to_bf16_bits(np.nan_to_num(x, nan=0.0, posinf=3e38, neginf=-3e38))
    p = mxp().mxp_quantize(to_dev_bf16(bits), mode)
    assert_planes_equal(p, oracle.quantize(bits, mode, bf16_bits=True), mode, "bf16")


@pytest.mark.parametrize("mode", [MX, MXP, MXPP])
def test_every_bf16_pattern_as_block_max(mode):
    # all 65536 bf16 bit patterns, each once as the first element of a block
    bits = np.zeros((2048, 32 * 32), np.uint16)
    allp = np.arange(65536, dtype=np.uint16).reshape(2048, 32)
    bits[:, ::32] = allp
    bits[:, 1::32] = 0x3E80  # 0.25
    bits[:, 5::32] = 0xBF40  # -0.75
    p = mxp().mxp_quantize(to_dev_bf16(bits), mode)
    assert_planes_equal(p, oracle.quantize(bits, mode, bf16_bits=True), mode)


@pytest.mark.parametrize("shape", [(1, 32), (3, 96), (5, 8192), (257, 2080), (1000, 32), (64, 4096)])
@pytest.mark.parametrize("mode", [MX, MXP, MXPP])
def test_ragged_sizes_bf16(shape, mode):
    bits = synth.config2(shape[0], shape[1], seed=shape[0] + shape[1])
    p = mxp().mxp_quantize(to_dev_bf16(bits), mode)
    assert_planes_equal(p, oracle.quantize(bits, mode, bf16_bits=True), mode, str(shape))


def test_strided_source_and_guard_bytes():
    m = mxp()
    x = synth.activations_normal(37, 256, seed=9)
    wide = torch.zeros((37, 384), dtype=torch.float32, device="cuda")
    wide[:, :256] = to_dev(x)
    out = m.alloc_packed(37 + 1, 256, MXP)  # one spare row as a canary
    for t in (out.nibbles, out.scales, out.bm_index):
        t.fill_(0xA5)
    view = m.Packed(out.nibbles[:37], out.scales[:37], out.bm_index[:37], 37, 256, MXP)
    m.mxp_quantize(wide[:, :256], MXP, out=view)
    assert_planes_equal(view, oracle.quantize(x, MXP), MXP)
    for t in (out.nibbles, out.scales, out.bm_index):
        assert bool((t[37] == 0xA5).all())


def test_mxfp4_mode_zero_fills_a_given_index_plane():
    m = mxp()
    x = synth.activations_normal(16, 128, seed=2)
    out = m.alloc_packed(16, 128, MX, index_for_mxfp4=True)
    out.bm_index.fill_(7)
    m.mxp_quantize(to_dev(x), MX, out=out)
    assert int(out.bm_index.sum()) == 0


def test_empty_input_is_a_no_op():
    m = mxp()
    x = torch.empty((0, 64), dtype=torch.bfloat16, device="cuda")
    p = m.mxp_quantize(x, MXP)
    assert p.nibbles.numel() == 0


@pytest.mark.parametrize("mode", [MX, MXP, MXPP])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_dequantize_bit_exact(mode, dtype):
    m = mxp()
    x = np.concatenate([adversarial_f32()[:, :128], synth.activations_normal(64, 128, seed=5)])
    x = np.nan_to_num(x, nan=0.0, posinf=3e38, neginf=-3e38)
    nib, sc, idx = oracle.quantize(x, mode)
    ref = oracle.dequantize(nib, sc, idx, mode)
    got = m.mxp_dequantize(host_to_packed(nib, sc, idx if mode != MX else None, mode), dtype)
    g = got.float().cpu().numpy().astype(np.float64)
    # decode is exact in both output types, signed zeros included (MX++ NBMs of blocks at the
    # very bottom of the range fall below bf16's subnormal grid: nearest-even there)
    if mode == MXPP and dtype == torch.bfloat16:
        ref = bf16_round(ref)
    assert np.array_equal(g, ref)
    assert np.array_equal(np.signbit(g), np.signbit(ref))


def test_dequantize_all_codes_every_position():
    m = mxp()
    rows = []
    for pos in range(32):
        for nibv in range(16):
            rows.append((pos, nibv))
    nib = np.zeros((len(rows), 16), np.uint8)
    idx = np.zeros((len(rows), 1), np.uint8)
    sc = np.zeros((len(rows), 1), np.uint8)
    for r, (pos, nibv) in enumerate(rows):
        nib[r, :] = 0x21  # 0.5 / 1.0 background
        byte = nib[r, pos // 2]
        nib[r, pos // 2] = (byte & 0x0F) | (nibv << 4) if pos & 1 else (byte & 0xF0) | nibv
        idx[r, 0] = pos | 0xE0  # reserved bits set: must be ignored
        sc[r, 0] = [1, 126, 127, 130, 252, 0][r % 6]  # 252: largest byte the quantizer emits
    for mode in (MX, MXP, MXPP):   # in MX++ mode the top index bits are delta = 7
        ref = oracle.dequantize(nib, sc, idx, mode)
        got = m.mxp_dequantize(host_to_packed(nib, sc, idx, mode), torch.float32)
        assert np.array_equal(got.cpu().numpy().astype(np.float64), ref)


def test_mxpp_second_maximum_cases():
    # MX++ (Sec. 4.3): blocks that exercise the NBM exponent: maximum occurring twice,
    # NBMs all zero, NBM maximum in every binade below the BM, subnormal NBMs, tiny blocks
    rows = []
    for sh in (0, 40, -40, -110, -118, 100):
        for gap in range(0, 12):
            b = np.zeros(32, np.float32)
            b[7] = -1.75
            b[20] = 1.3 * 2.0 ** -gap
            b[21] = -0.9 * 2.0 ** -gap
            b[3] = 0.11 * 2.0 ** -gap
            rows.append(b * np.float32(2.0 ** sh))
    b = np.zeros(32, np.float32); b[9] = 5.0; rows.append(b.copy())                 # NBMs all zero
    b[30] = 5.0; rows.append(b.copy())                                              # maximum twice
    b = np.zeros(32, np.float32); b[0] = 2.0 ** -100; b[1] = 1e-41; rows.append(b.copy())  # subnormal NBM
    b = np.zeros(32, np.float32); b[0] = 2.0 ** -121; b[1] = 2.0 ** -127; rows.append(b.copy())
    x = np.stack(rows)
    x = np.concatenate([x, np.zeros(((-x.shape[0]) % 4, 32), np.float32)]).reshape(-1, 128)
    p = mxp().mxp_quantize(to_dev(x), MXPP)
    ref = oracle.quantize(x, MXPP)
    assert_planes_equal(p, ref, MXPP, "fp32")
    assert int((ref[2] >> 5).max()) == 7 and int((ref[2] >> 5).min()) == 0
    bits = synth.f32_to_bf16_bits(x)
    p = mxp().mxp_quantize(to_dev_bf16(bits), MXPP)
    assert_planes_equal(p, oracle.quantize(bits, MXPP, bf16_bits=True), MXPP, "bf16")
    wide = torch.zeros((x.shape[0], 256), dtype=torch.bfloat16, device="cuda")      # strided bf16
    wide[:, :128] = to_dev_bf16(bits)
    p = mxp().mxp_quantize(wide[:, :128], MXPP)
    assert_planes_equal(p, oracle.quantize(bits, MXPP, bf16_bits=True), MXPP, "bf16 strided")
    got = mxp().mxp_dequantize(p, torch.float32).cpu().numpy().astype(np.float64)
    assert np.array_equal(got, oracle.dequantize(*oracle.quantize(bits, MXPP, bf16_bits=True), MXPP))
