"""GPU parity: mxp_gemm through the C ABI vs the oracle's fp64 product of decoded operands."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_gemm, host_to_packed, to_dev, to_dev_bf16
from paper_2510_14557_b200 import synth

pytestmark = pytest.mark.gpu
MX, MXP = 0, 1


def mxp():
    import paper_2510_14557_b200 as m
    return m


@pytest.fixture
def force():
    """Forces a kernel choice for the duration of a test (mxp_debug_override)."""
    m = mxp()
    knobs = {"inplace": m.KNOB_INPLACE_KERNEL, "halves": m.KNOB_STREAM_HALVES, "weight_only": m.KNOB_WEIGHT_ONLY_KERNEL,
             "one_sided": m.KNOB_ONE_SIDED}
    names = {"single": 1, "pair": 2, "old": 1, "stream": 2, "1": 1, "2": 2, "wide": 1}
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


# ------------------------------------------------------------------ weight-only form
@pytest.mark.parametrize("wmode", [MX, MXP])
@pytest.mark.parametrize("M,N,K", [(1, 64, 128), (8, 48, 256), (16, 100, 4096), (5, 17, 96),
                                   (16, 33, 32), (40, 64, 512)])
def test_weight_only_small(M, N, K, wmode):
    a_bits, w_bits = synth.config3(M, N, K, seed=M + N + K)
    wp, dw = quantized(w_bits, wmode, bf16=True)
    da = oracle.bf16_bits_to_f64(a_bits)
    for dt in (torch.float32, torch.bfloat16):
        d = mxp().mxp_gemm(to_dev_bf16(a_bits), wp, out_dtype=dt)
        check_gemm(d, da, dw)


def test_weight_only_extreme_scales_and_one_hot():
    # one-hot activations select single decoded weights: exact equality in fp32
    K, N = 128, 32
    g = synth.rng(5)
    w = g.standard_normal((N, K)).astype(np.float32)
    w *= np.exp2(g.integers(-100, 100, (N, 1))).astype(np.float32)
    w[3, 32:64] = 0
    wp, dw = quantized(w, MXP)
    a = np.zeros((16, K), np.float32)
    for m in range(16):
        a[m, (m * 9) % K] = 1.0
    d = mxp().mxp_gemm(to_dev_bf16(synth.f32_to_bf16_bits(a)), wp, out_dtype=torch.float32)
    got = d.cpu().numpy().astype(np.float64)
    for m in range(16):
        assert np.array_equal(got[m], dw[:, (m * 9) % K])


@pytest.mark.parametrize("M", [1, 8, 16])
def test_weight_only_config3_sampled(M):
    a_bits, w_bits = synth.config3(M)
    wq = oracle.quantize(w_bits, MXP, bf16_bits=True)
    m = mxp()
    # encodings of the full weight matrix are bit-exact
    p = m.mxp_quantize(to_dev_bf16(w_bits), MXP)
    assert torch.equal(p.nibbles.cpu(), torch.from_numpy(wq[0]))
    assert torch.equal(p.scales.cpu(), torch.from_numpy(wq[1]))
    assert torch.equal(p.bm_index.cpu(), torch.from_numpy(wq[2]))
    d = m.mxp_gemm(to_dev_bf16(a_bits), p, out_dtype=torch.bfloat16)
    rows = np.unique(np.concatenate([np.arange(0, 11008, 97), [11007, 11006, 5503]]))
    dw = oracle.dequantize(wq[0][rows], wq[1][rows], wq[2][rows], MXP)
    da = oracle.bf16_bits_to_f64(a_bits)
    check_gemm(d[:, torch.from_numpy(rows).cuda()], da, dw)


@pytest.mark.parametrize("kernel", ["old", "stream"])
@pytest.mark.parametrize("wmode", [MX, MXP, 2])
@pytest.mark.parametrize("M,N,K", [(1, 32, 256), (3, 48, 2304), (8, 160, 4352), (9, 64, 512),
                                   (16, 2384, 4096), (40, 64, 768), (5, 77, 1024), (16, 300, 512),
                                   (1, 19000, 512), (1, 11008, 4096), (7, 20000, 1536),
                                   (2, 300, 512), (3, 2384, 4096), (4, 40000, 1024), (1, 64, 8192)])
def test_weight_only_both_kernels(M, N, K, wmode, kernel, force):
    # shapes the streamed kernel takes (N % 16 == 0, K % 256 == 0): several 2048-element stages,
    # a ragged last stage, more row groups than SMs, one and two 8-column activation tiles
    # (every other shape falls through to the general kernel)
    force("weight_only", kernel)
    a_bits, w_bits = synth.config3(M, N, K, seed=M + N + K)
    wp, dw = quantized(w_bits, wmode, bf16=True)
    da = oracle.bf16_bits_to_f64(a_bits)
    for dt in (torch.float32, torch.bfloat16):
        d = mxp().mxp_gemm(to_dev_bf16(a_bits), wp, out_dtype=dt)
        check_gemm(d, da, dw)


@pytest.mark.parametrize("wmode", [MXP, 2])
@pytest.mark.parametrize("M,N,K", [(1, 48, 2304), (2, 160, 4352), (3, 2384, 4096), (8, 64, 512),
                                   (5, 20000, 1536), (1, 64, 8192)])
def test_weight_only_bm_by_correction_warps_or_by_patch(M, N, K, wmode, force):
    # the streamed kernel's two ways of handling the BM: correction warps for M <= 2, patched
    # fragments above
    force("weight_only", "stream")
    a_bits, w_bits = synth.config3(M, N, K, seed=M + N + K + 1)
    wp, dw = quantized(w_bits, wmode, bf16=True)
    da = oracle.bf16_bits_to_f64(a_bits)
    for dt in (torch.float32, torch.bfloat16):
        check_gemm(mxp().mxp_gemm(to_dev_bf16(a_bits), wp, out_dtype=dt), da, dw)


@pytest.mark.parametrize("kernel", ["old", "stream"])
def test_weight_only_one_hot_and_scale_spread(kernel, force):
    # one-hot activations select single decoded weights (exact in fp32), with weight rows and
    # activation rows spread over 60 binades each, a flushed block and a zero block
    force("weight_only", kernel)
    K, N = 512, 48
    g = synth.rng(11)
    w = g.standard_normal((N, K)).astype(np.float32)
    w *= np.exp2(g.integers(-30, 30, (N, 1))).astype(np.float32)
    w[3, 32:64] = 0
    w[5, 64:96] = 1e-44
    wp, dw = quantized(w, MXP)
    a = np.zeros((16, K), np.float32)
    for m in range(16):
        a[m, (m * 37) % K] = 2.0 ** (4 * m - 30)
    d = mxp().mxp_gemm(to_dev_bf16(synth.f32_to_bf16_bits(a)), wp, out_dtype=torch.float32)
    got = d.cpu().numpy().astype(np.float64)
    for m in range(16):
        want = (dw[:, (m * 37) % K] * 2.0 ** (4 * m - 30)).astype(np.float32).astype(np.float64)
        assert np.array_equal(got[m], want)


@pytest.mark.parametrize("wmode", [MX, MXP, 2])
@pytest.mark.parametrize("M,NK,layers", [(1, 1024, 6), (8, 4096, 4), (16, 2048, 5)])
def test_weight_only_chained_layers(M, NK, layers, wmode):
    # A chain of decode GEMMs launched as programmatic dependents: layer i's output is layer
    # i+1's activation, so a grid that read its input (or wrote its output) before the previous
    # one had finished would show.  First layer against the oracle; the whole chain bit for bit
    # against the same chain of ordinary launches, eagerly and replayed from a CUDA graph.
    m = mxp()
    a_bits, _ = synth.config3(M, 16, NK, seed=NK + M)
    ws, decs = [], []
    for i in range(layers):
        _, w_bits = synth.config3(1, NK, NK, seed=100 + i)
        wp, dw = quantized(w_bits, wmode, bf16=True)
        ws.append(wp)
        decs.append(dw)
    a0 = to_dev_bf16(a_bits)
    status = torch.zeros(16, dtype=torch.uint8, device="cuda")

    def chain(fn):
        bufs = [torch.zeros((M, NK), dtype=torch.bfloat16, device="cuda") for _ in range(layers)]
        x = a0
        for i in range(layers):
            fn(x, ws[i], bufs[i])
            x = bufs[i]
        return bufs

    plain = chain(lambda x, w, o: m.mxp_gemm(x, w, out=o))
    chained = chain(lambda x, w, o: m.mxp_gemm_decode_chained(x, w, o, status))
    torch.cuda.synchronize()
    assert m.mxp_gemm_status(status) == 0
    check_gemm(chained[0], oracle.bf16_bits_to_f64(a_bits), decs[0])
    for p_, c_ in zip(plain, chained):
        assert torch.equal(p_.view(torch.int16), c_.view(torch.int16))

    # the same chain captured: the launches become programmatic dependency edges
    bufs = [torch.zeros((M, NK), dtype=torch.bfloat16, device="cuda") for _ in range(layers)]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        x = a0
        for i in range(layers):
            m.mxp_gemm_decode_chained(x, ws[i], bufs[i], status)
            x = bufs[i]
    torch.cuda.current_stream().wait_stream(side)
    for b_ in bufs:
        b_.zero_()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        x = a0
        for i in range(layers):
            m.mxp_gemm_decode_chained(x, ws[i], bufs[i], status)
            x = bufs[i]
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert m.mxp_gemm_status(status) == 0
    for p_, c_ in zip(plain, bufs):
        assert torch.equal(p_.view(torch.int16), c_.view(torch.int16))


def test_weight_only_chained_rejects_what_it_cannot_run():
    m = mxp()
    a_bits, w_bits = synth.config3(4, 24, 256, seed=3)  # N % 16 != 0
    wp, _ = quantized(w_bits, MXP, bf16=True)
    out = torch.zeros((4, 24), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(m.MxpError) as e:
        m.mxp_gemm_decode_chained(to_dev_bf16(a_bits), wp, out)
    assert e.value.status == 2


# ------------------------------------------------------------------ weight-only form, prefill sizes
@pytest.mark.parametrize("wmode", [MX, MXP, 2])
@pytest.mark.parametrize("M,N,K", [(65, 128, 128), (128, 520, 1024), (300, 1000, 384), (513, 129, 2048)])
def test_weight_only_many_rows_on_the_tensor_cores(M, N, K, wmode):
    # more than 64 activation rows: bf16 activations enter the block-scaled tensor-core kernel as
    # two E4M3 planes (hi + lo) with a power-of-two scale per block of 32
    a_bits, w_bits = synth.config3(M, N, K, seed=M + N + K)
    wp, dw = quantized(w_bits, wmode, bf16=True)
    da = oracle.bf16_bits_to_f64(a_bits)
    m = mxp()
    need = m.mxp_gemm_workspace_bytes(M, N, K, True, 0, wmode)
    assert need > 4096                                  # the tensor-core path is on offer
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    for dt in (torch.float32, torch.bfloat16):
        d = m.mxp_gemm(to_dev_bf16(a_bits), wp, out_dtype=dt, workspace=ws)
        assert m.mxp_gemm_status(ws) == 0
        check_gemm(d, da, dw)
    # without the workspace the general kernel answers, same result within the same bound
    d = m.mxp_gemm(to_dev_bf16(a_bits), wp, out_dtype=torch.float32,
                   workspace=torch.zeros(4096, dtype=torch.uint8, device="cuda"))
    check_gemm(d, da, dw)


@pytest.mark.parametrize("wmode", [MX, MXP, 2])
@pytest.mark.parametrize("M,N,K", [(1, 256, 512), (16, 1000, 384), (65, 520, 1024), (300, 129, 2048)])
def test_weight_only_with_prepacked_weights(M, N, K, wmode):
    # the same tensor-core path with the weights prepared once; any number of activation rows
    a_bits, w_bits = synth.config3(M, N, K, seed=M + N + K + 2)
    wp, dw = quantized(w_bits, wmode, bf16=True)
    da = oracle.bf16_bits_to_f64(a_bits)
    m = mxp()
    pre = m.mxp_gemm_prepack(wp, True)
    a = to_dev_bf16(a_bits)
    for dt in (torch.float32, torch.bfloat16):
        d = m.mxp_gemm_dense_prepacked(a, wp, pre, out_dtype=dt)
        check_gemm(d, da, dw)
    if M > 64:   # what mxp_gemm's own tensor-core path returns, bit for bit
        d0 = m.mxp_gemm(a, wp, out_dtype=torch.float32)
        d1 = m.mxp_gemm_dense_prepacked(a, wp, pre, out_dtype=torch.float32)
        assert torch.equal(d0.view(torch.int32), d1.view(torch.int32))
    from paper_2510_14557_b200 import MxpError
    with pytest.raises(MxpError):   # workspace too small
        m.mxp_gemm_dense_prepacked(a, wp, pre, workspace=torch.zeros(256, dtype=torch.uint8, device="cuda"))


def test_weight_only_many_rows_one_hot_and_magnitude_spread():
    # one-hot activation rows return single decoded weights exactly (hi carries the value, lo is
    # zero); rows whose blocks mix magnitudes 2^20 apart stay inside the bound (the small
    # elements lose bits of their lo part only)
    M, N, K = 128, 256, 512
    g = synth.rng(17)
    w = g.standard_normal((N, K)).astype(np.float32) * np.exp2(g.integers(-20, 20, (N, 1))).astype(np.float32)
    wp, dw = quantized(w, MXP)
    a = np.zeros((M, K), np.float32)
    for r in range(64):
        a[r, (r * 37) % K] = 2.0 ** (r - 30) * (1.0 + (r % 8) / 8.0)
    a[64:] = g.standard_normal((64, K)) * np.exp2(g.integers(-20, 1, (64, K)))
    a_bits = synth.f32_to_bf16_bits(a)
    da = oracle.bf16_bits_to_f64(a_bits)
    d = mxp().mxp_gemm(to_dev_bf16(a_bits), wp, out_dtype=torch.float32)
    got = d.cpu().numpy().astype(np.float64)
    for r in range(64):
        want = (dw[:, (r * 37) % K] * da[r, (r * 37) % K]).astype(np.float32).astype(np.float64)
        assert np.array_equal(got[r], want)
    check_gemm(d, da, dw)


# ------------------------------------------------------------------ tensor-core form
MODES = [(MX, MX), (MXP, MX), (MX, MXP), (MXP, MXP)]


@pytest.mark.parametrize("amode,bmode", MODES)
def test_tc_config1(amode, bmode):
    a, b = synth.config1()
    ap, da = quantized(a, amode)
    bp, db = quantized(b, bmode)
    m = mxp()
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    d = m.mxp_gemm(ap, bp, out_dtype=torch.float32, workspace=ws)
    assert m.mxp_gemm_status(ws) == 0
    check_gemm(d, da, db)
    d16 = m.mxp_gemm(ap, bp, out_dtype=torch.bfloat16, workspace=ws)
    check_gemm(d16, da, db)


@pytest.mark.parametrize("amode,bmode", MODES)
@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (128, 256, 256), (100, 72, 384), (300, 520, 1024),
                                   (1, 8, 128), (257, 129, 2176)])
def test_tc_shapes(M, N, K, amode, bmode):
    a = synth.activations_normal(M, K, seed=M + K, outlier_frac=0.02)
    b = synth.weights(N, K, seed=N + K)
    ap, da = quantized(a, amode)
    bp, db = quantized(b, bmode)
    d = mxp().mxp_gemm(ap, bp, out_dtype=torch.float32)
    check_gemm(d, da, db)


@pytest.mark.parametrize("amode,bmode", MODES)
def test_tc_one_hot_b_returns_decoded_a(amode, bmode):
    # B = identity (1.0 is an exactly representable BM): D must equal dec(A) bit for bit,
    # which exercises the BM residual passes exactly
    K = 256
    a = synth.activations_normal(192, K, seed=77, outlier_frac=0.03)
    ap, da = quantized(a, amode)
    bp, db = quantized(np.eye(K, dtype=np.float32), bmode)
    d = mxp().mxp_gemm(ap, bp, out_dtype=torch.float32)
    assert np.array_equal(d.cpu().numpy().astype(np.float64), da)


def test_tc_bm_positions_coincide():
    # both operands MX+ with the BM of every block at the same position: the BM_L x BM_L
    # term of the expansion is then non-zero everywhere
    M, N, K = 64, 64, 512
    g = synth.rng(3)
    a = (g.standard_normal((M, K)) * 0.3).astype(np.float32)
    b = (g.standard_normal((N, K)) * 0.3).astype(np.float32)
    pos = g.integers(0, 32, K // 32)
    for j, p in enumerate(pos):
        a[:, 32 * j + p] = g.choice([4.5, 5.5, 6.5, 7.5, -5.0, -7.0], M)
        b[:, 32 * j + p] = g.choice([4.5, 5.5, 6.5, 7.5, -4.5, -6.5], N)
    ap, da = quantized(a, MXP)
    bp, db = quantized(b, MXP)
    d = mxp().mxp_gemm(ap, bp, out_dtype=torch.float32)
    check_gemm(d, da, db)
    ref = oracle.gemm_fp64(da, db)
    # values are small dyadic rationals: fp32 accumulation is exact here
    assert np.array_equal(d.cpu().numpy().astype(np.float64), ref)


def test_tc_flushed_and_zero_blocks():
    M, N, K = 128, 128, 256
    a = synth.activations_normal(M, K, seed=1)
    b = synth.weights(N, K, seed=2)
    a[:, 64:96] = 0
    b[5, :] = 0
    b[:, 128:160] *= 1e-42
    ap, da = quantized(a, MXP)
    bp, db = quantized(b, MXP)
    d = mxp().mxp_gemm(ap, bp, out_dtype=torch.float32)
    check_gemm(d, da, db)
    assert float(d[:, 5].abs().max()) == 0.0


@pytest.mark.parametrize("kernel", ["single", "pair"])
@pytest.mark.parametrize("amode,bmode", MODES)
def test_tc_both_kernels_every_mode(kernel, amode, bmode, force):
    # the library picks the single-CTA or the CTA-pair kernel per mode; force each in turn
    force("inplace", kernel)
    M, N, K = 520, 777, 1280  # ragged in M and N, several tiles, K a multiple of 128 only
    a = synth.activations_normal(M, K, seed=5, outlier_frac=0.02)
    b = synth.weights(N, K, seed=6)
    ap, da = quantized(a, amode)
    bp, db = quantized(b, bmode)
    for dt in (torch.float32, torch.bfloat16):
        d = mxp().mxp_gemm(ap, bp, out_dtype=dt)
        check_gemm(d, da, db)


# ------------------------------------------------------------------ streamed kernel, prepack
MXPP = 2   # MX++ (Sec. 4.3): delta in the index byte's top three bits


def _raw_operand(rows, K, mode, seed, scale_lo=120, scale_hi=134):
    """Packed planes filled directly: every code, BM position, mantissa (and delta) occurs."""
    g = synth.rng(seed)
    nib = g.integers(0, 256, (rows, K // 2), dtype=np.uint8)
    sc = g.integers(scale_lo, scale_hi, (rows, K // 32), dtype=np.uint8)
    idx = None
    if mode == MXP:
        idx = g.integers(0, 32, (rows, K // 32), dtype=np.uint8)
    if mode == MXPP:
        idx = g.integers(0, 256, (rows, K // 32), dtype=np.uint8)
    dec = oracle.dequantize(nib, sc, idx, mode)
    return host_to_packed(nib, sc, idx, mode), dec


@pytest.mark.parametrize("amode,bmode", MODES)
def test_tc_stream_every_code_position_and_mantissa(amode, bmode):
    # B = identity (exactly representable): D must equal the oracle's decode of A bit for bit
    # for random raw planes, i.e. for every E2M1 code, BM position and BM mantissa; shapes go
    # to the streamed kernel (M, N > 128)
    M, K = 384, 256
    ap, da = _raw_operand(M, K, amode, seed=21)
    eye = np.eye(K, dtype=np.float32)
    bp, db = quantized(eye, bmode)
    assert np.array_equal(db, eye.astype(np.float64))
    d = mxp().mxp_gemm(ap, bp, out_dtype=torch.float32)
    assert np.array_equal(d.cpu().numpy().astype(np.float64), da)


@pytest.mark.parametrize("amode,bmode", MODES)
@pytest.mark.parametrize("M,N,K", [(300, 520, 1024), (257, 129, 2176), (512, 512, 128)])
def test_tc_prepacked_weights_match_mxp_gemm(M, N, K, amode, bmode):
    ap, da = _raw_operand(M, K, amode, seed=M + 1)
    bp, db = _raw_operand(N, K, bmode, seed=N + 2)
    m = mxp()
    pre = m.mxp_gemm_prepack(bp, m.mxp_gemm_prepack_form(amode, bmode))
    for dt in (torch.float32, torch.bfloat16):
        d0 = m.mxp_gemm(ap, bp, out_dtype=dt)
        d1 = m.mxp_gemm_prepacked(ap, bp, pre, out_dtype=dt)
        check_gemm(d1, da, db)
        assert torch.equal(d0, d1)


@pytest.mark.parametrize("halves", ["1", "2"])
@pytest.mark.parametrize("amode,bmode", [(MX, MX), (MXP, MXP), (MX, 2)])
@pytest.mark.parametrize("M,N,K", [(300, 250, 256), (257, 481, 384), (300, 959, 256), (513, 1000, 128),
                                   (256, 448, 512), (384, 960, 128)])
def test_tc_stream_tile_halves_and_ragged_edges(M, N, K, amode, bmode, halves, force):
    # the streamed kernel's output tile has one or two halves of 240 (plain MXFP4: 224) columns;
    # N values just past a half, just past a tile, exact multiples, and ragged on both sides,
    # with either tile shape forced
    force("halves", halves)
    ap, da = _raw_operand(M, K, amode, seed=M + N)
    bp, db = _raw_operand(N, K, bmode, seed=N + K)
    m = mxp()
    ws = torch.zeros(m.mxp_gemm_workspace_bytes(M, N, K, False, amode, bmode), dtype=torch.uint8, device="cuda")
    for dt in (torch.float32, torch.bfloat16):
        d = m.mxp_gemm(ap, bp, out_dtype=dt, workspace=ws)
        assert m.mxp_gemm_status(ws) == 0
        check_gemm(d, da, db)


def test_tc_stream_clock_stamp():
    # the streamed kernel leaves the SM cycles and nanoseconds its first CTA ran for; the in-place
    # kernels clear the stamp
    from paper_2510_14557_b200 import MxpError
    M, N, K = 512, 1024, 1024
    ap, _ = _raw_operand(M, K, MXP, seed=1)
    bp, _ = _raw_operand(N, K, MXP, seed=2)
    m = mxp()
    ws = torch.zeros(m.mxp_gemm_workspace_bytes(M, N, K, False, MXP, MXP), dtype=torch.uint8, device="cuda")
    m.mxp_gemm(ap, bp, workspace=ws)
    cycles, ns = m.mxp_gemm_clock_stamp(ws)
    assert 500 < ns < 10_000_000
    assert 0.1 < cycles / ns < 2.5          # GHz
    small = ws[:4096]
    m.mxp_gemm(ap, bp, workspace=small)      # too small for the streamed path: in-place kernels
    with pytest.raises(MxpError):
        m.mxp_gemm_clock_stamp(small)


def test_tc_prepack_rejects_bad_arguments():
    from paper_2510_14557_b200 import MxpError
    m = mxp()
    bp, _ = _raw_operand(256, 256, MXP, seed=5)
    with pytest.raises(MxpError):  # an MXFP4+ operand has no narrow prepacked form
        m.mxp_gemm_prepack(bp, False)
    pre = m.mxp_gemm_prepack(bp, True)
    small, _ = _raw_operand(64, 256, MXP, seed=6)
    with pytest.raises(MxpError):  # M <= 128: no streamed kernel, the caller uses mxp_gemm
        m.mxp_gemm_prepacked(small, bp, pre)
    with pytest.raises(MxpError):
        m.mxp_gemm_prepack(bp, True, out=torch.empty(1024, dtype=torch.uint8, device="cuda"))


def test_tc_stream_flushed_blocks_and_bm_coincidence():
    # streamed-kernel shapes: BMs of both operands at the same position in every block,
    # plus flushed (scale byte 0) and all-zero blocks
    M, N, K = 192, 320, 512
    g = synth.rng(9)
    a = (g.standard_normal((M, K)) * 0.3).astype(np.float32)
    b = (g.standard_normal((N, K)) * 0.3).astype(np.float32)
    pos = g.integers(0, 32, K // 32)
    for j, p in enumerate(pos):
        a[:, 32 * j + p] = g.choice([4.5, 5.5, 6.5, 7.5, -5.0, -7.0], M)
        b[:, 32 * j + p] = g.choice([4.5, 5.5, 6.5, 7.5, -4.5, -6.5], N)
    a[5, 64:96] = 0
    a[6, 96:128] = 1e-44
    b[7, 0:32] = 0
    b[8, 32:64] = -1e-44
    ap, da = quantized(a, MXP)
    bp, db = quantized(b, MXP)
    d = mxp().mxp_gemm(ap, bp, out_dtype=torch.float32)
    ref = oracle.gemm_fp64(da, db)
    assert np.array_equal(d.cpu().numpy().astype(np.float64), ref)


# ------------------------------------------------------------------ MX++ operands (Sec. 4.3)
PP_MODES = [(MXPP, MX), (MX, MXPP), (MXPP, MXP), (MXP, MXPP), (MXPP, MXPP)]


@pytest.mark.parametrize("amode,bmode", PP_MODES)
def test_tc_mxpp_every_code_position_mantissa_and_delta(amode, bmode):
    # identity on one side: D must equal the oracle's decode of the other operand bit for bit,
    # for random raw planes (every code, BM position, BM mantissa and delta 0..7)
    K = 256
    eye = np.eye(K, dtype=np.float32)
    if amode == MXPP:
        ap, da = _raw_operand(384, K, amode, seed=31)
        bp, db = quantized(eye, bmode)
        d = mxp().mxp_gemm(ap, bp, out_dtype=torch.float32)
        assert np.array_equal(d.cpu().numpy().astype(np.float64), da)
    if bmode == MXPP:
        ap, da = quantized(eye, amode)
        bp, db = _raw_operand(384, K, bmode, seed=32)
        d = mxp().mxp_gemm(ap, bp, out_dtype=torch.float32)
        assert np.array_equal(d.cpu().numpy().astype(np.float64), db.T)


def test_tc_mxpp_tiny_scale_bytes():
    # scale bytes 1..8 with every delta: the shift handed to the tensor core is limited by the
    # scale byte, the NBMs go down to E4M3 subnormals
    K = 256
    ap, da = _raw_operand(256, K, MXPP, seed=41, scale_lo=1, scale_hi=9)
    bp, db = quantized(np.eye(K, dtype=np.float32) * np.float32(2.0 ** 100), MXP)
    d = mxp().mxp_gemm(ap, bp, out_dtype=torch.float32)
    want = (da * 2.0 ** 100).astype(np.float32).astype(np.float64)
    assert np.array_equal(d.cpu().numpy().astype(np.float64), want)


@pytest.mark.parametrize("amode,bmode", PP_MODES)
def test_tc_mxpp_quantized_operands_and_prepack(amode, bmode):
    M, N, K = 300, 520, 1024
    a = synth.activations_normal(M, K, seed=3, outlier_frac=0.02)
    b = synth.weights(N, K, seed=4).astype(np.float32)
    ap, da = quantized(a, amode)
    bp, db = quantized(b, bmode)
    m = mxp()
    pre = m.mxp_gemm_prepack(bp, True)
    for dt in (torch.float32, torch.bfloat16):
        d0 = m.mxp_gemm(ap, bp, out_dtype=dt)
        check_gemm(d0, da, db)
        assert torch.equal(d0, m.mxp_gemm_prepacked(ap, bp, pre, out_dtype=dt))


def test_mxpp_without_the_prepacked_path_is_reported():
    from paper_2510_14557_b200 import MxpError
    m = mxp()
    ap, _ = _raw_operand(64, 256, MXPP, seed=1)
    bp, _ = _raw_operand(256, 256, MXP, seed=2)
    small = torch.zeros(4096, dtype=torch.uint8, device="cuda")   # minimum workspace only:
    with pytest.raises(MxpError) as e:                            # the in-place kernels
        m.mxp_gemm(ap, bp, workspace=small)
    assert e.value.status == 2                        # MXP_ERR_UNSUPPORTED


@pytest.mark.parametrize("M,N,K", [(1, 1, 128), (64, 256, 256), (129, 7, 384), (100, 72, 1024)])
def test_tc_mxpp_small_shapes(M, N, K):
    # MX++ with M or N <= 128 goes through the streamed kernel too (TMA zero-fills the rest)
    ap, da = _raw_operand(M, K, MXPP, seed=M + 7)
    bp, db = _raw_operand(N, K, MXPP, seed=N + 9)
    for dt in (torch.float32, torch.bfloat16):
        check_gemm(mxp().mxp_gemm(ap, bp, out_dtype=dt), da, db)
