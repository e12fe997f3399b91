"""GPU parity of the decode GEMM on re-tiled weights (mxp_gemm_decode_prepack /
mxp_gemm_decode_prepacked, 1 <= M <= 16) against the oracle's fp64 product of the bf16
activations and the decoded weights."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from helpers import check_gemm, host_to_packed, to_dev_bf16
from paper_2510_14557_b200 import synth

pytestmark = pytest.mark.gpu
MX, MXP = 0, 1


def mxp():
    import paper_2510_14557_b200 as m
    return m


def raw_weights(N, K, mode, seed, lo=118, hi=136):
    """Planes filled directly: every code, BM position and BM mantissa occurs."""
    g = synth.rng(seed)
    nib = g.integers(0, 256, (N, K // 2), dtype=np.uint8)
    sc = g.integers(lo, hi, (N, K // 32), dtype=np.uint8)
    idx = g.integers(0, 32, (N, K // 32), dtype=np.uint8) if mode == MXP else None
    return host_to_packed(nib, sc, idx, mode), oracle.dequantize(nib, sc, idx, mode)


@pytest.mark.parametrize("wmode", [MX, MXP])
@pytest.mark.parametrize("M,N,K", [(1, 64, 256), (1, 11008, 4096), (2, 300, 512), (3, 2384, 4096), (4, 77, 1024),
                                   (5, 1000, 768), (7, 19000, 512), (8, 11008, 4096), (9, 160, 4352),
                                   (12, 40000, 256), (13, 333, 1280), (16, 11008, 4096), (16, 8, 256), (1, 1, 256),
                                   (2, 40000, 256), (1, 40000, 256), (1, 19000, 8192), (1, 700, 16384), (2, 700, 16384),
                                   (2, 11008, 4096), (3, 11008, 4096), (3, 40000, 256), (3, 700, 16384)])
def test_decode_prepacked_parity(M, N, K, wmode):
    # ragged N (last CTA short, rows not a multiple of 8), more than 128 rows per CTA (several
    # tiles), every activation-operand width (16 .. 80 rows), K from one stage to seventeen.
    # A single row takes the form in which every CTA converts the activations for itself and
    # adds the BM's lower part on the CUDA cores: also with several tiles per CTA, with images
    # that leave room for few ring slots (K = 8192) and with images that do not fit at all
    # (K = 16384: back to the conversion kernel)
    m = mxp()
    a_bits, w_bits = synth.config3(M, N, K, seed=M + N + K)
    q = oracle.quantize(w_bits, wmode, bf16_bits=True)
    wp = host_to_packed(q[0], q[1], q[2] if wmode != MX else None, wmode)
    dw = oracle.dequantize(q[0], q[1], q[2], wmode)
    da = oracle.bf16_bits_to_f64(a_bits)
    w = m.mxp_gemm_decode_prepack(wp)
    ws = torch.zeros(m.mxp_gemm_decode_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
    for dt in (torch.float32, torch.bfloat16):
        d = m.mxp_gemm_decode_prepacked(to_dev_bf16(a_bits), w, out_dtype=dt, workspace=ws)
        assert m.mxp_gemm_status(ws) == 0
        check_gemm(d, da, dw)


@pytest.mark.parametrize("wmode", [MX, MXP])
def test_decode_prepacked_one_hot_rows_return_decoded_weights(wmode):
    # a one-hot activation row (its single digit is exact in every plane) selects one decoded
    # weight per output: equality in fp32, for raw planes with every code, BM position and
    # mantissa and scales spread over 18 binades
    m = mxp()
    N, K = 700, 1024
    wp, dw = raw_weights(N, K, wmode, seed=5)
    w = m.mxp_gemm_decode_prepack(wp)
    g = synth.rng(9)
    for M in (1, 4, 16):
        a = np.zeros((M, K), np.float32)
        ks = g.integers(0, K, M)
        vals = np.exp2(g.integers(-6, 7, M)).astype(np.float32) * np.where(g.random(M) < 0.5, -1, 1)
        a[np.arange(M), ks] = vals
        d = m.mxp_gemm_decode_prepacked(to_dev_bf16(synth.f32_to_bf16_bits(a)), w, out_dtype=torch.float32)
        got = d.cpu().numpy().astype(np.float64)
        for i in range(M):
            assert np.array_equal(got[i], dw[:, ks[i]] * float(vals[i])), (M, i)


def test_decode_prepacked_special_blocks():
    # flushed blocks (scale byte 0, also with non-zero codes behind it: they decode to zero),
    # BM at the first and last position, all-zero activations, activations with a wide spread
    # inside a block (the small ones are rounded at 2^-13 of the block's binade: inside the bound)
    m = mxp()
    N, K, M = 96, 512, 3
    g = synth.rng(3)
    nib = g.integers(0, 256, (N, K // 2), dtype=np.uint8)
    sc = g.integers(120, 130, (N, K // 32), dtype=np.uint8)
    idx = g.choice(np.array([0, 31, 1, 30], np.uint8), (N, K // 32))
    sc[::3, ::2] = 0
    dw = oracle.dequantize(nib, sc, idx, MXP)
    assert (dw[::3].reshape(32, -1, 32)[:, ::2] == 0).all()
    w = m.mxp_gemm_decode_prepack(host_to_packed(nib, sc, idx, MXP))
    a = (g.standard_normal((M, K)) * np.exp2(g.integers(-12, 6, (M, K)))).astype(np.float32)
    a[1] = 0
    a_bits = synth.f32_to_bf16_bits(a)
    d = m.mxp_gemm_decode_prepacked(to_dev_bf16(a_bits), w, out_dtype=torch.float32)
    check_gemm(d, oracle.bf16_bits_to_f64(a_bits), dw)
    assert not d[1].any()


def test_decode_prepacked_chained_layers_and_graph():
    # a chain of layers, each reading the previous one's output, launched as programmatic
    # dependents; eagerly and replayed from a CUDA graph: bit-identical to unchained calls
    m = mxp()
    K = N = 1024
    M = 4
    layers = []
    for i in range(4):
        _, w_bits = synth.config3(1, N, K, seed=20 + i)
        layers.append(m.mxp_gemm_decode_prepack(m.mxp_quantize(to_dev_bf16(w_bits * 1), MXP)))
    a_bits, _ = synth.config3(M, 32, K, seed=1)
    x0 = to_dev_bf16(a_bits)
    ws = torch.zeros(m.mxp_gemm_decode_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")

    def run(chained):
        x = x0
        outs = []
        for w in layers:
            y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            m.mxp_gemm_decode_prepacked(x, w, out=y, workspace=ws, chained=chained)
            outs.append(y)
            x = y
        return outs

    ref = run(False)
    torch.cuda.synchronize()
    got = run(True)
    torch.cuda.synchronize()
    for a, b in zip(ref, got):
        assert torch.equal(a, b)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        run(True)
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        outs = run(True)
    for o in outs:
        o.zero_()
    graph.replay()
    torch.cuda.synchronize()
    for a, b in zip(ref, outs):
        assert torch.equal(a, b)
    assert m.mxp_gemm_status(ws) == 0


@pytest.mark.parametrize("M", [1, 2, 5, 16])
def test_decode_prepacked_with_a_hint_for_the_next_layers_weights(M):
    # the hint only prefetches: layers of three different shapes and both modes in a chain, each
    # call naming the next one's weights (the last one none), give bit for bit what the calls
    # without a hint give; a tiny next matrix (less than a CTA's share) and one whose CTAs are
    # fewer than the SMs are among them
    m = mxp()
    shapes = [(1024, 1024, MXP), (4096, 1024, MX), (1024, 4096, MXP), (40, 1024, MX), (1024, 1024, MXP)]
    layers = []
    for i, (N, K, mode) in enumerate(shapes):
        _, w_bits = synth.config3(1, N, K, seed=40 + i)
        layers.append(m.mxp_gemm_decode_prepack(m.mxp_quantize(to_dev_bf16(w_bits * 1), mode)))
    a_bits, _ = synth.config3(M, 32, 1024, seed=2)
    x0 = to_dev_bf16(a_bits)
    ws = torch.zeros(m.mxp_gemm_decode_workspace_bytes(M, 4096), dtype=torch.uint8, device="cuda")

    def run(hint):
        x, outs = x0, []
        for i, w in enumerate(layers):
            y = torch.empty((M, w.rows), dtype=torch.bfloat16, device="cuda")
            nxt = layers[i + 1] if hint and i + 1 < len(layers) else None
            m.mxp_gemm_decode_prepacked(x[:, :w.cols].contiguous() if x.shape[1] != w.cols else x, w, out=y,
                                        workspace=ws, next_w=nxt)
            outs.append(y)
            x = y if y.shape[1] >= 1024 else x0
        return outs

    ref = run(False)
    got = run(True)
    torch.cuda.synchronize()
    for a, b in zip(ref, got):
        assert torch.equal(a, b)
    assert m.mxp_gemm_status(ws) == 0
    # pointer without size, size without pointer, misaligned pointer: rejected before any launch
    lib = m.binding.lib()
    w, y = layers[0], torch.empty((M, 1024), dtype=torch.bfloat16, device="cuda")

    def call(nptr, nbytes):
        return lib.mxp_gemm_decode_prepacked_next(M, 1024, 1024, x0.data_ptr(), 1024, MXP, w.buf.data_ptr(),
                                                  w.buf.numel(), y.data_ptr(), 1, 1024, ws.data_ptr(), ws.numel(), 0,
                                                  nptr, nbytes, None)
    assert call(layers[1].buf.data_ptr(), layers[1].buf.numel()) == 0
    assert call(None, 0) == 0
    assert call(layers[1].buf.data_ptr(), 0) == 1
    assert call(None, 4096) == 1
    assert call(layers[1].buf.data_ptr() + 16, layers[1].buf.numel() - 16) == 1
    torch.cuda.synchronize()


def test_decode_prepacked_argument_checks():
    m = mxp()
    lib = m.binding.lib()
    N, K = 256, 512
    wp, _ = raw_weights(N, K, MXP, seed=1)
    w = m.mxp_gemm_decode_prepack(wp)
    a = torch.zeros((2, K), dtype=torch.bfloat16, device="cuda")
    d = torch.zeros((2, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(m.mxp_gemm_decode_workspace_bytes(2, K), dtype=torch.uint8, device="cuda")

    def call(M=2, n=N, k=K, mode=MXP, nbytes=None, wsb=None):
        return lib.mxp_gemm_decode_prepacked(M, n, k, a.data_ptr(), K, mode, w.buf.data_ptr(),
                                             w.buf.numel() if nbytes is None else nbytes, d.data_ptr(), 1, N,
                                             ws.data_ptr(), ws.numel() if wsb is None else wsb, 0, None)
    assert call() == 0
    assert call(mode=MX) == 1            # re-tiled for MXFP4+, used as MXFP4: sizes differ
    assert call(n=N - 16) == 1           # another shape
    assert call(nbytes=w.buf.numel() - 16) == 1
    assert call(wsb=256) == 3            # workspace too small
    assert call(M=17) == 2               # more rows than the decode path takes
    assert lib.mxp_gemm_decode_prepack_bytes(N, 500, MXP) == 0
    assert lib.mxp_gemm_decode_prepack_bytes(N, K, 2) == 0     # MX++: not on this path
    torch.cuda.synchronize()
