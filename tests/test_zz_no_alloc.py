"""mxp_gemm_noalloc: the GEMM entry point for callers that cannot allocate device memory
(hosts living inside another framework's memory pool).  Its scratch is a fixed array inside
the library, so the test checks that two calls in a row give what mxp_gemm gives with a
caller-provided workspace.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_gemm, packed_to_host, to_dev
from paper_2510_14557_b200 import synth

pytestmark = pytest.mark.gpu


def test_noalloc_matches_mxp_gemm_twice_in_a_row():
    import paper_2510_14557_b200 as m
    M, N, K = 200, 264, 768
    a = to_dev(synth.activations_normal(M, K, seed=21, outlier_frac=0.02))
    results = []
    for call, (amode, bmode, seed) in enumerate([(1, 1, 31), (1, 0, 32)]):
        w = to_dev(synth.weights(N, K, seed=seed))
        pa, pw = m.mxp_quantize(a, amode), m.mxp_quantize(w, bmode)
        ref = m.mxp_gemm(pa, pw, out_dtype=torch.float32)          # existing entry point
        out = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        status = m.mxp_gemm_noalloc(pa, pw, out, read_status=True)  # the one under test
        assert status == 0
        # tolerance of the GEMM parity tests: 1e-3 * |a_m| * |b_n| on the decoded operands
        da = m.mxp_dequantize(pa, torch.float32).double()
        dw = m.mxp_dequantize(pw, torch.float32).double()
        tol = 1e-3 * da.norm(dim=1)[:, None] * dw.norm(dim=1)[None, :]
        err = (out.double() - ref.double()).abs()
        assert bool((err <= tol).all()), "call %d: max err/tol %g" % (call, float((err / tol).max()))
        # and against the oracle: the fp64 product of its own decode of the same planes
        na, sa, ia = packed_to_host(pa)
        nw, sw, iw = packed_to_host(pw)
        check_gemm(out, oracle.dequantize(na, sa, ia, amode), oracle.dequantize(nw, sw, iw, bmode))
        results.append(out)
    # asynchronous form (no status read) on a bf16 output, after the two calls above
    out16 = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    assert m.mxp_gemm_noalloc(pa, pw, out16) is None
    torch.cuda.synchronize()
    assert torch.equal(out16, m.mxp_gemm(pa, pw, out_dtype=torch.bfloat16))


def test_noalloc_rejects_bad_arguments():
    import paper_2510_14557_b200 as m
    a = to_dev(synth.activations_normal(8, 128, seed=1))
    pa = m.mxp_quantize(a, 1)
    pb = m.mxp_quantize(to_dev(synth.weights(16, 256, seed=2)), 1)  # K mismatch
    out = torch.empty((8, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(m.MxpError) as e:
        m.mxp_gemm_noalloc(pa, pb, out)
    assert e.value.status == 1
    # modes that need operands prepared in a workspace are "unsupported", as for mxp_gemm
    pp = m.mxp_quantize(to_dev(synth.weights(16, 128, seed=3)), m.MODE_MXFP4_PP)
    with pytest.raises(m.MxpError) as e:
        m.mxp_gemm_noalloc(pa, pp, out)
    assert e.value.status == 2
