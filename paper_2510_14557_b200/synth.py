"""Seeded synthetic inputs shared by the tests, the benchmark and the oracle checks.

Holds no MX / MX+ arithmetic: only random draws, outlier scaling and the dtype cast to
bfloat16 bit patterns.  Everything is drawn on the host with
``numpy.random.Generator(PCG64(seed))`` so that the CPU oracle and the CUDA path see
the same bytes.

The arrays stand in for the paper's workloads: LLM activations whose outliers sit in a
few channels (Sec. 3.2), benign weights with rare spikes, and the matmul shapes of
Sec. 7 (N = K = 4096 at small and large M, Llama-like prefill / decode).
"""
from __future__ import annotations

import numpy as np


def rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def outlier_columns(g: np.random.Generator, cols: int, frac: float) -> np.ndarray:
    n_out = max(1, int(round(frac * cols)))
    return np.sort(g.choice(cols, size=n_out, replace=False))


def activations_normal(rows: int, cols: int, seed: int, outlier_frac: float = 0.01,
                       outlier_scale: float = 30.0) -> np.ndarray:
    """N(0,1) float32 with a fraction of the columns scaled up (outlier channels)."""
    g = rng(seed)
    x = g.standard_normal((rows, cols), dtype=np.float32)
    oc = outlier_columns(g, cols, outlier_frac)
    x[:, oc] *= np.float32(outlier_scale)
    return x


def activations_student_t(rows: int, cols: int, seed: int, outlier_frac: float = 0.005,
                          outlier_scale: float = 50.0) -> np.ndarray:
    """Student-t (nu = 3) float32, z0 / sqrt((z1^2 + z2^2 + z3^2) / 3), plus outlier columns."""
    g = rng(seed)
    z0 = g.standard_normal((rows, cols), dtype=np.float32)
    s = np.zeros((rows, cols), np.float32)
    for _ in range(3):
        z = g.standard_normal((rows, cols), dtype=np.float32)
        s += z * z
    x = z0 / np.sqrt(s / np.float32(3.0))
    oc = outlier_columns(g, cols, outlier_frac)
    x[:, oc] *= np.float32(outlier_scale)
    return x.astype(np.float32)


def weights(rows: int, cols: int, seed: int, sigma: float = 0.02, spike_prob: float = 0.001,
            spike_scale: float = 20.0) -> np.ndarray:
    """N(0, sigma) float32 with Bernoulli(spike_prob) entries scaled up."""
    g = rng(seed)
    w = g.standard_normal((rows, cols), dtype=np.float32) * np.float32(sigma)
    spikes = g.random((rows, cols), dtype=np.float32) < np.float32(spike_prob)
    w[spikes] *= np.float32(spike_scale)
    return w


def config1(seed: int = 0):
    """256 x 256 x 256 round trip: A N(0,1) with 1 % outlier columns x30, B N(0,1); fp32."""
    a = activations_normal(256, 256, seed, 0.01, 30.0)
    b = rng(seed + 100).standard_normal((256, 256), dtype=np.float32)
    return a, b


def config2(rows: int = 8192, cols: int = 8192, seed: int = 1) -> np.ndarray:
    """Quantize-only input: Student-t activations, 0.5 % columns x50, bfloat16 bit patterns."""
    return f32_to_bf16_bits(activations_student_t(rows, cols, seed, 0.005, 50.0))


def config3(m: int, n: int = 11008, k: int = 4096, seed: int = 2):
    """Decode weight-only GEMM: (A bf16 bits [m,k], W bf16 bits [n,k])."""
    a = f32_to_bf16_bits(activations_normal(m, k, seed, 0.01, 30.0))
    w = f32_to_bf16_bits(weights(n, k, seed + 100))
    return a, w


def config4(m: int = 2048, n: int = 4096, k: int = 4096, seed: int = 3):
    """Prefill GEMM operands before quantization: (A bf16 bits [m,k], W bf16 bits [n,k])."""
    a = f32_to_bf16_bits(activations_normal(m, k, seed, 0.01, 30.0))
    w = f32_to_bf16_bits(weights(n, k, seed + 100))
    return a, w


def config5(m: int = 8192, n: int = 28672, k: int = 8192, seed: int = 4):
    """Large prefill GEMM operands (Llama-70B MLP-like shape), same distributions as config4."""
    return config4(m, n, k, seed)
