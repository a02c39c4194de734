"""Seeded synthetic inputs for the BFP16 x BF16 GEMM workloads.

Counter-based: element ``i`` of tensor ``tag`` under ``seed`` is a pure function
of ``(seed, tag, i)``, so arrays are reproducible, order independent and can be
generated in chunks.  This module holds no arithmetic of the method itself (no
quantiser, no GEMM): it only draws numbers and rounds fp32 to bf16 bit patterns
for the operand that is *given* in bf16.  Both the CUDA path and the CPU oracle
are fed from here.

The paper measures on bare GEMM shapes with no public dataset, so these
distributions stand in for activations (A) and weights (B):

====== =========================== ============================= ==============
config shape (M, N, K)             A (fp32, then BFP16)          B (bf16)
====== =========================== ============================= ==============
1      256, 256, 256               N(0,1)                        N(0,1)
2      4096, 4096, 4096            N(0,1)                        0.02 N(0,1)
3      8192, 8192, 8192            Laplace(0,1)                  N(0,1)
4a     16384, 14336, 4096          N(0,1), 1% of entries x20     N(0, 1/K)
4b     16384, 4096, 14336          N(0,1), 1% of entries x20     N(0, 1/K)
====== =========================== ============================= ==============
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

BASE_SEED = 251116041
TAG_A, TAG_B, TAG_MASK = 1, 2, 3
_CHUNK = 1 << 20
_THREADS = min(16, os.cpu_count() or 1)
_U64 = np.uint64


def _splitmix64(x: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = x + _U64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> _U64(30))) * _U64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> _U64(27))) * _U64(0x94D049BB133111EB)
        return z ^ (z >> _U64(31))


def _key(seed: int, tag: int) -> np.uint64:
    k = _splitmix64(np.array([seed & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))
    k = _splitmix64(k ^ np.array([tag], dtype=np.uint64))
    return k[0]


def _bits(seed: int, tag: int, start: int, count: int) -> np.ndarray:
    idx = np.arange(start, start + count, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _splitmix64(idx * _U64(0xD1342543DE82EF95) + _key(seed, tag))


def _fill(shape, fn, dtype=np.float32) -> np.ndarray:
    """out[i] = fn(start, count)[i - start], chunk by chunk (chunks are independent: threads)."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype)

    def work(s):
        c = min(_CHUNK, n - s)
        out[s:s + c] = fn(s, c)

    starts = range(0, n, _CHUNK)
    if _THREADS > 1 and n > _CHUNK:
        with ThreadPoolExecutor(_THREADS) as pool:
            list(pool.map(work, starts))
    else:
        for s in starts:
            work(s)
    return out.reshape(shape)


def normal(seed: int, tag: int, shape, scale: float = 1.0) -> np.ndarray:
    """fp32 samples of N(0, scale^2) (Box-Muller on two 32-bit uniforms)."""
    def fn(s, c):
        z = _bits(seed, tag, s, c)
        u1 = ((z >> _U64(32)).astype(np.float64) + 1.0) * 2.0 ** -32      # (0, 1]
        u2 = (z & _U64(0xFFFFFFFF)).astype(np.float64) * 2.0 ** -32       # [0, 1)
        g = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
        return (g * scale).astype(np.float32)
    return _fill(shape, fn)


def laplace(seed: int, tag: int, shape) -> np.ndarray:
    """fp32 samples of Laplace(0, 1): x = -sgn(u) ln(1 - 2|u|), u in (-1/2, 1/2)."""
    def fn(s, c):
        z = _bits(seed, tag, s, c)
        u = ((z >> _U64(11)).astype(np.float64) + 0.5) * 2.0 ** -53 - 0.5
        return (-np.sign(u) * np.log1p(-2.0 * np.abs(u))).astype(np.float32)
    return _fill(shape, fn)


def bernoulli(seed: int, tag: int, shape, p: float) -> np.ndarray:
    """Boolean mask, each entry True with probability p."""
    def fn(s, c):
        z = _bits(seed, tag, s, c)
        return (z >> _U64(11)).astype(np.float64) * 2.0 ** -53 < p
    return _fill(shape, fn, bool)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even; NaN stays NaN."""
    w = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (w + (np.uint32(0x7FFF) + ((w >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    nan = (w & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
    return np.where(nan, (w >> np.uint32(16)) | np.uint32(0x40), rounded).astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


CONFIGS = {
    "cfg1_256": dict(M=256, N=256, K=256, A="normal", B="normal", b_scale=1.0),
    "cfg2_4096": dict(M=4096, N=4096, K=4096, A="normal", B="normal", b_scale=0.02),
    "cfg3_8192": dict(M=8192, N=8192, K=8192, A="laplace", B="normal", b_scale=1.0),
    "cfg4_ffn_up": dict(M=16384, N=14336, K=4096, A="outlier", B="normal", b_scale=None),
    "cfg4_ffn_down": dict(M=16384, N=4096, K=14336, A="outlier", B="normal", b_scale=None),
    # shallow-K cut of the headline shape: same tiles per wave, a quarter of the K-steps; small
    # enough for a multi-pass profiler capture while operands + output still exceed the L2
    "prof_8192x8192x2048": dict(M=8192, N=8192, K=2048, A="laplace", B="normal", b_scale=1.0),
}


def make_A(kind: str, M: int, K: int, seed: int = BASE_SEED) -> np.ndarray:
    """fp32 A[M][K] before quantisation: 'normal', 'laplace' or 'outlier'."""
    if kind == "normal":
        return normal(seed, TAG_A, (M, K))
    if kind == "laplace":
        return laplace(seed, TAG_A, (M, K))
    if kind == "outlier":
        a = normal(seed, TAG_A, (M, K))
        a[bernoulli(seed, TAG_MASK, (M, K), 0.01)] *= np.float32(20.0)
        return a
    raise ValueError(kind)


def make_B_bits(K: int, N: int, scale: float | None = 1.0, seed: int = BASE_SEED) -> np.ndarray:
    """bf16 bit patterns of B[K][N] ~ N(0, scale^2); scale=None means K^-1/2."""
    if scale is None:
        scale = float(K) ** -0.5
    return to_bf16_bits(normal(seed, TAG_B, (K, N), scale))


def make_config(name: str, seed: int = BASE_SEED, M: int | None = None):
    """(A fp32 [M][K], B bf16 bits [K][N]) of a named workload; ``M`` may shrink the row count."""
    c = CONFIGS[name]
    m = c["M"] if M is None else M
    return make_A(c["A"], m, c["K"], seed), make_B_bits(c["K"], c["N"], c["b_scale"], seed)


SWEEP_SIZES = (1024, 2048, 4096, 8192, 16384)


def device_normal(shape, seed: int, tag: int, device, dtype=None):
    """N(0,1) samples drawn ON THE DEVICE by torch's seeded generator, for the 125-shape sweep, whose
    operands (up to 1 GB each) would take minutes to draw on the host.  Reproducible for a given torch
    build; a consumer that needs the values on the host copies them back, so both sides of a comparison
    always see the same numbers.  fp32, or rounded to ``dtype`` (bf16: torch rounds to nearest even)."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + tag) & 0x7FFFFFFFFFFFFFFF)
    x = torch.randn(shape, device=device, dtype=torch.float32, generator=g)
    return x if dtype is None else x.to(dtype)
