"""Seeded synthetic inputs shared by the CPU oracle's tests and the GPU tests.

Only random-number draws, shapes and storage-type conversion live here: none of
the arithmetic of the structured contractions.  The paper's evaluation
(Section 7) gives no tensor sizes or value distributions in its text and its
datasets are not available, so the five named configurations below stand in for
its covariance workloads (Section 7.2, Figure "covar") and its sparsity kernels
(Table 1): same operations, same structures, seeded i.i.d. values.

All arrays are generated on the host in float32 with numpy's PCG64
``default_rng(seed)``.
"""
from __future__ import annotations

import numpy as np

SEEDS = {
    "moment2": 1001,
    "moment3": 1002,
    "mttkrp_B": 1003, "mttkrp_C": 1013, "mttkrp_D": 1023,
    "ttm_B": 1004, "ttm_U": 1014,
    "moment2_large": 1005,
}

# name -> shape parameters of the five named configurations
CONFIGS = {
    "moment2": dict(N=4096, d=64, dist="uniform"),
    "moment3": dict(N=65536, d=64, dist="normal"),
    "mttkrp": dict(I=512, K=512, R=32, dist="uniform"),
    "ttm": dict(nb=64, bs=64, K=256, R=64, dist="normal"),
    "moment2_large": dict(N=1 << 20, d=1024, dist="normal"),
}


def tri(d: int) -> int:
    return d * (d + 1) // 2


def tet(d: int) -> int:
    return d * (d + 1) * (d + 2) // 6


def draw(shape, dist: str, seed: int) -> np.ndarray:
    """float32 array of i.i.d. uniform[-1,1) or N(0,1) values."""
    rng = np.random.default_rng(seed)
    if dist == "uniform":
        a = rng.random(shape, dtype=np.float32)
        a *= 2.0
        a -= 1.0
        return a
    if dist == "normal":
        return rng.standard_normal(shape, dtype=np.float32)
    if dist == "ones":
        return np.ones(shape, np.float32)
    raise ValueError(dist)


def draw_rows(N: int, d: int, dist: str, seed: int, chunk: int = 1 << 16) -> np.ndarray:
    """[N, d] float32, generated in row chunks so that a prefix of the rows does
    not depend on N (the first rows of a large draw equal a smaller draw)."""
    out = np.empty((N, d), np.float32)
    rng = np.random.default_rng(seed)
    for r0 in range(0, N, chunk):
        r1 = min(N, r0 + chunk)
        if dist == "uniform":
            blk = rng.random((r1 - r0, d), dtype=np.float32)
            blk *= 2.0
            blk -= 1.0
        elif dist == "normal":
            blk = rng.standard_normal((r1 - r0, d), dtype=np.float32)
        else:
            raise ValueError(dist)
        out[r0:r1] = blk
    return out


def draw_rows_bf16(N: int, d: int, dist: str, seed: int, chunk: int = 1 << 16) -> np.ndarray:
    """bfloat16 bit patterns (uint16) of draw_rows(N, d, dist, seed), produced chunk by chunk so
    that the float32 array is never held whole."""
    out = np.empty((N, d), np.uint16)
    rng = np.random.default_rng(seed)
    for r0 in range(0, N, chunk):
        r1 = min(N, r0 + chunk)
        if dist == "uniform":
            blk = rng.random((r1 - r0, d), dtype=np.float32)
            blk *= 2.0
            blk -= 1.0
        elif dist == "normal":
            blk = rng.standard_normal((r1 - r0, d), dtype=np.float32)
        else:
            raise ValueError(dist)
        out[r0:r1] = f32_to_bf16_bits(blk)
    return out


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns to float32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def moment_input(name: str, N: int | None = None, d: int | None = None) -> np.ndarray:
    cfg = CONFIGS[name]
    N = cfg["N"] if N is None else N
    d = cfg["d"] if d is None else d
    return draw_rows(N, d, cfg["dist"], SEEDS[name])


def mttkrp_inputs(I: int | None = None, K: int | None = None, R: int | None = None):
    """Packed B [tri(I), K] (values for the positions i<=j only), C [I, R], D [K, R]."""
    cfg = CONFIGS["mttkrp"]
    I = cfg["I"] if I is None else I
    K = cfg["K"] if K is None else K
    R = cfg["R"] if R is None else R
    Bp = draw((tri(I), K), cfg["dist"], SEEDS["mttkrp_B"])
    C = draw((I, R), cfg["dist"], SEEDS["mttkrp_C"])
    D = draw((K, R), cfg["dist"], SEEDS["mttkrp_D"])
    return Bp, C, D


def ttm_inputs(nb: int | None = None, bs: int | None = None, K: int | None = None,
               R: int | None = None):
    """Packed B [nb, bs, bs, K] (the diagonal blocks only) and U [K, R]."""
    cfg = CONFIGS["ttm"]
    nb = cfg["nb"] if nb is None else nb
    bs = cfg["bs"] if bs is None else bs
    K = cfg["K"] if K is None else K
    R = cfg["R"] if R is None else R
    Bp = draw((nb, bs, bs, K), cfg["dist"], SEEDS["ttm_B"])
    U = draw((K, R), cfg["dist"], SEEDS["ttm_U"])
    return Bp, U
