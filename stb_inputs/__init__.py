"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module holds none of the method's arithmetic: it draws random numbers
with the shapes and value distributions of the workloads (LLaMA-2 linear
shapes; fp16 weights ~ N(0, 0.02) with 1 % of the columns scaled x10;
activations ~ N(0, 1) with 0.5 % of the channels scaled x20) and, for the
large cases, logical structured-binary layers drawn directly (random N-of-8
masks, signs, region ids, salient columns and scales) so that no quantizer has
to run.  Neither the CPU oracle nor the CUDA library is imported here.
"""
from __future__ import annotations

from itertools import combinations

import numpy as np

SEED_BASE = 0x57B00000
BLOCK = 128
GROUP = 8


def seed_for(config: int, item: int = 0) -> int:
    """Seed of tensor `item` (layer / tensor index) of workload `config` (1..5)."""
    return SEED_BASE + 16 * config + item


def _rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, stream]))


def outlier_channels(m: int, seed: int, frac: float, stream: int) -> np.ndarray:
    k = int(round(frac * m))
    return np.sort(_rng(seed, stream).permutation(m)[:k])


def dense_weight(n: int, m: int, seed: int) -> np.ndarray:
    """fp16 W[n][m] ~ N(0, 0.02^2); exactly round(0.01 m) columns scaled x10."""
    g = _rng(seed, 1)
    W = g.standard_normal((n, m), dtype=np.float32) * np.float32(0.02)
    W[:, outlier_channels(m, seed, 0.01, 2)] *= np.float32(10.0)
    return W.astype(np.float16)


def activations(T: int, m: int, seed: int, dtype=np.float16) -> np.ndarray:
    """x[T][m] ~ N(0,1); exactly round(0.005 m) channels scaled x20 (float32 values that are
    exactly representable in `dtype`: np.float16, or "bf16" for bfloat16 kept as float32)."""
    g = _rng(seed, 3)
    x = g.standard_normal((T, m), dtype=np.float32)
    x[:, outlier_channels(m, seed, 0.005, 4)] *= np.float32(20.0)
    if dtype == "bf16":
        return round_to_bf16(x)
    return x.astype(dtype)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bfloat16 (ties to even); result stays float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are exactly representable in bfloat16."""
    return (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)


def calib_norms(m: int, seed: int, r: int = 256) -> np.ndarray:
    """||X_:,j||_2 over r calibration rows drawn from the activation law with the same
    outlier channels as activations(., m, seed) (separate random sub-stream)."""
    g = _rng(seed, 5)
    X = g.standard_normal((r, m), dtype=np.float32).astype(np.float64)
    X[:, outlier_channels(m, seed, 0.005, 4)] *= 20.0
    return np.sqrt((X * X).sum(axis=0))


def _mask_table(N: int) -> np.ndarray:
    return np.array([sum(1 << c for c in comb) for comb in combinations(range(GROUP), N)],
                    dtype=np.uint8)


def logical_layer(n: int, m: int, N: int, seed: int, max_salient: int = 3,
                  region_p=(0.68, 0.26, 0.06), salient_counts=None) -> dict:
    """Draw a logical structured-binary layer directly (no quantizer).

    Returns a dict of C-contiguous numpy arrays in the logical format:
      keep u8[n][m/8], sign u8[n][m/8], region u16[n][m/8], sign2 u32[n][m/128],
      salient u64[m/128][2], scale u16[n][m/128][5] (fp16 bits).
    Structure: every group of 8 columns keeps exactly N (uniform over the C(8,N) masks);
    1..max_salient salient columns per 128-column block (or salient_counts[b % len] of them in block b,
    when that list is given); non-salient kept weights get
    region 0/1/2 (dense/intermediate/sparse) with probabilities region_p; kept weights in
    salient columns get region 3 and a residual sign; scales are positive fp16.
    """
    assert m % BLOCK == 0 and 1 <= N <= 8
    g = _rng(seed, 7)
    nblk, ngrp = m // BLOCK, m // GROUP
    table = _mask_table(N)
    keep = table[g.integers(0, len(table), size=(n, ngrp))]
    sign = g.integers(0, 1 << N, size=(n, ngrp), dtype=np.uint16).astype(np.uint8) if N < 8 \
        else g.integers(0, 256, size=(n, ngrp), dtype=np.uint16).astype(np.uint8)

    salflag = np.zeros((nblk, BLOCK), dtype=bool)
    for b in range(nblk):
        k = 0 if max_salient == 0 else int(g.integers(1, max_salient + 1))
        if salient_counts is not None:
            k = int(salient_counts[b % len(salient_counts)])
        salflag[b, g.permutation(BLOCK)[:k]] = True
    sal_bits = np.packbits(salflag, axis=1, bitorder="little")         # [nblk][16] bytes
    salient = np.ascontiguousarray(sal_bits).view(np.uint64).reshape(nblk, 2).copy()

    region = np.zeros((n, ngrp), dtype=np.uint16)
    sign2 = np.zeros((n, nblk), dtype=np.uint32)
    cum_p = np.cumsum(region_p)
    rows_per_chunk = max(1, (1 << 24) // m)
    salcol = salflag.reshape(m)
    for r0 in range(0, n, rows_per_chunk):
        r1 = min(n, r0 + rows_per_chunk)
        kb = np.unpackbits(keep[r0:r1, :, None], axis=2, bitorder="little").astype(bool)
        rank = np.cumsum(kb, axis=2) - 1                                # [rows][ngrp][8]
        u = g.random((r1 - r0, ngrp, GROUP), dtype=np.float32)
        code = (u >= cum_p[0]).astype(np.uint16) + (u >= cum_p[1]).astype(np.uint16)
        code = np.where(salcol.reshape(1, ngrp, GROUP), np.uint16(3), code)
        contrib = np.where(kb, code << (2 * np.maximum(rank, 0)).astype(np.uint16), 0)
        region[r0:r1] = contrib.sum(axis=2).astype(np.uint16)
        # residual sign bits: t-th salient column (ascending) of each block, only if kept
        kcol = kb.reshape(r1 - r0, m)
        rb = g.integers(0, 2, size=(r1 - r0, m), dtype=np.uint8).astype(bool)
        for b in range(nblk):
            cols = np.nonzero(salflag[b])[0]
            for t, c in enumerate(cols):
                j = b * BLOCK + c
                sign2[r0:r1, b] |= ((kcol[:, j] & rb[:, j]).astype(np.uint32) << np.uint32(t))

    base = np.array([0.0125, 0.028, 0.06, 0.16, 0.05], dtype=np.float32)
    jitter = np.exp(0.25 * g.standard_normal((n, nblk, 5), dtype=np.float32))
    scale = (base * jitter).astype(np.float16).view(np.uint16)
    return {"n": n, "m": m, "N": N,
            "keep": np.ascontiguousarray(keep), "sign": np.ascontiguousarray(sign),
            "region": region, "sign2": sign2, "salient": salient,
            "scale": np.ascontiguousarray(scale)}


# LLaMA-2 linear shapes of the five workloads (n = output rows, m = input columns).
SHAPES_7B = {"q": (4096, 4096), "k": (4096, 4096), "v": (4096, 4096), "o": (4096, 4096),
             "gate": (11008, 4096), "up": (11008, 4096), "down": (4096, 11008)}
SHAPES_13B = {"q": (5120, 5120), "k": (5120, 5120), "v": (5120, 5120), "o": (5120, 5120),
              "gate": (13824, 5120), "up": (13824, 5120), "down": (5120, 13824)}
SHAPES_70B = {"q": (8192, 8192), "k": (1024, 8192), "v": (1024, 8192), "o": (8192, 8192),
              "gate": (28672, 8192), "up": (28672, 8192), "down": (8192, 28672)}


# Which dense layer (shape, N, seed) stands behind every named linear of the five workloads.  The seed
# feeds dense_weight / calib_norms; item numbers: workload 2: gate, up, down = 0, 1, 2; workloads 3 and 4:
# q, k, v, o, gate, up, down = 0..6; workload 5: one layer per (shape, N) family, item = 3 * shape + (N - 4)
# with shape 0 = 4096 x 4096, 1 = 11008 x 4096, 2 = 4096 x 11008 (the 32 decoder layers reuse the family's
# layer at distinct addresses: the kernels' work does not depend on which layer of a family it is).
_ORDER = ("q", "k", "v", "o", "gate", "up", "down")


def workload_layer(config: int, name: str, N: int = 0):
    """(n, m, N, seed) of linear `name` of workload `config` (1..5)."""
    if config == 1:
        return 4096, 4096, 4, seed_for(1, 0)
    if config == 2:
        n, m = SHAPES_7B[name]
        return n, m, 6, seed_for(2, ("gate", "up", "down").index(name))
    if config == 3:
        n, m = SHAPES_13B[name]
        return n, m, 5, seed_for(3, _ORDER.index(name))
    if config == 4:
        n, m = SHAPES_70B[name]
        return n, m, 4, seed_for(4, _ORDER.index(name))
    if config == 5:
        n, m = SHAPES_7B[name]
        shape = {(4096, 4096): 0, (11008, 4096): 1, (4096, 11008): 2}[(n, m)]
        assert N in (4, 5, 6)
        return n, m, N, seed_for(5, 3 * shape + (N - 4))
    raise ValueError(config)


def stack_N_per_layer(layers: int = 32):
    """Workload 5: N of each decoder layer, drawn from {4, 5, 6} (seeded)."""
    rng = np.random.default_rng(seed_for(5, 15))
    return [int(v) for v in rng.choice([4, 5, 6], size=layers)]
