"""The workloads' layers as the method makes them: dense synthetic weights and calibration norms
(stb_inputs) put through the oracle's quantizer (Algorithm 1 without the Hessian update, Algorithm 2),
with the logical arrays cached on disk because a LLaMA-sized layer takes the CPU quantizer tens of seconds.

TEST INFRASTRUCTURE like the rest of this package: used by tests/, by the smoke check and by bench.py to
PREPARE inputs and reference values.  Nothing here is on the product path.
"""
from __future__ import annotations

import hashlib
import os
import sys
import tempfile
import time

import numpy as np

import stb_inputs as si

from . import Logical, _SRC, quantize

_FIELDS = ("keep", "sign", "region", "sign2", "salient", "scale")


def cache_dir() -> str:
    d = os.environ.get("STB_CACHE_DIR") or os.path.join(tempfile.gettempdir(), "stb_quantized_layers")
    os.makedirs(d, exist_ok=True)
    return d


def _key(n, m, N, seed) -> str:
    h = hashlib.sha256()
    h.update(open(_SRC, "rb").read())
    h.update(open(si.__file__, "rb").read())
    return "q_%dx%d_N%d_s%x_%s.npz" % (n, m, N, seed, h.hexdigest()[:12])


def quantized_layer(n: int, m: int, N: int, seed: int, use_cache: bool = True, verbose: bool = False) -> dict:
    """Logical layer (dict of numpy arrays, the fields of stb_logical plus n, m, N) of
    quantize(dense_weight(n, m, seed), calib_norms(m, seed), N)."""
    path = os.path.join(cache_dir(), _key(n, m, N, seed))
    if use_cache and os.path.exists(path):
        try:
            z = np.load(path)
            d = {k: np.ascontiguousarray(z[k]) for k in _FIELDS}
            d.update(n=n, m=m, N=N)
            return d
        except Exception:  # noqa: BLE001  (a truncated file from an interrupted run: make it again)
            pass
    t0 = time.time()
    W = si.dense_weight(n, m, seed).astype(np.float64)
    L, _, _ = quantize(W, si.calib_norms(m, seed), N)
    del W
    d = {k: getattr(L, k) for k in _FIELDS}
    if use_cache:
        tmp = path + ".tmp%d.npz" % os.getpid()
        np.savez(tmp, **d)
        os.replace(tmp, path)
    d.update(n=n, m=m, N=N)
    if verbose:
        print("quantized %dx%d at %d:8 (seed %x) in %.1f s" % (n, m, N, seed, time.time() - t0), file=sys.stderr, flush=True)
    return d


def as_logical(d: dict) -> Logical:
    return Logical(d["n"], d["m"], d["N"], *(d[k] for k in _FIELDS))


def salient_counts(d: dict) -> np.ndarray:
    """Salient columns per 128-column block."""
    return np.array([bin(int(a) | (int(b) << 64)).count("1") for a, b in d["salient"]], dtype=np.int32)


def stream_bytes(d: dict) -> int:
    """Bytes of the layer that one decode pass reads: 16 (mask) + 2 N (signs) + 4 N (regions) + 10 (five
    scales) per row and block, plus two residual bits per salient column of the block rounded up to a byte;
    rows padded to tiles of 32."""
    rows = -(-d["n"] // 32) * 32
    return int(rows * sum(26 + 6 * d["N"] + -(-int(s) // 4) for s in salient_counts(d)))
