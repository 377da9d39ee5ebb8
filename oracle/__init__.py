"""ctypes front end of the CPU oracle (oracle/stb_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this package, and this package never imports them.

All arithmetic lives in the C++ file; this module only compiles it (g++) and
marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "stb_oracle.cpp")
_LIB = os.path.join(_HERE, "libstb_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle into oracle/libstb_oracle.so (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread",
                               "-ffp-contract=off", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.stbo_half_to_float.restype = C.c_float
        _lib.stbo_half_to_float.argtypes = [C.c_uint16]
        _lib.stbo_double_to_half.restype = C.c_uint16
        _lib.stbo_double_to_half.argtypes = [C.c_double]
        _lib.stbo_average_bits.restype = C.c_double
        _lib.stbo_average_bits.argtypes = [C.c_int, C.c_double]
        _lib.stbo_counted_bits.restype = C.c_double
        _lib.stbo_salient_search.restype = C.c_int
        _lib.stbo_breakpoint_search.restype = C.c_int
        _lib.stbo_hardware_threads.restype = C.c_int
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _c(a, dt):
    return np.ascontiguousarray(a, dtype=dt)


def hardware_threads() -> int:
    return int(lib().stbo_hardware_threads())


@dataclass
class Logical:
    """Logical (unpacked) structured-binary layer; field layout as in stb_oracle.cpp."""
    n: int
    m: int
    N: int
    keep: np.ndarray      # u8  [n][m/8]
    sign: np.ndarray      # u8  [n][m/8]
    region: np.ndarray    # u16 [n][m/8]
    sign2: np.ndarray     # u32 [n][m/128]
    salient: np.ndarray   # u64 [m/128][2]
    scale: np.ndarray     # u16 [n][m/128][5]  (fp16 bits)

    def check(self):
        n, m = self.n, self.m
        assert self.keep.shape == (n, m // 8) and self.keep.dtype == np.uint8
        assert self.sign.shape == (n, m // 8) and self.sign.dtype == np.uint8
        assert self.region.shape == (n, m // 8) and self.region.dtype == np.uint16
        assert self.sign2.shape == (n, m // 128) and self.sign2.dtype == np.uint32
        assert self.salient.shape == (m // 128, 2) and self.salient.dtype == np.uint64
        assert self.scale.shape == (n, m // 128, 5) and self.scale.dtype == np.uint16
        for a in (self.keep, self.sign, self.region, self.sign2, self.salient, self.scale):
            assert a.flags["C_CONTIGUOUS"]


def half_to_float(h: int) -> float:
    return float(lib().stbo_half_to_float(int(h)))


def double_to_half(x: float) -> int:
    return int(lib().stbo_double_to_half(float(x)))


def si_scores(W, xnorm):
    W = _c(W, np.float64); xnorm = _c(xnorm, np.float64)
    n, m = W.shape
    S = np.empty((n, m), np.float64)
    lib().stbo_si_scores(_p(W), _p(xnorm), C.c_int(n), C.c_int(m), _p(S))
    return S


def nm_select(S, N):
    S = _c(S, np.float64)
    n, m = S.shape
    keep = np.empty((n, m // 8), np.uint8)
    lib().stbo_nm_select(_p(S), C.c_int(n), C.c_int(m), C.c_int(N), _p(keep))
    return keep


def salient_search(W, keep, xnorm, lam, b):
    """Returns (n_star, candidate order[32], errors[32]) for block b."""
    W = _c(W, np.float64); keep = _c(keep, np.uint8); xnorm = _c(xnorm, np.float64)
    n, m = W.shape
    order = np.empty(32, np.int32); errs = np.empty(32, np.float64)
    ns = lib().stbo_salient_search(_p(W), _p(keep), _p(xnorm), C.c_double(lam), C.c_int(n),
                                   C.c_int(m), C.c_int(b), _p(order), _p(errs))
    return int(ns), order, errs


def breakpoint_search(W, keep, salflag, b):
    """Returns (p1*, p2*, evaluated, errors[160]) for block b; salflag is u8[128]."""
    W = _c(W, np.float64); keep = _c(keep, np.uint8); salflag = _c(salflag, np.uint8)
    n, m = W.shape
    p1 = C.c_double(); p2 = C.c_double(); errs = np.empty(160, np.float64)
    ev = lib().stbo_breakpoint_search(_p(W), _p(keep), _p(salflag), C.c_int(n), C.c_int(m),
                                      C.c_int(b), C.byref(p1), C.byref(p2), _p(errs))
    return p1.value, p2.value, int(ev), errs


def quantize(W, xnorm, N, lam=-1.0, nthreads=0):
    """Run the quantizer; returns (Logical, breakpoints[nblk][2], nsal[nblk])."""
    W = _c(W, np.float64); xnorm = _c(xnorm, np.float64)
    n, m = W.shape
    assert m % 128 == 0 and 1 <= N <= 8
    L = Logical(n, m, N,
                np.zeros((n, m // 8), np.uint8), np.zeros((n, m // 8), np.uint8),
                np.zeros((n, m // 8), np.uint16), np.zeros((n, m // 128), np.uint32),
                np.zeros((m // 128, 2), np.uint64), np.zeros((n, m // 128, 5), np.uint16))
    bp = np.zeros((m // 128, 2), np.float64); nsal = np.zeros(m // 128, np.int32)
    lib().stbo_quantize(_p(W), _p(xnorm), C.c_int(n), C.c_int(m), C.c_int(N), C.c_double(lam),
                        _p(L.keep), _p(L.sign), _p(L.region), _p(L.sign2), _p(L.salient),
                        _p(L.scale), _p(bp), _p(nsal),
                        C.c_int(nthreads or hardware_threads()))
    return L, bp, nsal


def decode(L: Logical):
    """fp32 decode of the logical layer, [n][m]."""
    L.check()
    What = np.empty((L.n, L.m), np.float32)
    lib().stbo_decode(C.c_int(L.n), C.c_int(L.m), _p(L.keep), _p(L.sign), _p(L.region),
                      _p(L.sign2), _p(L.salient), _p(L.scale), _p(What))
    return What


def matmul(What, x, nthreads=0):
    """float64 y[T][n] = x[T][m] @ What^T from the fp32-decoded matrix."""
    What = _c(What, np.float32); x = _c(np.atleast_2d(x), np.float64)
    n, m = What.shape
    T = x.shape[0]
    assert x.shape[1] == m
    y = np.empty((T, n), np.float64)
    lib().stbo_matmul(_p(What), C.c_int(n), C.c_int(m), _p(x), C.c_int(T), C.c_int(m), _p(y),
                      C.c_int(nthreads or hardware_threads()))
    return y


def layer_rows(L: Logical, rows, x, nthreads=0):
    """float64 y[T][len(rows)] for the listed output rows (decode + multiply)."""
    L.check()
    rows = _c(rows, np.int32); x = _c(np.atleast_2d(x), np.float64)
    T = x.shape[0]
    assert x.shape[1] == L.m
    y = np.empty((T, len(rows)), np.float64)
    lib().stbo_layer_rows(C.c_int(L.n), C.c_int(L.m), _p(L.keep), _p(L.sign), _p(L.region),
                          _p(L.sign2), _p(L.salient), _p(L.scale), _p(rows),
                          C.c_int(len(rows)), _p(x), C.c_int(T), C.c_int(L.m), _p(y),
                          C.c_int(nthreads or hardware_threads()))
    return y


def silu_mul(a, b):
    """fp16 values (as float64) of silu(a) * b evaluated in float64: the gated MLP activation (not from the paper)."""
    a = _c(a, np.float64); b = _c(b, np.float64)
    assert a.shape == b.shape
    out = np.empty(a.shape, np.uint16)
    lib().stbo_silu_mul(_p(a), _p(b), C.c_int(a.size), _p(out))
    return out.view(np.float16).astype(np.float64)


def allocate_nm(l2norms, r_target):
    """Layer-wise N:M assignment (Section 3.3): returns (N per layer, unrounded ratios)."""
    w = _c(l2norms, np.float64)
    N = np.empty(len(w), np.int32); ratio = np.empty(len(w), np.float64)
    lib().stbo_allocate_nm(_p(w), C.c_int(len(w)), C.c_double(r_target), _p(N), _p(ratio))
    return N, ratio


def average_bits(N, r_salient):
    return float(lib().stbo_average_bits(C.c_int(N), C.c_double(r_salient)))


def counted_bits(L: Logical):
    """(bits per weight position carried by sign + residual-sign fields, r_salient)."""
    r = C.c_double()
    v = lib().stbo_counted_bits(C.c_int(L.n), C.c_int(L.m), _p(L.keep), _p(L.salient),
                                C.byref(r))
    return float(v), r.value
