"""The C-ABI library loads on a machine without a GPU, exports every symbol that include/stb.h
declares, and rejects bad arguments on the host before any CUDA call."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def stb():
    from paper_2408_01803_b200 import build
    build.build()
    import paper_2408_01803_b200 as stb
    return stb


def test_every_declared_symbol_is_exported(stb):
    hdr = open(os.path.join(ROOT, "include", "stb.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(stb_[a-z_0-9]+)\s*\(", hdr))
    assert {"stb_pack", "stb_gemv", "stb_gemm", "stb_layer_stack", "stb_pack_size", "stb_dequant"} <= names
    lib = C.CDLL(stb.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert names == set(stb.EXPORTS)


def test_pack_size_formula_and_errors(stb):
    # 50 / 56 / 62 bytes per row-block at 4:8 / 5:8 / 6:8 plus at most 8 residual bytes
    # (two bits for each of up to 32 salient columns)
    for N, per in ((4, 50), (5, 56), (6, 62)):
        n, m = 4096, 4096
        hdr = (64 + 128 * (m // 128) + 255) // 256 * 256       # header, block table, residual word table
        assert stb.pack_size(n, m, N) == hdr + (n // 32) * (m // 128) * 32 * (per + 8)
    assert stb.pack_size(33, 128, 4) == 256 + 2 * 32 * 58      # ragged rows pad to a tile of 32
    for args, code in (((0, 128, 4), stb.STB_ERR_SHAPE), ((8, 100, 4), stb.STB_ERR_SHAPE),
                       ((8, 0, 4), stb.STB_ERR_SHAPE), ((8, 128, 0), stb.STB_ERR_NM), ((8, 128, 9), stb.STB_ERR_NM)):
        with pytest.raises(stb.StbError) as e:
            stb.pack_size(*args)
        assert e.value.status == code


def test_host_side_argument_checks_launch_nothing(stb):
    lib = stb._lib
    null = C.c_void_p(0)
    one = C.c_void_p(256)          # never dereferenced: every call below fails validation first
    assert lib.stb_pack(None, one, 1 << 20, null, null) == stb.STB_ERR_ARG
    L = stb._Logical(32, 128, 4, 256, 256, 256, 256, 256, 256)
    assert lib.stb_pack(C.byref(L), null, 1 << 20, null, null) == stb.STB_ERR_ARG
    assert lib.stb_pack(C.byref(L), one, 16, null, null) == stb.STB_ERR_SIZE
    L.N = 9
    assert lib.stb_pack(C.byref(L), one, 1 << 20, null, null) == stb.STB_ERR_NM
    L.N = 4; L.m = 130
    assert lib.stb_pack(C.byref(L), one, 1 << 20, null, null) == stb.STB_ERR_SHAPE
    L.m = 128; L.keep = 257
    assert lib.stb_pack(C.byref(L), one, 1 << 20, null, null) == stb.STB_ERR_ARG      # misaligned
    assert lib.stb_gemv(null, 32, 128, 4, one, 1, 128, one, stb.STB_F32, 32, null, null) == stb.STB_ERR_ARG
    assert lib.stb_gemv(one, 32, 128, 4, one, 0, 128, one, stb.STB_F32, 32, null, null) == stb.STB_ERR_SIZE
    assert lib.stb_gemv(one, 32, 128, 4, one, 65, 128, one, stb.STB_F32, 32, null, null) == stb.STB_ERR_SIZE
    assert lib.stb_gemv(one, 32, 128, 4, one, 1, 64, one, stb.STB_F32, 32, null, null) == stb.STB_ERR_ARG
    assert lib.stb_gemv(one, 32, 128, 4, one, 1, 128, one, stb.STB_BF16, 32, null, null) == stb.STB_ERR_UNSUPPORTED
    assert lib.stb_dequant(one, 32, 128, 4, one, 7, 128, null) == stb.STB_ERR_UNSUPPORTED
    assert lib.stb_dequant(one, 32, 128, 4, one, stb.STB_F32, 64, null) == stb.STB_ERR_ARG
    assert lib.stb_layer_stack(None, 1, null, null) == stb.STB_ERR_ARG
    assert stb.status_str(stb.STB_ERR_TIMEOUT).startswith("a bounded")


def test_packed_layout_and_byte_permute_decode_on_the_host(tmp_path):
    """tests/host_layout_check.cu: the layout's index arithmetic, the pack-side word builder and the
    byte-permute decode used by the tensor-core kernels, compiled for the host and checked against the
    logical fields for N = 1..8."""
    import shutil
    import subprocess
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    exe = str(tmp_path / "host_layout_check")
    subprocess.check_call([nvcc, "-std=c++17", "-O1", "-Wno-deprecated-gpu-targets", "-o", exe,
                           os.path.join(ROOT, "tests", "host_layout_check.cu")])
    out = subprocess.run([exe], capture_output=True, text=True)
    assert out.returncode == 0, out.stdout[-2000:]
    assert "OK: 0 errors" in out.stdout


def test_layerwise_assignment_host_arithmetic_matches_the_oracle(stb):
    """stb_allocate_nm (host arithmetic of the library) against the oracle's Section 3.3 assignment."""
    import numpy as np
    import oracle
    g = np.random.default_rng(11)
    for R in (0.5, 0.625, 0.75):
        norms = g.random(37) * 10 + 0.05
        want, _ = oracle.allocate_nm(norms, R)
        arr = (C.c_double * 37)(*[float(v * v) for v in norms])
        out = (C.c_int * 37)()
        assert stb._lib.stb_allocate_nm(arr, 37, R, out) == stb.STB_OK
        assert [int(v) for v in out] == [int(v) for v in want]
    assert stb._lib.stb_allocate_nm(None, 3, 0.5, out) == stb.STB_ERR_ARG
    assert stb._lib.stb_allocate_nm(arr, 3, 0.0, out) == stb.STB_ERR_ARG
