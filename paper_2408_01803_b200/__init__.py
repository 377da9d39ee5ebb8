"""Python binding of libstb.so: the N:M structured-binary linear layer on B200 (sm_100a).

Argument marshalling only: every step of the path (pack, dequant, GEMV, GEMM, layer stack)
runs in the CUDA kernels behind the C ABI declared in include/stb.h.  torch is used for
device memory and streams.  There is no CPU fallback: the shared library is loaded on the
first call of any function here, and a missing library raises ImportError at that point
(`python -m paper_2408_01803_b200.build` compiles it; importing the package alone must work
without it so that the build module can be reached).
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libstb.so")

STB_OK, STB_ERR_ARG, STB_ERR_SHAPE, STB_ERR_NM, STB_ERR_SIZE = 0, 1, 2, 3, 4
STB_ERR_UNSUPPORTED, STB_ERR_CORRUPT, STB_ERR_TIMEOUT, STB_ERR_CUDA = 5, 6, 7, 8
STB_F16, STB_BF16, STB_F32 = 0, 1, 2
STB_IN_PLAIN, STB_IN_SILU_MUL = 0, 1

EXPORTS = ["stb_pack_size", "stb_pack", "stb_packed_info", "stb_dequant", "stb_gemv", "stb_gemv_wait_selftest",
           "stb_gemm_workspace", "stb_gemm_workspace_min", "stb_gemm", "stb_gemm_f16_workspace", "stb_gemm_f16", "stb_gemm_noalloc", "stb_layer_stack", "stb_layer_stack_host",
           "stb_layer_stack_resident_workspace", "stb_layer_stack_resident", "stb_layer_stack_resident_host",
           "stb_layer_stack_resident_wait_selftest", "stb_layer_stack_checksum", "stb_quantize_workspace", "stb_quantize", "stb_weight_sumsq",
           "stb_allocate_nm", "stb_status_str"]


class StbError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, status_str(status), status))


class _Logical(C.Structure):
    _fields_ = [("n", C.c_int), ("m", C.c_int), ("N", C.c_int),
                ("keep", C.c_void_p), ("sign", C.c_void_p), ("region", C.c_void_p),
                ("sign2", C.c_void_p), ("salient", C.c_void_p), ("scale", C.c_void_p)]


class _Info(C.Structure):
    _fields_ = [("n", C.c_int), ("m", C.c_int), ("N", C.c_int), ("status", C.c_int),
                ("used_bytes", C.c_uint64), ("stream_bytes", C.c_uint64)]


class _Step(C.Structure):
    _fields_ = [("packed", C.c_void_p), ("n", C.c_int), ("m", C.c_int), ("N", C.c_int),
                ("inp", C.c_void_p), ("out", C.c_void_p), ("odt", C.c_int), ("batch", C.c_int),
                ("ldin", C.c_size_t), ("ldout", C.c_size_t), ("in2", C.c_void_p), ("input", C.c_int)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError("libstb.so is not built (%s): run `python -m paper_2408_01803_b200.build`; "
                          "there is no CPU fallback" % LIB_PATH)
    lib = C.CDLL(LIB_PATH)
    v, i, z, p = C.c_void_p, C.c_int, C.c_size_t, C.POINTER
    lib.stb_pack_size.argtypes = [i, i, i, p(z)]
    lib.stb_pack.argtypes = [p(_Logical), v, z, v, v]
    lib.stb_packed_info.argtypes = [v, p(_Info), v]
    lib.stb_dequant.argtypes = [v, i, i, i, v, i, z, v]
    lib.stb_gemv.argtypes = [v, i, i, i, v, i, z, v, i, z, v, v]
    lib.stb_gemv_wait_selftest.argtypes = [v, i, i, i, v, i, z, v, i, z, v, v]
    lib.stb_gemm_workspace.argtypes = [i, i, i, i, p(z)]
    lib.stb_gemm_workspace_min.argtypes = [i, i, i, i, p(z)]
    lib.stb_gemm.argtypes = [v, i, i, i, v, i, z, v, i, z, v, z, v, v]
    lib.stb_gemm_f16_workspace.argtypes = [i, i, i, i, p(z)]
    lib.stb_gemm_f16.argtypes = [v, i, i, i, v, i, z, v, i, z, v, z, v, v]
    lib.stb_gemm_noalloc.argtypes = [v, i, i, i, v, i, z, v, i, z, v, v]
    lib.stb_layer_stack.argtypes = [p(_Step), i, v, v]
    lib.stb_layer_stack_host.argtypes = [p(_Step), i, v, z, v, z, v, v]
    lib.stb_layer_stack_resident_workspace.argtypes = [p(_Step), i, p(z)]
    lib.stb_layer_stack_resident.argtypes = [p(_Step), i, v, z, v, v]
    lib.stb_layer_stack_resident_wait_selftest.argtypes = [p(_Step), i, v, z, v, v]
    lib.stb_layer_stack_resident_host.argtypes = [p(_Step), i, v, z, v, z, v, z, v, v]
    lib.stb_layer_stack_checksum.argtypes = [p(_Step), i, v, v, v]
    lib.stb_quantize_workspace.argtypes = [i, i, p(z)]
    lib.stb_quantize.argtypes = [v, z, v, i, i, i, C.c_double, p(_Logical), v, z, v]
    lib.stb_weight_sumsq.argtypes = [v, i, i, z, v, v]
    lib.stb_allocate_nm.argtypes = [p(C.c_double), i, C.c_double, p(i)]
    lib.stb_status_str.argtypes = [i]
    lib.stb_status_str.restype = C.c_char_p
    for name in EXPORTS:
        if name != "stb_status_str":
            getattr(lib, name).restype = i
    return lib


class _LazyLib:
    """Loads libstb.so on first attribute access; raises ImportError if it is not built."""
    _real = None

    def __getattr__(self, name):
        if _LazyLib._real is None:
            _LazyLib._real = _load()
        return getattr(_LazyLib._real, name)


_lib = _LazyLib()


def status_str(status: int) -> str:
    return _lib.stb_status_str(int(status)).decode()


def _check(rc: int, where: str):
    if rc != STB_OK:
        raise StbError(rc, where)


def _stream(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(0)


def pack_size(n: int, m: int, N: int) -> int:
    out = C.c_size_t()
    _check(_lib.stb_pack_size(n, m, N, C.byref(out)), "stb_pack_size")
    return out.value


@dataclass
class PackedLayer:
    """A packed layer: the device buffer and the three integers every call needs."""
    n: int
    m: int
    N: int
    buf: "object"        # torch.uint8 CUDA tensor
    dev_status: "object"  # torch.int32[1] CUDA tensor

    def info(self, stream=None) -> dict:
        inf = _Info()
        _check(_lib.stb_packed_info(_ptr(self.buf), C.byref(inf), _stream(stream)), "stb_packed_info")
        return {"n": inf.n, "m": inf.m, "N": inf.N, "status": inf.status,
                "used_bytes": inf.used_bytes, "stream_bytes": inf.stream_bytes}


def pack(n, m, N, keep, sign, region, sign2, salient, scale, stream=None, buf=None) -> PackedLayer:
    """stb_pack: logical CUDA tensors (uint8/uint8/int16-as-u16/int32-as-u32/int64-as-u64/
    int16-as-fp16-bits, C-contiguous) -> PackedLayer."""
    import torch
    dev = keep.device
    for t in (keep, sign, region, sign2, salient, scale):
        assert t.is_cuda and t.is_contiguous()
    if buf is None:
        buf = torch.empty(pack_size(n, m, N), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    L = _Logical(n, m, N, keep.data_ptr(), sign.data_ptr(), region.data_ptr(), sign2.data_ptr(),
                 salient.data_ptr(), scale.data_ptr())
    _check(_lib.stb_pack(C.byref(L), _ptr(buf), buf.numel(), _ptr(status), _stream(stream)), "stb_pack")
    return PackedLayer(n, m, N, buf, status)


def pack_numpy(d: dict, device="cuda", stream=None) -> PackedLayer:
    """Convenience: upload a logical layer given as numpy arrays (the dict of
    stb_inputs.logical_layer or the fields of an oracle.Logical) and pack it."""
    import numpy as np
    import torch
    def up(a, view):
        return torch.from_numpy(np.ascontiguousarray(a).view(view)).to(device)
    return pack(int(d["n"]), int(d["m"]), int(d["N"]), up(d["keep"], np.uint8), up(d["sign"], np.uint8),
                up(d["region"], np.int16), up(d["sign2"], np.int32), up(d["salient"], np.int64),
                up(d["scale"], np.int16), stream=stream)


def dequant(layer: PackedLayer, dtype=None, out=None, stream=None):
    import torch
    dtype = dtype or torch.float32
    dt = {torch.float32: STB_F32, torch.float16: STB_F16, torch.bfloat16: STB_BF16}[dtype]
    if out is None:
        out = torch.empty((layer.n, layer.m), dtype=dtype, device=layer.buf.device)
    assert out.dtype == dtype and out.stride(1) == 1
    _check(_lib.stb_dequant(_ptr(layer.buf), layer.n, layer.m, layer.N, _ptr(out), dt, out.stride(0),
                            _stream(stream)), "stb_dequant")
    return out


def gemv(layer: PackedLayer, x, out=None, out_dtype=None, stream=None):
    """stb_gemv: x fp16 [batch][m] (or [m]) -> y [batch][n] fp32 (or fp16)."""
    import torch
    x2 = x if x.dim() == 2 else x.unsqueeze(0)
    assert x2.dtype == torch.float16 and x2.is_cuda and x2.stride(1) == 1
    batch = x2.shape[0]
    if out is None:
        out = torch.empty((batch, layer.n), dtype=out_dtype or torch.float32, device=x.device)
    ydt = {torch.float32: STB_F32, torch.float16: STB_F16}[out.dtype]
    _check(_lib.stb_gemv(_ptr(layer.buf), layer.n, layer.m, layer.N, _ptr(x2), batch, x2.stride(0),
                         _ptr(out), ydt, out.stride(0), _ptr(layer.dev_status), _stream(stream)), "stb_gemv")
    return out if x.dim() == 2 else out[0]


def gemv_wait_selftest(layer: PackedLayer, x, out, dev_status, stream=None):
    """stb_gemv_wait_selftest: the GEMV kernel with its copies off and a short wait limit; dev_status
    (torch.int32[1], zeroed) becomes STB_ERR_TIMEOUT."""
    x2 = x if x.dim() == 2 else x.unsqueeze(0)
    ydt = STB_F32 if out.element_size() == 4 else STB_F16
    _check(_lib.stb_gemv_wait_selftest(_ptr(layer.buf), layer.n, layer.m, layer.N, _ptr(x2), x2.shape[0], x2.stride(0),
                                       _ptr(out), ydt, out.stride(-2) if out.dim() == 2 else layer.n, _ptr(dev_status),
                                       _stream(stream)), "stb_gemv_wait_selftest")


def gemm_workspace(n, m, N, T, minimum=False) -> int:
    out = C.c_size_t()
    fn = _lib.stb_gemm_workspace_min if minimum else _lib.stb_gemm_workspace
    _check(fn(n, m, N, T, C.byref(out)), "stb_gemm_workspace")
    return out.value


def gemm(layer: PackedLayer, X, out=None, out_dtype=None, ws=None, stream=None):
    """stb_gemm: X bf16 [T][m] -> Y [T][n] fp32 (or bf16)."""
    import torch
    assert X.dtype == torch.bfloat16 and X.is_cuda and X.dim() == 2 and X.stride(1) == 1
    T = X.shape[0]
    if out is None:
        out = torch.empty((T, layer.n), dtype=out_dtype or torch.float32, device=X.device)
    ydt = {torch.float32: STB_F32, torch.bfloat16: STB_BF16}[out.dtype]
    need = gemm_workspace(layer.n, layer.m, layer.N, T)
    if need and (ws is None or ws.numel() * ws.element_size() < need):
        ws = torch.empty(need, dtype=torch.uint8, device=X.device)
    _check(_lib.stb_gemm(_ptr(layer.buf), layer.n, layer.m, layer.N, _ptr(X), T, X.stride(0), _ptr(out),
                         ydt, out.stride(0), _ptr(ws), (ws.numel() * ws.element_size()) if ws is not None else 0,
                         _ptr(layer.dev_status), _stream(stream)), "stb_gemm")
    return out


def gemm_f16_workspace(n, m, N, T) -> int:
    out = C.c_size_t()
    _check(_lib.stb_gemm_f16_workspace(n, m, N, T, C.byref(out)), "stb_gemm_f16_workspace")
    return out.value


def gemm_f16(layer: PackedLayer, X, out=None, out_dtype=None, ws=None, stream=None):
    """stb_gemm_f16: X fp16 [T][m] -> Y [T][n] fp32 (or fp16); exact fp16 scales, the small token tile for T <= 64."""
    import torch
    assert X.dtype == torch.float16 and X.is_cuda and X.dim() == 2 and X.stride(1) == 1
    T = X.shape[0]
    if out is None:
        out = torch.empty((T, layer.n), dtype=out_dtype or torch.float32, device=X.device)
    ydt = {torch.float32: STB_F32, torch.float16: STB_F16}[out.dtype]
    need = gemm_f16_workspace(layer.n, layer.m, layer.N, T)
    if ws is None or ws.numel() * ws.element_size() < need:
        ws = torch.empty(max(need, 256), dtype=torch.uint8, device=X.device)
    _check(_lib.stb_gemm_f16(_ptr(layer.buf), layer.n, layer.m, layer.N, _ptr(X), T, X.stride(0), _ptr(out),
                             ydt, out.stride(0), _ptr(ws), ws.numel() * ws.element_size(),
                             _ptr(layer.dev_status), _stream(stream)), "stb_gemm_f16")
    return out


def gemm_noalloc(layer: PackedLayer, X, out, stream=None):
    """stb_gemm_noalloc: like gemm(), for hosts that may not allocate device memory while running:
    the caller brings X and `out` (fp32 or bf16 [T][n]); split-K partial sums use the 8 MiB array
    built into the library.  Raises StbError(STB_ERR_SIZE) for shapes that need more."""
    import torch
    assert X.dtype == torch.bfloat16 and X.is_cuda and X.dim() == 2 and X.stride(1) == 1
    assert out.is_cuda and out.dim() == 2 and out.stride(1) == 1 and out.shape == (X.shape[0], layer.n)
    ydt = {torch.float32: STB_F32, torch.bfloat16: STB_BF16}[out.dtype]
    _check(_lib.stb_gemm_noalloc(_ptr(layer.buf), layer.n, layer.m, layer.N, _ptr(X), X.shape[0], X.stride(0),
                                 _ptr(out), ydt, out.stride(0), _ptr(layer.dev_status), _stream(stream)),
           "stb_gemm_noalloc")
    return out


def make_steps(steps):
    """Marshal a list of (layer, x, out) or (layer, (gate, up), out) into the C array stb_layer_stack takes; a pair
    as input means x = silu(gate) * up (STB_IN_SILU_MUL, stb_layer_stack_resident only)."""
    import torch
    arr = (_Step * len(steps))()
    for k, (layer, x, out) in enumerate(steps):
        second = None
        if isinstance(x, (tuple, list)):
            x, second = x
        x2 = x if x.dim() == 2 else x.unsqueeze(0)
        o2 = out if out.dim() == 2 else out.unsqueeze(0)
        assert x2.dtype == torch.float16 and x2.stride(1) == 1 and o2.stride(1) == 1
        in2, mode = 0, STB_IN_PLAIN
        if second is not None:
            s2 = second if second.dim() == 2 else second.unsqueeze(0)
            assert s2.dtype == torch.float16 and s2.stride(1) == 1 and s2.stride(0) == x2.stride(0) and s2.shape == x2.shape
            in2, mode = s2.data_ptr(), STB_IN_SILU_MUL
        odt = {torch.float32: STB_F32, torch.float16: STB_F16}[o2.dtype]
        arr[k] = _Step(layer.buf.data_ptr(), layer.n, layer.m, layer.N, x2.data_ptr(), o2.data_ptr(), odt,
                       x2.shape[0], x2.stride(0), o2.stride(0), in2, mode)
    return arr


def layer_stack(steps, dev_status=None, stream=None, marshalled=None):
    """stb_layer_stack over a list of (PackedLayer, x, out) triples (or a pre-marshalled array)."""
    arr = marshalled if marshalled is not None else make_steps(steps)
    _check(_lib.stb_layer_stack(arr, len(arr), _ptr(dev_status), _stream(stream)), "stb_layer_stack")


def layer_stack_host(marshalled, x_host, y_host, dev_status=None, stream=None):
    """stb_layer_stack_host: x_host / y_host are pinned CPU tensors; the first step's input and
    the last step's output (device tensors named in `marshalled`) are the staging buffers."""
    _check(_lib.stb_layer_stack_host(marshalled, len(marshalled), C.c_void_p(x_host.data_ptr()),
                                     x_host.numel() * x_host.element_size(), C.c_void_p(y_host.data_ptr()),
                                     y_host.numel() * y_host.element_size(), _ptr(dev_status), _stream(stream)),
           "stb_layer_stack_host")


def resident_workspace(marshalled, device="cuda"):
    """A zeroed workspace (torch.uint8 CUDA tensor) of the size stb_layer_stack_resident wants for these steps."""
    import torch
    out = C.c_size_t()
    _check(_lib.stb_layer_stack_resident_workspace(marshalled, len(marshalled), C.byref(out)),
           "stb_layer_stack_resident_workspace")
    return torch.zeros(max(out.value, 256), dtype=torch.uint8, device=device)


def layer_stack_resident(steps, ws, dev_status=None, stream=None, marshalled=None, selftest=False):
    """stb_layer_stack_resident over a list of (PackedLayer, x, out) triples (or a pre-marshalled array);
    ws from resident_workspace().  selftest=True runs the wait self-test instead."""
    arr = marshalled if marshalled is not None else make_steps(steps)
    fn = _lib.stb_layer_stack_resident_wait_selftest if selftest else _lib.stb_layer_stack_resident
    _check(fn(arr, len(arr), _ptr(ws), ws.numel(), _ptr(dev_status), _stream(stream)), "stb_layer_stack_resident")


def layer_stack_resident_host(marshalled, ws, x_host, y_host, dev_status=None, stream=None):
    """stb_layer_stack_resident_host: x_host / y_host are pinned CPU tensors."""
    _check(_lib.stb_layer_stack_resident_host(marshalled, len(marshalled), _ptr(ws), ws.numel(),
                                              C.c_void_p(x_host.data_ptr()), x_host.numel() * x_host.element_size(),
                                              C.c_void_p(y_host.data_ptr()), y_host.numel() * y_host.element_size(),
                                              _ptr(dev_status), _stream(stream)), "stb_layer_stack_resident_host")


def layer_stack_checksum(marshalled, sums=None, dev_status=None, stream=None):
    """stb_layer_stack_checksum: XOR of the streamed words of every step's packed layer -> torch.int64[count]."""
    import torch
    if sums is None:
        sums = torch.zeros(len(marshalled), dtype=torch.int64, device="cuda")
    _check(_lib.stb_layer_stack_checksum(marshalled, len(marshalled), _ptr(sums), _ptr(dev_status), _stream(stream)),
           "stb_layer_stack_checksum")
    return sums


def allocate_nm(weights, r_target, stream=None):
    """Layer-wise N:M assignment (stb_weight_sumsq per layer, then stb_allocate_nm): `weights` is a list of dense fp16
    CUDA matrices; returns the list of N."""
    import torch
    sums = torch.zeros(len(weights), dtype=torch.float64, device=weights[0].device)
    for k, W in enumerate(weights):
        assert W.dtype == torch.float16 and W.dim() == 2 and W.stride(1) == 1
        _check(_lib.stb_weight_sumsq(_ptr(W), W.shape[0], W.shape[1], W.stride(0), C.c_void_p(sums.data_ptr() + 8 * k),
                                     _stream(stream)), "stb_weight_sumsq")
    host = sums.cpu().numpy()
    arr = (C.c_double * len(weights))(*[float(vv) for vv in host])
    out = (C.c_int * len(weights))()
    _check(_lib.stb_allocate_nm(arr, len(weights), float(r_target), out), "stb_allocate_nm")
    return [int(vv) for vv in out], host


def quantize(W, xnorm, N, lam=-1.0, stream=None):
    """stb_quantize: dense fp16 CUDA matrix W[n][m] + float64 CUDA column norms xnorm[m] -> dict of logical CUDA
    tensors (keep, sign, region, sign2, salient, scale; the argument order of pack())."""
    import torch
    assert W.dtype == torch.float16 and W.is_cuda and W.dim() == 2 and W.stride(1) == 1
    assert xnorm.dtype == torch.float64 and xnorm.is_cuda and xnorm.is_contiguous()
    n, m = W.shape
    dev = W.device
    out = {"keep": torch.empty((n, m // 8), dtype=torch.uint8, device=dev), "sign": torch.empty((n, m // 8), dtype=torch.uint8, device=dev),
           "region": torch.empty((n, m // 8), dtype=torch.int16, device=dev), "sign2": torch.empty((n, m // 128), dtype=torch.int32, device=dev),
           "salient": torch.empty((m // 128, 2), dtype=torch.int64, device=dev), "scale": torch.empty((n, m // 128, 5), dtype=torch.int16, device=dev)}
    need = C.c_size_t()
    _check(_lib.stb_quantize_workspace(n, m, C.byref(need)), "stb_quantize_workspace")
    ws = torch.empty(need.value, dtype=torch.uint8, device=dev)
    L = _Logical(n, m, N, out["keep"].data_ptr(), out["sign"].data_ptr(), out["region"].data_ptr(), out["sign2"].data_ptr(),
                 out["salient"].data_ptr(), out["scale"].data_ptr())
    _check(_lib.stb_quantize(_ptr(W), W.stride(0), _ptr(xnorm), n, m, N, float(lam), C.byref(L), _ptr(ws), ws.numel(), _stream(stream)),
           "stb_quantize")
    out.update(n=n, m=m, N=N)
    return out
