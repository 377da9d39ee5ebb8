"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

  * stb_pack + stb_dequant: fp32 decode bit-exact against the oracle's decode (-0 == +0).
  * stb_gemv: max|y_gpu - y_ref| <= 5e-3 * max|y_ref| against the float64
    dequantise-then-matmul of the oracle.
"""
import numpy as np
import pytest

import oracle
import oracle.workloads as wl
import stb_inputs as si

pytestmark = pytest.mark.gpu
TOL = 5e-3          # max|y_gpu - y_ref| <= TOL * max|y_ref|, for fp32 and for 16-bit outputs alike


@pytest.fixture(scope="module")
def stb():
    import torch
    assert torch.cuda.is_available()
    from paper_2408_01803_b200 import build
    build.build()                      # no-op when libstb.so is newer than its sources
    import paper_2408_01803_b200 as stb
    return stb


def _fields(L):
    return {"n": L.n, "m": L.m, "N": L.N, "keep": L.keep, "sign": L.sign, "region": L.region,
            "sign2": L.sign2, "salient": L.salient, "scale": L.scale}


def _quantized(n, m, N, seed):
    W = si.dense_weight(n, m, seed).astype(np.float64)
    L, _, _ = oracle.quantize(W, si.calib_norms(m, seed), N)
    return L


def _salient_counts(d):
    return [bin(int(a) | (int(b) << 64)).count("1") for a, b in d["salient"]]


def _stream_bytes(d):
    """Bytes one pass streams: 26 + 6 N bytes per row and block plus one byte per four salient columns (rounded
    up) of that block, rows padded to tiles of 32."""
    rows = -(-d["n"] // 32) * 32
    return rows * sum(26 + 6 * d["N"] + -(-s // 4) for s in _salient_counts(d))


def _check_gemv(stb, layer, What, m, batch, seed, out_dtype=None):
    import torch
    x = si.activations(batch, m, seed)
    y_ref = oracle.matmul(What, x.astype(np.float64))
    xd = torch.from_numpy(x).cuda()
    y = stb.gemv(layer, xd, out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert int(layer.dev_status.item()) == 0
    err = np.abs(y.double().cpu().numpy() - y_ref).max()
    tol = TOL * np.abs(y_ref).max()
    assert err <= tol, (err, tol)
    if out_dtype is not None and out_dtype != torch.float32:
        # the 16-bit output is the fp32 sum of the same launch shape rounded to nearest even, bit for bit
        y32 = stb.gemv(layer, xd)
        torch.cuda.synchronize()
        assert torch.equal(y32.to(out_dtype), y)
    return err / np.abs(y_ref).max()


@pytest.mark.parametrize("N", [1, 2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("n,m", [(40, 256), (100, 384)])
def test_quantized_layer_dequant_bit_exact_and_gemv(stb, N, n, m):
    import torch
    L = _quantized(n, m, N, 1000 + 10 * N + n)
    What = oracle.decode(L)
    layer = stb.pack_numpy(_fields(L))
    info = layer.info()
    assert info["status"] == 0 and (info["n"], info["m"], info["N"]) == (n, m, N)
    assert int(layer.dev_status.item()) == 0
    got = stb.dequant(layer).cpu().numpy()
    assert np.array_equal(got, What)                       # bit-exact values (-0 == +0)
    for dt in (torch.float16, torch.bfloat16):
        g16 = stb.dequant(layer, dtype=dt).float().cpu().numpy()
        want = torch.from_numpy(What).to(dt).float().numpy()
        assert np.array_equal(g16, want)
    for batch in (1, 3, 4, 7, 16, 17, 33, 64):
        _check_gemv(stb, layer, What, m, batch, 7 + batch)
    _check_gemv(stb, layer, What, m, 2, 99, out_dtype=torch.float16)


def _sampled_rows(n, seed, count=192):
    g = np.random.default_rng(seed)
    rows = np.sort(g.choice(n, size=count, replace=False)).astype(np.int32)
    rows[:4] = [0, 1, n - 2, n - 1]
    return np.unique(rows)


def _check_layer_sampled(stb, d, batches, seed):
    """Sampled output rows of a full-size layer against the oracle's decode-and-multiply, and sampled rows
    of the dequantised matrix bit for bit."""
    import torch
    n, m, N = d["n"], d["m"], d["N"]
    L = wl.as_logical(d)
    layer = stb.pack_numpy(d)
    info = layer.info()
    assert info["status"] == 0
    assert info["stream_bytes"] == _stream_bytes(d) == wl.stream_bytes(d)
    rows = _sampled_rows(n, N)
    for batch in batches:
        x = si.activations(batch, m, seed + batch)
        y_ref = oracle.layer_rows(L, rows, x.astype(np.float64))
        y = stb.gemv(layer, torch.from_numpy(x).cuda())
        torch.cuda.synchronize()
        assert int(layer.dev_status.item()) == 0
        yg = y.double().cpu().numpy()[:, rows]
        assert np.abs(yg - y_ref).max() <= TOL * np.abs(y_ref).max(), batch
    Wg = stb.dequant(layer)
    sub = oracle.Logical(len(rows), m, N, d["keep"][rows].copy(), d["sign"][rows].copy(), d["region"][rows].copy(),
                         d["sign2"][rows].copy(), d["salient"], d["scale"][rows].copy())
    assert np.array_equal(Wg[torch.from_numpy(rows.astype(np.int64)).cuda()].cpu().numpy(), oracle.decode(sub))


@pytest.mark.parametrize("config,name", [(1, "q"), (2, "gate"), (2, "down"), (3, "q"), (3, "gate"), (3, "down")])
def test_full_size_quantized_layers_sampled_rows(stb, config, name):
    """The decode workloads' own layers: LLaMA-2 shapes, dense synthetic weights put through the oracle's
    quantizer (up to 32 salient columns in a block, a different count in every block)."""
    n, m, N, seed = si.workload_layer(config, name)
    d = wl.quantized_layer(n, m, N, seed)
    counts = wl.salient_counts(d)
    assert counts.min() >= 1 and counts.max() <= 32
    _check_layer_sampled(stb, d, (1, 4, 16, 64), si.seed_for(config, 8))


def test_full_size_layer_with_long_k_slices(stb):
    """9472 x 7168 at 6:8 is not a model shape: 296 row tiles leave all 56 blocks of a row tile to one CTA, a slice
    too long for the shared-memory copy of the activations, so it takes the kernel's other load path."""
    _check_layer_sampled(stb, si.logical_layer(9472, 7168, 6, si.seed_for(2, 6)), (1, 2, 8), si.seed_for(2, 8))


@pytest.mark.parametrize("N,max_salient", [(4, 7), (5, 14), (6, 30), (6, 32), (3, 20)])
def test_many_salient_columns(stb, N, max_salient):
    """Blocks with up to 8 / 16 / 32 salient columns use the wider residual fields."""
    import torch
    n, m = 70, 512
    d = si.logical_layer(n, m, N, 400 + max_salient, max_salient=max_salient)
    L = oracle.Logical(**d)
    What = oracle.decode(L)
    layer = stb.pack_numpy(d)
    assert layer.info()["status"] == 0
    assert layer.info()["stream_bytes"] == _stream_bytes(d)
    assert np.array_equal(stb.dequant(layer).cpu().numpy(), What)
    for batch in (1, 5, 8, 13):
        _check_gemv(stb, layer, What, m, batch, 30 + batch)


@pytest.mark.parametrize("N", [4, 5, 6])
def test_blocks_with_different_salient_counts_side_by_side(stb, N):
    """Blocks with 1, 5, 17, 32, 0 and 4 salient columns next to each other: every block stores its own number
    of residual words, and the bytes follow."""
    n, m = 100, 6 * 128 * 2
    d = si.logical_layer(n, m, N, 700 + N, salient_counts=[1, 5, 17, 32, 0, 4])
    L = oracle.Logical(**d)
    What = oracle.decode(L)
    layer = stb.pack_numpy(d)
    assert layer.info()["status"] == 0
    assert _salient_counts(d) == [1, 5, 17, 32, 0, 4] * 2
    assert layer.info()["stream_bytes"] == 128 * 2 * (6 * (26 + 6 * N) + 1 + 2 + 5 + 8 + 0 + 1)
    assert np.array_equal(stb.dequant(layer).cpu().numpy(), What)
    for batch in (1, 2, 8, 11, 40):
        _check_gemv(stb, layer, What, m, batch, 40 + batch)
    _check_gemm(stb, layer, L, 70, 12)


def test_a_wait_that_runs_out_is_reported_and_harmless(stb):
    """Failure detection: with the weight copies switched off every warp's bounded wait runs out; the kernel
    returns, the status word says STB_ERR_TIMEOUT, and the next ordinary call on the same layer is correct."""
    import torch
    for N in (4, 6):
        d = si.logical_layer(256, 1024, N, 800 + N)
        layer = stb.pack_numpy(d)
        What = oracle.decode(oracle.Logical(**d))
        x = torch.from_numpy(si.activations(1, 1024, 801)).cuda()
        y = torch.zeros(1, 256, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        stb.gemv_wait_selftest(layer, x, y, status)
        torch.cuda.synchronize()
        assert int(status.item()) == stb.STB_ERR_TIMEOUT
        assert int(layer.dev_status.item()) == 0
        _check_gemv(stb, layer, What, 1024, 1, 802)


def test_pack_flags_corrupt_layers(stb):
    import torch
    base = si.logical_layer(64, 256, 4, 5)
    def status_of(d):
        layer = stb.pack_numpy(d)
        torch.cuda.synchronize()
        return int(layer.dev_status.item()), layer.info()["status"]
    assert status_of(base) == (0, 0)
    d = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in base.items()}
    d["keep"][3, 5] = 0b00000111                      # three bits instead of four
    assert status_of(d) == (stb.STB_ERR_CORRUPT, stb.STB_ERR_CORRUPT)
    d = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in base.items()}
    d["sign"][0, 0] |= 0x10                           # sign bit beyond N
    assert status_of(d)[0] == stb.STB_ERR_CORRUPT
    d = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in base.items()}
    d["salient"][1, 0] = np.uint64(0xFFFFFFFFFF)      # 40 salient columns in one block
    assert status_of(d)[0] == stb.STB_ERR_CORRUPT
    d = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in base.items()}
    d["salient"][:] = 0                               # region 3 without a salient column
    assert status_of(d)[0] == stb.STB_ERR_CORRUPT
    # a layer packed for one shape must not be run as another: the kernel refuses and reports
    layer = stb.pack_numpy(base)
    wrong = stb.PackedLayer(64, 256, 5, layer.buf, layer.dev_status)
    y = torch.zeros(1, 64, device="cuda")
    stb.gemv(wrong, torch.zeros(1, 256, dtype=torch.float16, device="cuda"), out=y)
    torch.cuda.synchronize()
    assert int(layer.dev_status.item()) == stb.STB_ERR_CORRUPT


def test_degenerate_layers(stb):
    """No salient column at all, all weights kept (N = 8), a single tile with one row."""
    import torch
    d = si.logical_layer(1, 128, 8, 3, max_salient=0)
    L = oracle.Logical(**d)
    layer = stb.pack_numpy(d)
    assert np.array_equal(stb.dequant(layer).cpu().numpy(), oracle.decode(L))
    _check_gemv(stb, layer, oracle.decode(L), 128, 1, 4)
    d = si.logical_layer(33, 128, 3, 4, max_salient=0)
    L = oracle.Logical(**d)
    layer = stb.pack_numpy(d)
    assert layer.info()["stream_bytes"] == 2 * 32 * (16 + 6 + 12 + 10)
    assert np.array_equal(stb.dequant(layer).cpu().numpy(), oracle.decode(L))
    _check_gemv(stb, layer, oracle.decode(L), 128, 16, 5)


def test_layer_stack_chains_layers_with_per_layer_N(stb):
    import torch
    shapes = [(256, 384, 4), (128, 256, 6), (96, 128, 5)]          # (n, m, N): m of a layer = n of the previous
    layers, Ws = [], []
    for k, (n, m, N) in enumerate(shapes):
        d = si.logical_layer(n, m, N, 60 + k)
        layers.append(stb.pack_numpy(d)); Ws.append(oracle.decode(oracle.Logical(**d)))
    x0 = si.activations(2, 384, 61)
    bufs = [torch.from_numpy(x0).cuda(), torch.empty(2, 256, dtype=torch.float16, device="cuda"),
            torch.empty(2, 128, dtype=torch.float16, device="cuda"), torch.empty(2, 96, dtype=torch.float32, device="cuda")]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stb.layer_stack([(layers[k], bufs[k], bufs[k + 1]) for k in range(3)], dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # parity per layer: the oracle is fed the same (GPU-produced, fp16-rounded) input
    for k in range(3):
        xin = bufs[k].double().cpu().numpy()
        y_ref = oracle.matmul(Ws[k], xin)
        got = bufs[k + 1].double().cpu().numpy()
        assert np.abs(got - y_ref).max() <= TOL * np.abs(y_ref).max()


@pytest.mark.parametrize("batch", [1, 2, 5, 16])
def test_layer_stack_runs_same_input_layers_as_one_grid(stb, batch):
    """An MLP-shaped stack: gate and up read the same input (one fused launch, different row counts and
    output types), down reads gate's fp16 output; every layer is checked against the oracle fed the
    same input."""
    import torch
    m, n1, n2, N = 384, 200, 136, 6
    dg, du, dd = si.logical_layer(n1, m, N, 71), si.logical_layer(n2, m, N, 72), si.logical_layer(96, 256, N, 73)
    lg, lu, ld = (stb.pack_numpy(d) for d in (dg, du, dd))
    x = torch.from_numpy(si.activations(batch, m, 74)).cuda()
    hg = torch.zeros(batch, 256, dtype=torch.float16, device="cuda")        # wider than n1: ldout > n
    hu = torch.zeros(batch, n2, dtype=torch.float32, device="cuda")
    y = torch.zeros(batch, 96, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stb.layer_stack([(lg, x, hg), (lu, x, hu), (ld, hg, y)], dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    xin = x.double().cpu().numpy()
    for d, out, n in ((dg, hg, n1), (du, hu, n2)):
        ref = oracle.matmul(oracle.decode(oracle.Logical(**d)), xin)
        got = out.double().cpu().numpy()[:, :n]
        assert np.abs(got - ref).max() <= TOL * np.abs(ref).max()
    assert (hg.cpu().numpy()[:, n1:] == 0).all()                             # columns past n untouched
    ref = oracle.matmul(oracle.decode(oracle.Logical(**dd)), hg.double().cpu().numpy())
    assert np.abs(y.double().cpu().numpy() - ref).max() <= TOL * np.abs(ref).max()


def _check_gemm(stb, layer, L, T, seed, out_dtype=None, rows=None, toks=None):
    """stb_gemm against the float64 dequantise-then-matmul on bf16 activations."""
    import torch
    x = si.activations(T, L.m, seed, "bf16")                       # float32 values exactly representable in bf16
    xd = torch.from_numpy(x).cuda().to(torch.bfloat16)
    assert np.array_equal(xd.float().cpu().numpy(), x)
    y = stb.gemm(layer, xd, out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert int(layer.dev_status.item()) == 0
    if rows is None:
        y_ref = oracle.matmul(oracle.decode(L), x.astype(np.float64))
        got = y.double().cpu().numpy()
    else:
        y_ref = oracle.layer_rows(L, rows, x[toks].astype(np.float64))
        got = y.double().cpu().numpy()[np.ix_(toks, rows)]
    scale = np.abs(y_ref).max()
    err = np.abs(got - y_ref).max()
    assert err <= TOL * scale, (err, TOL * scale)
    if out_dtype is not None and out_dtype != torch.float32:
        # the bf16 output is the fp32 result of the same launch rounded to nearest even, bit for bit
        y32 = stb.gemm(layer, xd)
        torch.cuda.synchronize()
        assert torch.equal(y32.to(out_dtype), y)
    return err / scale


@pytest.mark.parametrize("N", [4, 5, 6])
@pytest.mark.parametrize("n,m,T", [(40, 256, 1), (100, 384, 37), (128, 128, 256), (300, 512, 300), (257, 1024, 513)])
def test_gemm_quantized_layers(stb, N, n, m, T):
    """Prefill GEMM on quantizer output: ragged rows (n not a multiple of 128), ragged tokens, several
    K stages, one and several output tiles."""
    import torch
    L = _quantized(n, m, N, 2000 + 10 * N + n)
    layer = stb.pack_numpy(_fields(L))
    _check_gemm(stb, layer, L, T, 50 + T)
    _check_gemm(stb, layer, L, T, 51 + T, out_dtype=torch.bfloat16)


@pytest.mark.parametrize("N,max_salient", [(4, 7), (6, 30)])
def test_gemm_many_salient_columns(stb, N, max_salient):
    d = si.logical_layer(200, 512, N, 500 + max_salient, max_salient=max_salient)
    L = oracle.Logical(**d)
    layer = stb.pack_numpy(d)
    _check_gemm(stb, layer, L, 70, 9)


def _check_gemm_f16(stb, layer, L, T, seed, out_dtype=None, rows=None):
    """stb_gemm_f16 against the float64 dequantise-then-matmul on fp16 activations."""
    import torch
    x = si.activations(T, L.m, seed)                                # fp16
    xd = torch.from_numpy(x).cuda()
    y = stb.gemm_f16(layer, xd, out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert int(layer.dev_status.item()) == 0
    if rows is None:
        y_ref = oracle.matmul(oracle.decode(L), x.astype(np.float64))
        got = y.double().cpu().numpy()
    else:
        y_ref = oracle.layer_rows(L, rows, x.astype(np.float64))
        got = y.double().cpu().numpy()[:, rows]
    scale = np.abs(y_ref).max()
    err = np.abs(got - y_ref).max()
    assert err <= TOL * scale, (err, TOL * scale)
    if out_dtype is not None and out_dtype != torch.float32:
        y32 = stb.gemm_f16(layer, xd)
        torch.cuda.synchronize()
        assert torch.equal(y32.to(out_dtype), y)                     # the fp16 output is the fp32 one rounded, bit for bit
    return y


@pytest.mark.parametrize("N", [4, 5, 6])
@pytest.mark.parametrize("n,m,T", [(40, 256, 1), (100, 384, 37), (300, 1024, 64), (257, 2048, 33), (200, 512, 65), (130, 640, 200)])
def test_gemm_f16_quantized_layers(stb, N, n, m, T):
    """The fp16 product on quantizer output: the 64-token tile (T <= 64: one to several row tiles, K split in parts,
    ragged rows and tokens) and the prefill tile beyond; fp32 and fp16 outputs."""
    import torch
    L = _quantized(n, m, N, 2100 + 10 * N + n)
    layer = stb.pack_numpy(_fields(L))
    y = _check_gemm_f16(stb, layer, L, T, 60 + T)
    _check_gemm_f16(stb, layer, L, T, 61 + T, out_dtype=torch.float16)
    if T <= 64:
        # the same operation as the decode GEMV: both within the tolerance of the oracle, hence of each other
        xd = torch.from_numpy(si.activations(T, m, 60 + T)).cuda()
        yv = stb.gemv(layer, xd)
        torch.cuda.synchronize()
        assert (y - yv).abs().max().item() <= 2 * TOL * yv.abs().max().item()


@pytest.mark.parametrize("max_salient", [0, 30])
def test_gemm_f16_salient_extremes(stb, max_salient):
    d = si.logical_layer(200, 1024, 6, 520 + max_salient, max_salient=max_salient)
    L = oracle.Logical(**d)
    layer = stb.pack_numpy(d)
    _check_gemm_f16(stb, layer, L, 48, 19)


@pytest.mark.parametrize("name", ["gate", "down"])
def test_gemm_f16_full_size_decode_batch(stb, name):
    """A decode batch of 64 on the LLaMA-2-7B MLP layers at 6:8 from the oracle's quantizer, sampled rows."""
    n, m, N, seed = si.workload_layer(2, name)
    d = wl.quantized_layer(n, m, N, seed)
    L = wl.as_logical(d)
    layer = stb.pack_numpy(d)
    g = np.random.default_rng(n + 3 * m)
    rows = np.unique(np.concatenate([[0, 1, 127, 128, n - 129, n - 1], g.choice(n, 64, replace=False)])).astype(np.int32)
    _check_gemm_f16(stb, layer, L, 64, si.seed_for(2, 12), rows=rows)
    with pytest.raises(stb.StbError) as e:                      # no workspace: refused on the host
        import torch
        x = torch.zeros(64, m, dtype=torch.float16, device="cuda")
        stb._check(stb._lib.stb_gemm_f16(stb._ptr(layer.buf), n, m, N, stb._ptr(x), 64, m, stb._ptr(torch.empty(64, n, device="cuda")),
                                         stb.STB_F32, n, None, 0, stb._ptr(layer.dev_status), stb._stream()), "stb_gemm_f16")
    assert e.value.status == stb.STB_ERR_SIZE


@pytest.mark.parametrize("n,ldy,shift", [(100, 104, 0), (200, 208, 0), (136, 136, 8), (136, 144, 2)])
def test_gemm_16_bit_output_layouts(stb, n, ldy, shift):
    """16-bit outputs leave through shared memory in 16-byte pieces when the output allows it (row stride a multiple of
    8, base 16-byte aligned) and element by element otherwise; a last piece of rows that crosses n is cut.  Every
    layout must give the fp32 result rounded, and must not touch what lies beside the output."""
    import torch
    m, N = 512, 5
    L = _quantized(n, m, N, 2300 + n)
    layer = stb.pack_numpy(_fields(L))
    for dt, act, T in ((torch.bfloat16, "bf16", 70), (torch.float16, None, 70), (torch.float16, None, 40)):
        x = si.activations(T, m, 77, act) if act else si.activations(T, m, 77)
        xd = torch.from_numpy(x).cuda().to(dt)
        fn = stb.gemm if act else stb.gemm_f16
        y32 = fn(layer, xd)
        buf = torch.full((T * ldy + 16,), 7.0, dtype=dt, device="cuda")
        out = buf[shift:shift + T * ldy].view(T, ldy)[:, :n]
        fn(layer, xd, out=out)
        torch.cuda.synchronize()
        assert int(layer.dev_status.item()) == 0
        assert torch.equal(out, y32.to(dt))
        mask = torch.ones(T * ldy + 16, dtype=torch.bool, device="cuda")
        mask[shift:shift + T * ldy].view(T, ldy)[:, :n] = False
        assert bool((buf[mask] == 7.0).all()), "wrote outside the output"
        ref = oracle.matmul(oracle.decode(L), x.astype(np.float64))
        assert np.abs(y32.double().cpu().numpy() - ref).max() <= TOL * np.abs(ref).max()


def test_gemm_split_k_uses_the_workspace(stb):
    """Few output tiles and a long K: the launch splits K, partial sums go through the caller's workspace."""
    import torch
    n, m, N, T = 128, 4096, 4, 200
    d = si.logical_layer(n, m, N, 610)
    L = oracle.Logical(**d)
    layer = stb.pack_numpy(d)
    assert stb.gemm_workspace(n, m, N, T) >= 2 * T * n * 4
    _check_gemm(stb, layer, L, T, 11)
    x = torch.zeros(T, m, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(stb.StbError) as e:                      # workspace too small: refused on the host
        stb._check(stb._lib.stb_gemm(stb._ptr(layer.buf), n, m, N, stb._ptr(x), T, m, stb._ptr(torch.empty(T, n, device="cuda")),
                                     stb.STB_F32, n, None, 0, stb._ptr(layer.dev_status), stb._stream()), "stb_gemm")
    assert e.value.status == stb.STB_ERR_SIZE


def test_gemm_splits_the_tiles_of_a_small_last_wave(stb):
    """150 output tiles on 148 SMs: the two tiles of the last wave are split along K when the caller gives the
    workspace stb_gemm_workspace asks for, and run unsplit without it; both must match the oracle (sampled
    rows, among them rows of the last two tiles) and each other."""
    import torch
    n, m, N, T = 150 * 128 - 5, 1024, 5, 100
    d = si.logical_layer(n, m, N, 612)
    L = oracle.Logical(**d)
    layer = stb.pack_numpy(d)
    need, least = stb.gemm_workspace(n, m, N, T), stb.gemm_workspace(n, m, N, T, minimum=True)
    assert need - least == 2 * 2 * 128 * 512 * 4               # two tiles, two parts each, fp32 partial tiles
    assert least == (T * (m // 4) * 2 + 255) // 256 * 256      # the gathered activations of the residual slots
    g = np.random.default_rng(5)
    rows = np.unique(np.concatenate([[0, 148 * 128 - 1, 148 * 128, 149 * 128 + 7, n - 1], g.choice(n, 64, replace=False)])).astype(np.int32)
    toks = np.arange(T)
    _check_gemm(stb, layer, L, T, 31, rows=rows, toks=toks)
    x = torch.from_numpy(si.activations(T, m, 31, "bf16")).cuda().to(torch.bfloat16)
    y_split = stb.gemm(layer, x)
    y_whole = torch.empty(T, n, device="cuda")
    ws_least = torch.empty(least, dtype=torch.uint8, device="cuda")
    stb._check(stb._lib.stb_gemm(stb._ptr(layer.buf), n, m, N, stb._ptr(x), T, m, stb._ptr(y_whole), stb.STB_F32, n,
                                 stb._ptr(ws_least), least, stb._ptr(layer.dev_status), stb._stream()), "stb_gemm")
    torch.cuda.synchronize()
    assert int(layer.dev_status.item()) == 0
    a, b = y_split.double().cpu().numpy(), y_whole.double().cpu().numpy()
    assert np.abs(a - b).max() <= 1e-4 * np.abs(b).max()       # the same bf16 products, another fp32 summation order


@pytest.mark.parametrize("name", ["q", "k", "gate", "down"])
def test_gemm_full_size_quantized_sampled(stb, name):
    """LLaMA-2-70B prefill shapes at 4:8, 2048 tokens, layers from the oracle's quantizer: sampled (token, row)
    pairs against the oracle.  gate (28672 x 8192: 896 output tiles, the last wave's eight are split along K)
    and down (8192 x 28672: K = 224 blocks) are the two shapes with the most work."""
    import torch
    n, m, N, seed = si.workload_layer(4, name)
    T = 2048
    d = wl.quantized_layer(n, m, N, seed)
    L = wl.as_logical(d)
    layer = stb.pack_numpy(d)
    assert layer.info()["status"] == 0 and layer.info()["stream_bytes"] == wl.stream_bytes(d)
    g = np.random.default_rng(n + m)
    rows = np.unique(np.concatenate([[0, 1, n - 129, n - 1], g.choice(n, 96, replace=False)])).astype(np.int32)
    toks = np.unique(np.concatenate([[0, 255, 256, 511, 512, T - 1], g.choice(T, 40, replace=False)]))
    _check_gemm(stb, layer, L, T, si.seed_for(4, 9), rows=rows, toks=toks)
    if name == "k":
        _check_gemm(stb, layer, L, T, si.seed_for(4, 10), out_dtype=torch.bfloat16, rows=rows, toks=toks)


def _run_stack_in_graph(stb, torch, steps, status, outs):
    stb.layer_stack(None, dev_status=status, marshalled=steps)            # warm (module load) outside capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        stb.layer_stack(None, dev_status=status, marshalled=steps)
    for t in outs:
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert int(status.item()) == 0


@pytest.mark.parametrize("batch", [1, 8])
def test_decoder_layer_stack_full_size_per_layer_N(stb, batch):
    """The seven linears of a LLaMA-2-7B decoder layer as one stb_layer_stack call in the launch
    configuration bench.py times (q/k/v and gate/up fused, programmatic dependent launches, CUDA
    graph), quantizer-made layers with N drawn per group of linears from {4, 5, 6}; every layer is checked
    on sampled rows against the oracle fed the same GPU-produced input."""
    import torch
    h, f = 4096, 11008
    Nq, No, Nm, Nd = (int(v) for v in np.random.default_rng(si.seed_for(5, 1)).choice([4, 5, 6], size=4))
    g = np.random.default_rng(si.seed_for(5, batch))
    spec = [("q", Nq), ("k", Nq), ("v", Nq), ("o", No), ("gate", Nm), ("up", Nm), ("down", Nd)]
    ds = []
    for i, (name, N) in enumerate(spec):
        n, m, _, seed = si.workload_layer(5, name, N)
        ds.append(wl.quantized_layer(n, m, N, seed + 64 * i))           # seven different layers
    layers = [stb.pack_numpy(d) for d in ds]
    x = torch.from_numpy(si.activations(batch, h, si.seed_for(5, 9))).cuda()
    q, k, v = (torch.empty(batch, h, dtype=torch.float16, device="cuda") for _ in range(3))
    o = torch.empty(batch, h, dtype=torch.float16, device="cuda")
    gate, up = (torch.empty(batch, f, dtype=torch.float16, device="cuda") for _ in range(2))
    y = torch.empty(batch, h, dtype=torch.float32, device="cuda")
    io = [(x, q), (x, k), (x, v), (q, o), (o, gate), (o, up), (gate, y)]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    steps = stb.make_steps([(layers[i], io[i][0], io[i][1]) for i in range(7)])
    _run_stack_in_graph(stb, torch, steps, status, (q, k, v, o, gate, up, y))
    for i, (name, N) in enumerate(spec):
        n = ds[i]["n"]
        rows = np.unique(np.concatenate([[0, n - 1], g.choice(n, 48, replace=False)])).astype(np.int32)
        xin = io[i][0].double().cpu().numpy()
        ref = oracle.layer_rows(wl.as_logical(ds[i]), rows, xin)
        got = io[i][1].double().cpu().numpy()[:, rows]
        assert np.abs(got - ref).max() <= TOL * np.abs(ref).max(), (name, N)


def test_13b_decoder_block_chained(stb):
    """The seven linears of a LLaMA-2-13B decoder block at 5:8 (quantizer-made), batch 1, chained on one stream in
    dependency order: q, k, v read x; o reads q's output; gate and up read o's; down reads gate's.  Every layer
    is checked on sampled rows against the oracle fed the same GPU-produced input."""
    import torch
    h, f = 5120, 13824
    names = ["q", "k", "v", "o", "gate", "up", "down"]
    ds = [wl.quantized_layer(*si.workload_layer(3, nm)) for nm in names]
    layers = [stb.pack_numpy(d) for d in ds]
    x = torch.from_numpy(si.activations(1, h, si.seed_for(3, 8))).cuda()
    q, k, v, o = (torch.empty(1, h, dtype=torch.float16, device="cuda") for _ in range(4))
    gate, up = (torch.empty(1, f, dtype=torch.float16, device="cuda") for _ in range(2))
    y = torch.empty(1, h, dtype=torch.float32, device="cuda")
    io = [(x, q), (x, k), (x, v), (q, o), (o, gate), (o, up), (gate, y)]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    steps = stb.make_steps([(layers[i], io[i][0], io[i][1]) for i in range(7)])
    _run_stack_in_graph(stb, torch, steps, status, (q, k, v, o, gate, up, y))
    g = np.random.default_rng(13)
    for i, name in enumerate(names):
        n = ds[i]["n"]
        rows = np.unique(np.concatenate([[0, n - 1], g.choice(n, 48, replace=False)])).astype(np.int32)
        ref = oracle.layer_rows(wl.as_logical(ds[i]), rows, io[i][0].double().cpu().numpy())
        got = io[i][1].double().cpu().numpy()[:, rows]
        assert np.abs(got - ref).max() <= TOL * np.abs(ref).max(), name


def test_layerwise_nm_assignment_from_dense_weights(stb):
    """Section 3.3: N per layer from the L2 norms of the dense weights, the norms summed on the GPU."""
    import torch
    shapes = [(256, 384), (100, 128), (512, 1024), (64, 136)]
    Ws = [si.dense_weight(n, m, 1200 + k) * np.float16(1 + 3 * k) for k, (n, m) in enumerate(shapes)]
    norms = [np.sqrt((W.astype(np.float64) ** 2).sum()) for W in Ws]
    for R in (0.5, 0.75):
        got, sums = stb.allocate_nm([torch.from_numpy(W).cuda() for W in Ws], R)
        assert np.allclose(np.sqrt(sums), norms, rtol=1e-13, atol=0)
        want, _ = oracle.allocate_nm(norms, R)
        assert got == [int(v) for v in want]


def _gpu_quantize(stb, torch, n, m, N, seed):
    W = si.dense_weight(n, m, seed)
    xn = si.calib_norms(m, seed)
    return stb.quantize(torch.from_numpy(W).cuda(), torch.from_numpy(xn).cuda(), N), W, xn


def _same_logical(got, L):
    views = {"keep": np.uint8, "sign": np.uint8, "region": np.uint16, "sign2": np.uint32, "salient": np.uint64, "scale": np.uint16}
    for k, v in views.items():
        g = got[k].cpu().numpy().view(v)
        assert np.array_equal(g, getattr(L, k)), k


@pytest.mark.parametrize("N", [1, 3, 4, 5, 6, 8])
@pytest.mark.parametrize("n,m", [(40, 256), (300, 384)])
def test_gpu_quantizer_matches_the_oracle_bit_for_bit(stb, N, n, m):
    """stb_quantize against the oracle's quantizer on the same dense weights and calibration norms: keep masks, signs,
    region codes, residual signs, salient masks and fp16 scales, all equal."""
    import torch
    got, W, xn = _gpu_quantize(stb, torch, n, m, N, 3000 + 10 * N + n)
    L, _, _ = oracle.quantize(W.astype(np.float64), xn, N)
    _same_logical(got, L)
    layer = stb.pack(n, m, N, got["keep"], got["sign"], got["region"], got["sign2"], got["salient"], got["scale"])
    torch.cuda.synchronize()
    assert int(layer.dev_status.item()) == 0
    assert np.array_equal(stb.dequant(layer).cpu().numpy(), oracle.decode(L))


def test_gpu_quantizer_full_size_layer(stb):
    """The 7B down projection (4096 x 11008 at 6:8): the GPU quantizer's logical arrays equal the oracle's."""
    import torch
    n, m, N, seed = si.workload_layer(2, "down")
    got, W, xn = _gpu_quantize(stb, torch, n, m, N, seed)
    torch.cuda.synchronize()
    _same_logical(got, wl.as_logical(wl.quantized_layer(n, m, N, seed)))
