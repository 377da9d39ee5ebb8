"""GPU parity of stb_layer_stack_resident (a whole list of decode steps as one resident kernel) against the CPU
oracle: every layer of a stack is checked against the oracle fed the same, GPU-produced, input."""
import numpy as np
import pytest

import oracle
import oracle.workloads as wl
import stb_inputs as si

pytestmark = pytest.mark.gpu
TOL = 5e-3


@pytest.fixture(scope="module")
def stb():
    import torch
    assert torch.cuda.is_available()
    from paper_2408_01803_b200 import build
    build.build()
    import paper_2408_01803_b200 as stb
    return stb


def _run(stb, torch, triples, graph=False):
    """Runs the triples (layer, x, out) through the resident kernel; returns (status word, workspace)."""
    steps = stb.make_steps(triples)
    ws = stb.resident_workspace(steps)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    if graph:
        stb.layer_stack_resident(None, ws, dev_status=status, marshalled=steps)      # warm outside capture
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            stb.layer_stack_resident(None, ws, dev_status=status, marshalled=steps)
        for _, _, out in triples:
            out.zero_()
        g.replay()
    else:
        stb.layer_stack_resident(None, ws, dev_status=status, marshalled=steps)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert int(ws[:16].view(torch.int32).abs().max().item()) == 0, "the counters at the head of the workspace are not zero after the call"
    return status, ws


def _check_layers(triples, logicals, rows_of=None):
    for k, ((_, x, out), L) in enumerate(zip(triples, logicals)):
        xin = x.double().cpu().numpy()
        got = out.double().cpu().numpy()[:, :L.n]
        if rows_of is None:
            ref = oracle.matmul(oracle.decode(L), xin)
        else:
            rows = rows_of(L.n, k)
            ref = oracle.layer_rows(L, rows, xin)
            got = got[:, rows]
        assert np.abs(got - ref).max() <= TOL * np.abs(ref).max(), k


@pytest.mark.parametrize("batch", [1, 2, 5, 8])
def test_chain_with_per_layer_N(stb, batch):
    """Three chained layers with N = 4, 6, 5 (ragged row counts), then an MLP-shaped tail: gate and up read the same
    input (one phase), down reads gate's fp16 output."""
    import torch
    shapes = [(260, 384, 4), (128, 256 + 128, 6), (100, 128, 5)]      # (n, m, N); m of a layer <= ld of the previous output
    ds = [si.logical_layer(n, m, N, 60 + k, max_salient=9) for k, (n, m, N) in enumerate(shapes)]
    dg = si.logical_layer(200, 384, 6, 71, salient_counts=[1, 17, 32])
    du = si.logical_layer(136, 384, 6, 72, salient_counts=[0, 5, 2])
    dd = si.logical_layer(96, 256, 6, 73)
    layers = [stb.pack_numpy(d) for d in ds + [dg, du, dd]]
    x0 = torch.from_numpy(si.activations(batch, 384, 61)).cuda()
    h1 = torch.zeros(batch, 384, dtype=torch.float16, device="cuda")       # 260 outputs used as 384 inputs: the tail stays 0
    h2 = torch.zeros(batch, 128, dtype=torch.float16, device="cuda")
    y3 = torch.zeros(batch, 100, dtype=torch.float32, device="cuda")
    hg = torch.zeros(batch, 256, dtype=torch.float16, device="cuda")
    hu = torch.zeros(batch, 136, dtype=torch.float32, device="cuda")
    y = torch.zeros(batch, 96, dtype=torch.float32, device="cuda")
    triples = [(layers[0], x0, h1), (layers[1], h1, h2), (layers[2], h2, y3),
               (layers[3], x0, hg), (layers[4], x0, hu), (layers[5], hg, y)]
    _run(stb, torch, triples)
    _check_layers(triples, [oracle.Logical(**d) for d in ds + [dg, du, dd]])
    assert (hg.cpu().numpy()[:, 200:] == 0).all()                            # columns past n untouched


def test_results_are_reproducible_and_close_to_the_per_layer_launches(stb):
    import torch
    d1, d2 = si.logical_layer(700, 1024, 6, 81, max_salient=12), si.logical_layer(300, 768, 4, 82, max_salient=12)
    l1, l2 = stb.pack_numpy(d1), stb.pack_numpy(d2)
    x = torch.from_numpy(si.activations(2, 1024, 83)).cuda()
    outs = []
    for _ in range(2):
        h = torch.zeros(2, 768, dtype=torch.float16, device="cuda")
        y = torch.zeros(2, 300, dtype=torch.float32, device="cuda")
        _run(stb, torch, [(l1, x, h), (l2, h, y)])
        outs.append((h.clone(), y.clone()))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    h = torch.zeros(2, 768, dtype=torch.float16, device="cuda")
    y = torch.zeros(2, 300, dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    stb.layer_stack([(l1, x, h), (l2, h, y)], dev_status=st)
    torch.cuda.synchronize()
    a, b = outs[0][1].double().cpu().numpy(), y.double().cpu().numpy()
    assert np.abs(a - b).max() <= 2e-3 * np.abs(b).max()


def test_more_groups_than_one_launch_holds(stb):
    """70 small steps that alternate between two inputs (no two neighbours can share a group): more than the 64
    groups one launch takes, so the list runs as two launches."""
    import torch
    n = 128
    ds = [si.logical_layer(n, n, 4 + k % 3, 900 + k, max_salient=2) for k in range(4)]
    layers = [stb.pack_numpy(d) for d in ds]
    Ls = [oracle.Logical(**d) for d in ds]
    xs = [torch.from_numpy(si.activations(1, n, 98 + i)).cuda() for i in range(2)]
    outs = [torch.zeros(1, n, dtype=torch.float32, device="cuda") for _ in range(70)]
    triples = [(layers[k % 4], xs[k % 2], outs[k]) for k in range(70)]
    _run(stb, torch, triples)
    _check_layers(triples, [Ls[k % 4] for k in range(70)])


def test_a_wait_that_runs_out_is_reported_and_the_workspace_is_zero_again(stb):
    import torch
    d1, d2 = si.logical_layer(512, 1024, 6, 91), si.logical_layer(256, 512, 5, 92)
    l1, l2 = stb.pack_numpy(d1), stb.pack_numpy(d2)
    x = torch.from_numpy(si.activations(1, 1024, 93)).cuda()
    h = torch.zeros(1, 512, dtype=torch.float16, device="cuda")
    y = torch.zeros(1, 256, dtype=torch.float32, device="cuda")
    triples = [(l1, x, h), (l2, h, y)]
    steps = stb.make_steps(triples)
    ws = stb.resident_workspace(steps)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stb.layer_stack_resident(None, ws, dev_status=status, marshalled=steps, selftest=True)
    torch.cuda.synchronize()
    assert int(status.item()) == stb.STB_ERR_TIMEOUT
    assert int(ws[:16].view(torch.int32).abs().max().item()) == 0
    status.zero_()
    stb.layer_stack_resident(None, ws, dev_status=status, marshalled=steps)       # the same workspace, an ordinary call
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    _check_layers(triples, [oracle.Logical(**d1), oracle.Logical(**d2)])


def test_unsupported_steps_are_refused_on_the_host(stb):
    import torch
    d = si.logical_layer(64, 128, 3, 95)
    lay = stb.pack_numpy(d)
    x = torch.zeros(1, 128, dtype=torch.float16, device="cuda")
    y = torch.zeros(1, 64, device="cuda")
    steps = stb.make_steps([(lay, x, y)])
    out = stb.C.c_size_t()
    assert stb._lib.stb_layer_stack_resident_workspace(steps, 1, stb.C.byref(out)) == stb.STB_ERR_UNSUPPORTED      # N = 3
    d4 = si.logical_layer(64, 128, 4, 96)
    lay4 = stb.pack_numpy(d4)
    x9 = torch.zeros(9, 128, dtype=torch.float16, device="cuda")
    y9 = torch.zeros(9, 64, device="cuda")
    steps = stb.make_steps([(lay4, x9, y9)])
    assert stb._lib.stb_layer_stack_resident_workspace(steps, 1, stb.C.byref(out)) == stb.STB_ERR_UNSUPPORTED      # batch 9
    steps = stb.make_steps([(lay4, x, y)])
    ws = stb.resident_workspace(steps)
    assert stb._lib.stb_layer_stack_resident(steps, 1, stb._ptr(ws), 16, None, stb._stream()) == stb.STB_ERR_SIZE


def _check_gated_mlp(stb, torch, dg, du, dd, batch, graph=False, rows_of=None):
    """gate and up read x, down reads fp16(silu(gate) * up) formed while it stages its input (STB_IN_SILU_MUL): gate and
    up against the oracle as usual, down against the oracle fed the oracle's own float64 evaluation of the gated
    activation of the GPU's gate and up outputs."""
    m, f = dg["m"], dg["n"]
    lg, lu, ld = (stb.pack_numpy(d) for d in (dg, du, dd))
    x = torch.from_numpy(si.activations(batch, m, 74)).cuda()
    hg = torch.zeros(batch, f, dtype=torch.float16, device="cuda")
    hu = torch.zeros(batch, f, dtype=torch.float16, device="cuda")
    y = torch.zeros(batch, dd["n"], dtype=torch.float32, device="cuda")
    triples = [(lg, x, hg), (lu, x, hu), (ld, (hg, hu), y)]
    _run(stb, torch, triples, graph=graph)
    as_l = wl.as_logical
    _check_layers(triples[:2], [as_l(dg), as_l(du)], rows_of=rows_of)
    act = oracle.silu_mul(hg.double().cpu().numpy(), hu.double().cpu().numpy())
    got = y.double().cpu().numpy()
    if rows_of is None:
        ref = oracle.matmul(oracle.decode(as_l(dd)), act)
    else:
        rows = rows_of(dd["n"], 2)
        ref = oracle.layer_rows(as_l(dd), rows, act)
        got = got[:, rows]
    assert np.abs(got - ref).max() <= TOL * np.abs(ref).max()


@pytest.mark.parametrize("N,batch", [(6, 1), (6, 2), (6, 3), (4, 1), (5, 8)])
def test_gated_activation_is_formed_while_down_stages_its_input(stb, N, batch):
    import torch
    dg = si.logical_layer(384, 256, N, 171, max_salient=9)
    du = si.logical_layer(384, 256, N, 172, max_salient=9)
    dd = si.logical_layer(200, 384, N, 173, salient_counts=[3, 17, 0])
    _check_gated_mlp(stb, torch, dg, du, dd, batch)


def test_gated_mlp_full_size(stb):
    """The LLaMA-2-7B MLP at 6:8 (quantizer-made) with the gated activation, in a CUDA graph as bench.py runs it."""
    import torch
    dg, du, dd = (wl.quantized_layer(*si.workload_layer(2, nm)) for nm in ("gate", "up", "down"))
    _check_gated_mlp(stb, torch, dg, du, dd, 1, graph=True, rows_of=_rows_of)


def test_per_layer_launches_refuse_formed_inputs(stb):
    import torch
    d = si.logical_layer(64, 128, 4, 97)
    lay = stb.pack_numpy(d)
    a = torch.zeros(1, 128, dtype=torch.float16, device="cuda")
    y = torch.zeros(1, 64, device="cuda")
    steps = stb.make_steps([(lay, (a, a), y)])
    assert stb._lib.stb_layer_stack(steps, 1, None, stb._stream()) == stb.STB_ERR_UNSUPPORTED


def test_checksum_of_the_streamed_bytes(stb):
    """stb_layer_stack_checksum = XOR of the 32-bit words of [tiles offset, used_bytes) of every step's packed buffer;
    a flipped bit in a tile or in a residual record changes it."""
    import torch
    ds = [si.logical_layer(200, 1024, 6, 301, salient_counts=[1, 9, 32, 0]), si.logical_layer(130, 1024, 6, 302, max_salient=5),
          si.logical_layer(96, 256, 4, 303), si.logical_layer(4096, 1024, 5, 304, max_salient=20)]
    layers = [stb.pack_numpy(d) for d in ds]
    x = torch.zeros(1, 1024, dtype=torch.float16, device="cuda")
    x2 = torch.zeros(1, 256, dtype=torch.float16, device="cuda")
    outs = [torch.zeros(1, d["n"], device="cuda") for d in ds]
    steps = stb.make_steps([(layers[0], x, outs[0]), (layers[1], x, outs[1]), (layers[2], x2, outs[2]), (layers[3], x, outs[3])])

    def expected(lay):
        info = lay.info()
        nblk = lay.m // 128
        t0 = (64 + 128 * nblk + 255) // 256 * 256
        words = lay.buf[t0:info["used_bytes"]].cpu().numpy().view(np.uint32)
        return int(np.bitwise_xor.reduce(words))

    sums = stb.layer_stack_checksum(steps)
    torch.cuda.synchronize()
    got = [int(v) & 0xFFFFFFFFFFFFFFFF for v in sums.cpu().numpy()]
    assert got == [expected(l) for l in layers]
    # one flipped bit in the last byte a pass streams (a residual record), one in the first tile
    for lay, off in ((layers[0], layers[0].info()["used_bytes"] - 1), (layers[3], (64 + 128 * 8 + 255) // 256 * 256 + 5)):
        before = expected(lay)
        lay.buf[off] ^= 0x10
        after = stb.layer_stack_checksum(steps)
        torch.cuda.synchronize()
        k = layers.index(lay)
        assert (int(after[k].item()) & 0xFFFFFFFFFFFFFFFF) == expected(lay) != before
        lay.buf[off] ^= 0x10


def _rows_of(n, k):
    g = np.random.default_rng(1000 + k)
    return np.unique(np.concatenate([[0, 31, 32, n - 1], g.choice(n, 60, replace=False)])).astype(np.int32)


@pytest.mark.parametrize("batch", [1, 8])
def test_7b_decoder_layer_full_size_in_a_graph(stb, batch):
    """The seven linears of a LLaMA-2-7B decoder layer (quantizer-made, N per group of linears from {4, 5, 6}) through
    the resident kernel, captured in a CUDA graph as bench.py runs it."""
    import torch
    h, f = 4096, 11008
    Nq, No, Nm, Nd = (int(v) for v in np.random.default_rng(si.seed_for(5, 1)).choice([4, 5, 6], size=4))
    spec = [("q", Nq), ("k", Nq), ("v", Nq), ("o", No), ("gate", Nm), ("up", Nm), ("down", Nd)]
    ds = []
    for i, (name, N) in enumerate(spec):
        n, m, _, seed = si.workload_layer(5, name, N)
        ds.append(wl.quantized_layer(n, m, N, seed + 64 * i))
    layers = [stb.pack_numpy(d) for d in ds]
    x = torch.from_numpy(si.activations(batch, h, si.seed_for(5, 9))).cuda()
    q, k, v, o = (torch.zeros(batch, h, dtype=torch.float16, device="cuda") for _ in range(4))
    gate, up = (torch.zeros(batch, f, dtype=torch.float16, device="cuda") for _ in range(2))
    y = torch.zeros(batch, h, dtype=torch.float32, device="cuda")
    io = [(x, q), (x, k), (x, v), (q, o), (o, gate), (o, up), (gate, y)]
    triples = [(layers[i], io[i][0], io[i][1]) for i in range(7)]
    _run(stb, torch, triples, graph=True)
    _check_layers(triples, [wl.as_logical(d) for d in ds], rows_of=_rows_of)


def test_mlp_6of8_and_13b_block_full_size(stb):
    """The benchmark's MLP pass (6:8, gate and up as one phase, down on gate's output) and the 13B decoder block at 5:8,
    quantizer-made layers, batch 1."""
    import torch
    ds = [wl.quantized_layer(*si.workload_layer(2, nm)) for nm in ("gate", "up", "down")]
    layers = [stb.pack_numpy(d) for d in ds]
    x = torch.from_numpy(si.activations(1, 4096, si.seed_for(2, 8))).cuda()
    hg, hu = (torch.zeros(1, 11008, dtype=torch.float16, device="cuda") for _ in range(2))
    y = torch.zeros(1, 4096, dtype=torch.float32, device="cuda")
    triples = [(layers[0], x, hg), (layers[1], x, hu), (layers[2], hg, y)]
    _run(stb, torch, triples, graph=True)
    _check_layers(triples, [wl.as_logical(d) for d in ds], rows_of=_rows_of)
    h, f = 5120, 13824
    names = ["q", "k", "v", "o", "gate", "up", "down"]
    ds = [wl.quantized_layer(*si.workload_layer(3, nm)) for nm in names]
    layers = [stb.pack_numpy(d) for d in ds]
    x = torch.from_numpy(si.activations(1, h, si.seed_for(3, 8))).cuda()
    q, k, v, o = (torch.zeros(1, h, dtype=torch.float16, device="cuda") for _ in range(4))
    gate, up = (torch.zeros(1, f, dtype=torch.float16, device="cuda") for _ in range(2))
    y = torch.zeros(1, h, dtype=torch.float32, device="cuda")
    io = [(x, q), (x, k), (x, v), (q, o), (o, gate), (o, up), (gate, y)]
    triples = [(layers[i], io[i][0], io[i][1]) for i in range(7)]
    _run(stb, torch, triples)
    _check_layers(triples, [wl.as_logical(d) for d in ds], rows_of=_rows_of)
