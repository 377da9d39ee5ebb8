"""stb_gemm_noalloc, the entry point for hosts that may not allocate device memory while they run
(a serving process whose memory budget went to one arena at start-up; a latency-critical loop where
a device-synchronising cudaMalloc is not allowed).  It must give what stb_gemm gives with a
caller-owned workspace: checked here on two calls in a row, the second with other activations, so
that nothing depends on what an earlier call left in the built-in scratch array.  Collected last on
purpose: a run that stops at the first failure has then already run every other test."""
import numpy as np
import pytest

import oracle
import stb_inputs as si

pytestmark = pytest.mark.gpu
TOL = 5e-3


def test_noalloc_gemm_matches_gemm_with_workspace_twice():
    import torch
    from paper_2408_01803_b200 import build
    build.build()
    import paper_2408_01803_b200 as stb
    n, m, N, T = 128, 4096, 4, 200                       # one output tile, long K: the launch splits K
    d = si.logical_layer(n, m, N, 910)
    layer = stb.pack_numpy(d)
    What = oracle.decode(oracle.Logical(**d))
    need = stb.gemm_workspace(n, m, N, T)
    assert 0 < need <= 8 << 20
    # every buffer of both calls exists before the first one, so that the free device memory can be compared
    xs = [si.activations(T, m, seed, "bf16") for seed in (21, 22)]
    xd = [torch.from_numpy(x).cuda().to(torch.bfloat16) for x in xs]
    wants = [stb.gemm(layer, x) for x in xd]                             # existing entry point, torch-owned workspace
    gots = [torch.full((T, n), float("nan"), dtype=torch.float32, device="cuda") for _ in xd]
    torch.cuda.synchronize()
    free = []
    for call in range(2):
        stb.gemm_noalloc(layer, xd[call], gots[call])
        torch.cuda.synchronize()
        free.append(torch.cuda.mem_get_info()[0])
        assert int(layer.dev_status.item()) == 0
    assert free[0] == free[1], "the second call changed the free device memory"
    for call in range(2):
        w, g = wants[call], gots[call]
        assert torch.isfinite(g).all(), "call %d left outputs unwritten" % call
        assert torch.equal(g, w), "same split, same order of the partial sums: the two entry points agree bit for bit"
        ref = oracle.matmul(What, xs[call].astype(np.float64))
        assert np.abs(g.double().cpu().numpy() - ref).max() <= TOL * np.abs(ref).max()
    # bf16 output, 6:8, a ragged number of rows (the second row tile has 72 of its 128) and of tokens
    x = torch.from_numpy(si.activations(300, m, 23, "bf16")).cuda().to(torch.bfloat16)
    layer2 = stb.pack_numpy(si.logical_layer(200, m, 6, 911))
    assert stb.gemm_workspace(200, m, 6, 300, minimum=True) <= 8 << 20
    want = stb.gemm(layer2, x, out_dtype=torch.bfloat16)
    got = torch.empty(300, 200, dtype=torch.bfloat16, device="cuda")
    stb.gemm_noalloc(layer2, x, got)
    torch.cuda.synchronize()
    assert torch.equal(got, want)
    # a shape whose partial sums do not fit the built-in array is refused on the host
    big = stb.PackedLayer(1024, 8192, 4, layer.buf, layer.dev_status)      # never launched: the size check comes first
    assert stb.gemm_workspace(1024, 8192, 4, 2048) > 8 << 20
    xb = torch.empty(2048, 8192, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(stb.StbError) as e:
        stb.gemm_noalloc(big, xb, torch.empty(2048, 1024, device="cuda"))
    assert e.value.status == stb.STB_ERR_SIZE
