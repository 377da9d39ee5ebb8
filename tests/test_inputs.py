"""The seeded synthetic-input generators: determinism and the stated structure."""
import numpy as np

import stb_inputs as si


def test_dense_weight_and_activation_recipe():
    W = si.dense_weight(64, 1024, si.seed_for(1, 0))
    assert W.dtype == np.float16 and W.shape == (64, 1024)
    assert np.array_equal(W, si.dense_weight(64, 1024, si.seed_for(1, 0)))
    out = si.outlier_channels(1024, si.seed_for(1, 0), 0.01, 2)
    assert len(out) == 10 == len(set(out.tolist()))
    rest = np.delete(W.astype(np.float64), out, axis=1)
    assert abs(rest.std() - 0.02) < 2e-3 and abs(W[:, out].astype(np.float64).std() - 0.2) < 3e-2
    x = si.activations(4, 4096, 9)
    assert x.dtype == np.float16 and len(si.outlier_channels(4096, 9, 0.005, 4)) == 20
    xb = si.activations(4, 4096, 9, "bf16")
    assert np.array_equal(si.round_to_bf16(xb), xb) and (xb.view(np.uint32) & 0xFFFF == 0).all()
    xn = si.calib_norms(4096, 9)
    big = si.outlier_channels(4096, 9, 0.005, 4)
    assert xn[big].min() > 5 * np.delete(xn, big).max() * 0.5


def test_logical_layer_structure():
    for N in (3, 4, 5, 6, 8):
        d = si.logical_layer(40, 384, N, 100 + N)
        keep = d["keep"]
        assert (np.unpackbits(keep[:, :, None], axis=2).sum(axis=2) == N).all()
        assert (d["sign"].astype(int) >> N == 0).all() and (d["region"].astype(int) >> (2 * N) == 0).all()
        for b in range(3):
            cols = [c for c in range(128) if (int(d["salient"][b, c >> 6]) >> (c & 63)) & 1]
            assert 1 <= len(cols) <= 3
            assert (d["sign2"][:, b].astype(np.int64) >> len(cols) == 0).all()
            for i in range(0, 40, 7):
                for gl in range(16):
                    gi = b * 16 + gl
                    pos = [c for c in range(8) if (int(keep[i, gi]) >> c) & 1]
                    for k, c8 in enumerate(pos):
                        code = (int(d["region"][i, gi]) >> (2 * k)) & 3
                        assert (code == 3) == ((gl * 8 + c8) in cols)
                for t, c in enumerate(cols):
                    kept = (int(keep[i, b * 16 + c // 8]) >> (c % 8)) & 1
                    if not kept:
                        assert (int(d["sign2"][i, b]) >> t) & 1 == 0
        assert (d["scale"].view(np.float16) > 0).all()
        d2 = si.logical_layer(40, 384, N, 100 + N)
        assert all(np.array_equal(d[k], d2[k]) for k in d if isinstance(d[k], np.ndarray))
