"""Pins of the CPU oracle against what the paper and the mathematics fix.

Nothing here touches the CUDA library.  Each test is chosen so that a plausible
mistake in oracle/stb_oracle.cpp (dropped term, wrong sign or index, transposed
operand, wrong comparison) fails it.
"""
import itertools
import math
import os

import numpy as np
import pytest

import oracle
import stb_inputs as si
from conftest import GOLDEN


def unpack_keep(keep):
    n, ng = keep.shape
    return np.unpackbits(keep[:, :, None], axis=2, bitorder="little").reshape(n, ng * 8).astype(bool)


# ----------------------------------------------------------------------------- fp16
def test_half_to_float_all_patterns_match_numpy():
    h = np.arange(65536, dtype=np.uint16)
    ref = h.view(np.float16).astype(np.float32)
    got = np.array([oracle.half_to_float(int(v)) for v in h], dtype=np.float32)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32))


def test_double_to_half_rounding_matches_numpy():
    g = np.random.default_rng(1)
    xs = np.concatenate([
        g.standard_normal(4000) * 0.02, g.standard_normal(2000) * 1e-6,      # normals, subnormals
        g.standard_normal(2000) * 3e4, [0.0, -0.0, 65504.0, 65519.9, 65520.0, 1e9, 2.0 ** -25,
                                        2.0 ** -24, 1.5 * 2.0 ** -24, 2.0 ** -14],
        # exact ties between neighbouring halfs (round to even)
        np.arange(1024, 1100, dtype=np.float64) * 2.0 ** -10 + 2.0 ** -11])
    for x in xs:
        for s in (1.0, -1.0):
            with np.errstate(over="ignore"):
                want = int(np.float64(s * x).astype(np.float16).view(np.uint16))
            assert oracle.double_to_half(s * x) == want, (s * x)


# ----------------------------------------------------------------------------- Eq. 3 (SI)
def test_si_hand_worked_example():
    """Golden: Eq. 3 worked by hand for a 2x2 matrix (tests/golden/si_worked_2x2.txt)."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "si_worked_2x2.txt"))
            if l.strip() and not l.startswith("#")]
    S = oracle.si_scores(np.array([[1.0, 3.0], [2.0, 2.0]]), np.array([2.0, 1.0]))
    for i, j, v in rows:
        assert abs(S[int(i), int(j)] - float(v)) < 2e-7


def test_si_rank_one_closed_form_and_invariances():
    g = np.random.default_rng(2)
    n, m = 12, 24
    u = g.random(n) + 0.1
    v = g.random(m) + 0.1
    xn = g.random(m) + 0.5
    sgn = g.choice([-1.0, 1.0], size=(n, m))
    W = np.outer(u, v) * sgn
    # |W| = u v^T  =>  mu_ij = v_j / sum(v) + u_i / sum(u)  (closed form of this special case)
    mu = v[None, :] / v.sum() + u[:, None] / u.sum()
    assert abs(mu.mean() - (n + m) / (n * m)) < 1e-15        # holds for any W without zero lines
    want = (mu - mu.mean()) / mu.std() * xn[None, :]
    S = oracle.si_scores(W, xn)
    assert np.allclose(S, want, rtol=1e-12, atol=1e-12)
    # invariances of Eq. 3: sign flips and a global rescale of W leave S unchanged;
    # permuting rows / columns permutes S
    Wg = g.standard_normal((n, m))
    S0 = oracle.si_scores(Wg, xn)
    assert np.allclose(oracle.si_scores(-3.7 * Wg, xn), S0, rtol=1e-11, atol=1e-12)
    pr, pc = g.permutation(n), g.permutation(m)
    assert np.allclose(oracle.si_scores(Wg[pr][:, pc], xn[pc]), S0[pr][:, pc], rtol=1e-11, atol=1e-12)
    # z has zero mean and unit population variance; scaling one column norm scales that column
    z = oracle.si_scores(Wg, np.ones(m))
    assert abs(z.mean()) < 1e-12 and abs(z.std() - 1) < 1e-12
    xn2 = xn.copy(); xn2[5] *= 4
    S2 = oracle.si_scores(Wg, xn2)
    assert np.allclose(S2[:, 5], 4 * S0[:, 5]) and np.allclose(np.delete(S2, 5, 1), np.delete(S0, 5, 1))


def test_si_zero_row_and_column_are_finite():
    W = np.zeros((4, 8)); W[1, 2] = 1.0; W[2, 3] = -2.0
    S = oracle.si_scores(W, np.ones(8))
    assert np.isfinite(S).all()


# ----------------------------------------------------------------------------- N:M
@pytest.mark.parametrize("N", [1, 2, 3, 4, 5, 6, 7, 8])
def test_nm_select_brute_force_8x16(N):
    """Section 3.3: the kept mask of every group maximises the summed score over all
    C(8,N) masks (brute-force enumeration on 8x16 matrices)."""
    g = np.random.default_rng(10 + N)
    for trial in range(5):
        S = g.standard_normal((8, 16))
        keep = oracle.nm_select(S, N)
        kb = unpack_keep(keep)
        assert (kb.reshape(8, 2, 8).sum(axis=2) == N).all()
        for i in range(8):
            for gr in range(2):
                s = S[i, gr * 8:(gr + 1) * 8]
                best = max(sum(s[c] for c in comb) for comb in itertools.combinations(range(8), N))
                got = s[kb[i, gr * 8:(gr + 1) * 8]].sum()
                assert abs(got - best) < 1e-12


def test_nm_select_ties_go_to_lower_column():
    S = np.zeros((1, 8)); S[0, 6] = 1.0
    kb = unpack_keep(oracle.nm_select(S, 3))[0]
    assert list(np.nonzero(kb)[0]) == [0, 1, 6]


# ----------------------------------------------------------------------------- Binary / residual
def _quantize_small(n, m, N, seed):
    W = si.dense_weight(n, m, seed).astype(np.float64)
    xn = si.calib_norms(m, seed)
    L, bp, nsal = oracle.quantize(W, xn, N, nthreads=2)
    return W, xn, L, bp, nsal


def test_binary_scale_is_the_l2_optimum_brute_force():
    """Eq. 1 / Algorithm 2 Binary: alpha = mean|w| and B = sign(w) minimise ||w - alpha b||^2
    over all sign patterns b and all alpha (brute force, k <= 6).  Checked on the decoded
    output of a layer whose blocks degenerate to one region."""
    g = np.random.default_rng(3)
    for k in (1, 2, 3, 6):
        w = g.standard_normal(k)
        best = (math.inf, None, None)
        for b in itertools.product([-1.0, 1.0], repeat=k):
            b = np.array(b)
            a = float(w @ b) / k                      # least-squares alpha for this pattern
            e = float(((w - a * b) ** 2).sum())
            if a >= 0 and e < best[0] - 1e-15:
                best = (e, a, b)
        e, a, b = best
        assert abs(a - np.abs(w).mean()) < 1e-12 and np.array_equal(b, np.where(w >= 0, 1.0, -1.0))
        assert abs(e - ((w * w).sum() - k * a * a)) < 1e-12        # closed form used in the search


def test_residual_scales_signs_and_error_closed_form():
    """Eq. 4 / Res_Approx on the kept salient weights of every row-block: alpha1 = mean|w|,
    r = w - alpha1 sign(w), alpha2 = mean|r|; residual error = single error - k alpha2^2 <= single."""
    n, m, N = 24, 256, 5
    W, xn, L, bp, nsal = _quantize_small(n, m, N, 21)
    kb = unpack_keep(L.keep)
    What = oracle.decode(L).astype(np.float64)
    for b in range(m // 128):
        sal = np.array([(int(L.salient[b, c >> 6]) >> (c & 63)) & 1 for c in range(128)], bool)
        assert sal.sum() == nsal[b] >= 1
        for i in range(n):
            sel = kb[i, b * 128:(b + 1) * 128] & sal
            w = W[i, b * 128:(b + 1) * 128][sel]
            k = len(w)
            if k == 0:
                assert L.scale[i, b, 3] == 0 and L.scale[i, b, 4] == 0
                continue
            a1 = np.abs(w).mean()
            s1 = np.where(w >= 0, 1.0, -1.0)
            r = w - a1 * s1
            a2 = np.abs(r).mean()
            s2 = np.where(r >= 0, 1.0, -1.0)
            h1 = np.float16(a1); h2 = np.float16(a2)
            assert L.scale[i, b, 3] == h1.view(np.uint16) and L.scale[i, b, 4] == h2.view(np.uint16)
            # residual sign bits: t-th salient column, ascending
            cols = np.nonzero(sal)[0]
            want_bits = 0
            for t, c in enumerate(cols):
                if kb[i, b * 128 + c]:
                    wc = W[i, b * 128 + c]
                    rc = wc - a1 * (1.0 if wc >= 0 else -1.0)
                    if rc >= 0:
                        want_bits |= 1 << t
            assert int(L.sign2[i, b]) == want_bits
            dec = What[i, b * 128:(b + 1) * 128][sel]
            want = (np.float32(float(h1)) * s1.astype(np.float32)
                    + np.float32(float(h2)) * s2.astype(np.float32)).astype(np.float64)
            assert np.array_equal(dec, want)
            e_single = (w * w).sum() - k * a1 * a1
            e_res = ((w - a1 * s1 - a2 * s2) ** 2).sum()
            assert abs(e_res - (e_single - k * a2 * a2)) < 1e-12 and e_res <= e_single + 1e-15


# ----------------------------------------------------------------------------- trisection
def test_breakpoint_search_matches_naive_second_loop_and_counts_70():
    """Algorithm 2 NonSalientAwareQuant re-evaluated with an independent naive loop: same error
    for each of the 160 grid points, exactly 70 evaluated (sigma = 2, skip p2 > 0.9 max),
    the first strict minimum is returned, and three regions never lose to one region."""
    n, m, N = 16, 256, 4
    W, xn, L, bp, nsal = _quantize_small(n, m, N, 33)
    kb = unpack_keep(L.keep)
    grid = np.linspace(0.1, 0.9, 160)
    for b in range(m // 128):
        sal = np.array([(int(L.salient[b, c >> 6]) >> (c & 63)) & 1 for c in range(128)], bool)
        p1, p2, ev, errs = oracle.breakpoint_search(W, L.keep, sal.astype(np.uint8), b)
        assert ev == 70 and np.isnan(errs[70:]).all() and np.isfinite(errs[:70]).all()
        assert (p1, p2) == (bp[b, 0], bp[b, 1])
        blk = W[:, b * 128:(b + 1) * 128]
        use = kb[:, b * 128:(b + 1) * 128] & ~sal[None, :]
        mx = np.abs(blk[use]).max()
        naive = []
        for frac in grid[:70]:
            q1, q2 = frac * mx, 2 * frac * mx
            e = 0.0
            for i in range(n):
                w = blk[i][use[i]]
                for part in (w[np.abs(w) > q2], w[(np.abs(w) > q1) & (np.abs(w) <= q2)], w[np.abs(w) <= q1]):
                    if len(part):
                        a = np.abs(part).mean()
                        e += ((part - a * np.where(part >= 0, 1, -1)) ** 2).sum()
            naive.append(e)
        naive = np.array(naive)
        assert np.allclose(errs[:70], naive, rtol=1e-10, atol=1e-14)
        t = int(np.argmin(naive))                       # argmin returns the first minimum
        assert abs(p1 - grid[t] * mx) < 1e-15 and abs(p2 - 2 * grid[t] * mx) < 1e-15
        one_region = sum(((w - np.abs(w).mean() * np.where(w >= 0, 1, -1)) ** 2).sum()
                         for w in (blk[i][use[i]] for i in range(n)) if len(w))
        assert naive.min() <= one_region + 1e-12
        assert grid[70] * 2 > 0.9 >= grid[69] * 2


def test_region_ids_follow_the_printed_comparisons():
    """Trisection: sparse |w| > p2, intermediate p1 < |w| <= p2, dense |w| <= p1; region 3 iff the
    column is salient; per-row per-region scale is the l1 mean rounded to fp16."""
    n, m, N = 16, 256, 6
    W, xn, L, bp, nsal = _quantize_small(n, m, N, 34)
    kb = unpack_keep(L.keep)
    for i in range(n):
        for b in range(m // 128):
            sums = np.zeros(3); cnt = np.zeros(3, int)
            for gl in range(16):
                gi = b * 16 + gl
                rank = 0
                for c8 in range(8):
                    j = gi * 8 + c8
                    if not kb[i, j]:
                        continue
                    code = (int(L.region[i, gi]) >> (2 * rank)) & 3
                    sbit = (int(L.sign[i, gi]) >> rank) & 1
                    assert sbit == (1 if W[i, j] >= 0 else 0)
                    c = j - b * 128
                    is_sal = (int(L.salient[b, c >> 6]) >> (c & 63)) & 1
                    a = abs(W[i, j])
                    if is_sal:
                        assert code == 3
                    else:
                        want = 2 if a > bp[b, 1] else (1 if a > bp[b, 0] else 0)
                        assert code == want
                        sums[code] += a; cnt[code] += 1
                    rank += 1
                assert rank == N and int(L.sign[i, gi]) >> N == 0 and int(L.region[i, gi]) >> (2 * N) == 0
            for r in range(3):
                want = np.float16(sums[r] / cnt[r]) if cnt[r] else np.float16(0)
                assert L.scale[i, b, r] == want.view(np.uint16)


# ----------------------------------------------------------------------------- salient search
def test_salient_search_naive_reevaluation():
    n, m, N = 12, 256, 4
    W, xn, L, bp, nsal = _quantize_small(n, m, N, 35)
    kb = unpack_keep(L.keep)
    lam = 0.01 * np.mean(2 * xn * xn)
    for b in range(m // 128):
        ns, order, errs = oracle.salient_search(W, L.keep, xn, lam, b)
        blk = W[:, b * 128:(b + 1) * 128]
        score = (2 * xn[b * 128:(b + 1) * 128] ** 2 + lam) * (blk * blk).sum(axis=0)
        assert list(order) == list(np.argsort(-score, kind="stable")[:32])
        naive = []
        for i in range(1, 33):
            sal = np.zeros(128, bool); sal[order[:i]] = True
            e = 0.0
            for r in range(n):
                for sel in (kb[r, b * 128:(b + 1) * 128] & sal, kb[r, b * 128:(b + 1) * 128] & ~sal):
                    w = blk[r][sel]
                    if len(w):
                        e += ((w - np.abs(w).mean() * np.where(w >= 0, 1, -1)) ** 2).sum()
            naive.append(e)
        assert np.allclose(errs, naive, rtol=1e-10)
        assert ns == int(np.argmin(naive)) + 1 >= 1 and ns == nsal[b]


def test_outlier_columns_are_found_salient():
    """The x10 weight columns of the synthetic layer dominate the column score, so whenever a
    block holds such a column the search must include it among the salient ones."""
    n, m, N, seed = 32, 512, 4, 36
    W, xn, L, bp, nsal = _quantize_small(n, m, N, seed)
    out = si.outlier_channels(m, seed, 0.01, 2)
    assert len(out) == 5
    for j in out:
        b, c = divmod(int(j), 128)
        assert (int(L.salient[b, c >> 6]) >> (c & 63)) & 1


# ----------------------------------------------------------------------------- decode + matmul
def test_decode_special_case_plain_binarization():
    """N = 8, no salient column, a single region: the layer is the textbook alpha*sign(W) of
    Eq. 1, and y is its product with x."""
    g = np.random.default_rng(5)
    n, m = 8, 256
    Wd = g.standard_normal((n, m))
    alpha = np.abs(Wd).reshape(n, 2, 128).mean(axis=2).astype(np.float16)
    sign = np.packbits((Wd >= 0).reshape(n, m // 8, 8), axis=2, bitorder="little").reshape(n, m // 8)
    scale = np.zeros((n, 2, 5), np.uint16); scale[:, :, 0] = alpha.view(np.uint16)
    L = oracle.Logical(n, m, 8, np.full((n, m // 8), 255, np.uint8), sign,
                       np.zeros((n, m // 8), np.uint16), np.zeros((n, 2), np.uint32),
                       np.zeros((2, 2), np.uint64), scale)
    What = oracle.decode(L)
    want = np.repeat(alpha.astype(np.float32), 128, axis=1) * np.where(Wd >= 0, 1, -1).astype(np.float32)
    assert np.array_equal(What, want)
    x = g.standard_normal((3, m))
    y = oracle.matmul(What, x)
    ref = np.zeros((3, n))
    for t in range(3):
        for i in range(n):
            ref[t, i] = math.fsum(float(want[i, j]) * x[t, j] for j in range(m))
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-12)
    rows = np.array([5, 0, 7], np.int32)
    assert np.allclose(oracle.layer_rows(L, rows, x), ref[:, rows], rtol=1e-12, atol=1e-12)


def test_decode_element_by_element_python():
    """Decode of a drawn logical layer re-derived element by element with Python integers:
    rank order of sign / region bits, residual bit of the t-th salient column, zeros where dropped."""
    d = si.logical_layer(8, 256, 5, 77)
    L = oracle.Logical(**d)
    What = oracle.decode(L)
    sc = L.scale.view(np.float16).astype(np.float32)
    for i in range(L.n):
        for b in range(2):
            cols = [c for c in range(128) if (int(L.salient[b, c >> 6]) >> (c & 63)) & 1]
            for gl in range(16):
                gi = b * 16 + gl
                pos = [c for c in range(8) if (int(L.keep[i, gi]) >> c) & 1]
                for c8 in range(8):
                    j = gi * 8 + c8
                    if c8 not in pos:
                        assert What[i, j] == 0
                        continue
                    k = pos.index(c8)
                    s = 1.0 if (int(L.sign[i, gi]) >> k) & 1 else -1.0
                    code = (int(L.region[i, gi]) >> (2 * k)) & 3
                    if code == 3:
                        t = cols.index(gl * 8 + c8)
                        s2 = 1.0 if (int(L.sign2[i, b]) >> t) & 1 else -1.0
                        want = np.float32(np.float32(s) * sc[i, b, 3] + np.float32(s2) * sc[i, b, 4])
                    else:
                        want = np.float32(s) * sc[i, b, code]
                    assert What[i, j] == want


def test_matmul_matches_numpy_float64_and_is_not_transposed():
    g = np.random.default_rng(6)
    What = g.standard_normal((40, 128)).astype(np.float32)
    x = g.standard_normal((5, 128))
    y = oracle.matmul(What, x, nthreads=3)
    assert y.shape == (5, 40)
    assert np.allclose(y, x @ What.astype(np.float64).T, rtol=1e-13, atol=1e-13)


# ----------------------------------------------------------------------------- bit accounting
def test_average_bits_against_table_1():
    """Section 3.4 "Average Bits": N_stbllm = (1 + r_sal) * N/8.  With r_sal read off the dense
    column (dense bits = 1 + r_sal) every N:8 entry of Table 1 is reproduced to its printed
    two decimals (both operands are rounded in print, hence the 0.0076 allowance)."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table1_average_bits.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 11
    for fam, size, dense, b48, b58, b68 in rows:
        r = float(dense) - 1.0
        assert abs(oracle.average_bits(8, r) - float(dense)) < 1e-12
        for N, printed in ((4, b48), (5, b58), (6, b68)):
            assert abs(oracle.average_bits(N, r) - float(printed)) <= 0.005 + 0.005 * N / 8 + 1e-9


def test_counted_bits_identity_and_six_bit_encoding():
    for N, seed in ((4, 41), (5, 42), (6, 43)):
        W, xn, L, bp, nsal = _quantize_small(32, 256, N, seed)
        bits, r = oracle.counted_bits(L)
        assert abs(bits - oracle.average_bits(N, r)) < 1e-12
        assert 0 < r < 0.25
    # Appendix C: a 2:4 group costs 4 index bits + 2 sign bits = 6 bits against 8 bits for four
    # 2-bit ternary codes: 25 % smaller, at most 8/6 = 1.333x faster when memory-bound.  The same
    # count per 8 columns at 4:8 with an 8-bit mask: 8 + 4 = 12 bits = 1.5 bit per weight.
    assert (8 - 6) / 8 == 0.25 and abs(8 / 6 - 1.333) < 1e-3 and (8 + 4) / 8 == 2 * 6 / 8


# ----------------------------------------------------------------------------- whole-quantizer invariants
@pytest.mark.parametrize("N", [3, 4, 5, 6])
def test_quantizer_invariants(N):
    n, m = 48, 384
    W, xn, L, bp, nsal = _quantize_small(n, m, N, 50 + N)
    kb = unpack_keep(L.keep)
    assert (kb.reshape(n, m // 8, 8).sum(axis=2) == N).all()           # exactly N of every 8
    What = oracle.decode(L).astype(np.float64)
    assert (What[~kb] == 0).all() and (What[kb] != 0).any()
    # structured-binary error on the kept weights never exceeds plain one-scale binarization of
    # the same kept weights per row-block (three regions + residual only remove error; the fp16
    # rounding of the scales is far below the margin)
    for b in range(m // 128):
        sl = slice(b * 128, (b + 1) * 128)
        for i in range(n):
            w = W[i, sl][kb[i, sl]]
            e1 = ((w - np.abs(w).mean() * np.where(w >= 0, 1, -1)) ** 2).sum()
            e3 = ((w - What[i, sl][kb[i, sl]]) ** 2).sum()
            assert e3 <= e1 * (1 + 1e-3) + 1e-9
    # determinism and thread-count independence
    L2, _, _ = oracle.quantize(W, xn, N, nthreads=1)
    for f in ("keep", "sign", "region", "sign2", "salient", "scale"):
        assert np.array_equal(getattr(L, f), getattr(L2, f))


def test_degenerate_all_zero_and_all_equal_blocks():
    n, m, N = 8, 256, 4
    W = np.zeros((n, m)); W[:, 128:] = 0.5
    L, bp, nsal = oracle.quantize(W, np.ones(m), N)
    kb = unpack_keep(L.keep)
    assert (kb.reshape(n, m // 8, 8).sum(axis=2) == N).all()
    What = oracle.decode(L)
    assert (What[:, :128] == 0).all()
    assert np.array_equal(What[:, 128:][kb[:, 128:]], np.full(kb[:, 128:].sum(), 0.5, np.float32))


def test_silu_mul_identities():
    """The gated activation fp16(silu(a) * b): silu(v) - silu(-v) = v, silu(0) = 0, silu(ln 3) = 0.75 ln 3, silu(v) -> v for
    large v, linear in b; results are fp16 values (checked against numpy's rounding of the closed forms)."""
    import math
    v = np.array([0.0, math.log(3.0), 30.0, -30.0, 2.5, -2.5, 0.125], np.float64)
    one = np.ones_like(v)
    s = oracle.silu_mul(v, one)
    want = np.array([0.0, 0.75 * math.log(3.0), 30.0, 0.0, 0.0, 0.0, 0.0])
    assert s[0] == 0.0 and s[1] == np.float64(np.float16(want[1])) and s[2] == 30.0 and abs(s[3]) < 1e-11
    # silu(v) - silu(-v) = v: with b = 1 both terms are rounded to fp16, so compare within fp16 rounding of each
    assert abs((s[4] - s[5]) - 2.5) <= 2.0 ** -10 * 2.5
    # linear in b (exactly: scaling by a power of two commutes with the rounding)
    assert np.array_equal(oracle.silu_mul(v, 4.0 * one), 4.0 * s)
    assert np.array_equal(oracle.silu_mul(v, -one), -s)
    # fp16 output: every value is representable
    assert np.array_equal(s.astype(np.float16).astype(np.float64), s)


def test_layerwise_nm_assignment():
    """Section 3.3: alpha_i = omega_i / sum omega, N_i / 8 = alpha_i + (1 - alpha_i) R.  Hand-worked: norms (3, 1), R = 1/2:
    alpha = (3/4, 1/4), ratios (7/8, 5/8), N = (7, 5).  Equal norms give equal N; the ratio never falls below R and
    reaches 1 only for a layer that holds all the norm; the mean ratio is R + (1 - R) / L."""
    N, ratio = oracle.allocate_nm([3.0, 1.0], 0.5)
    assert list(N) == [7, 5] and np.allclose(ratio, [0.875, 0.625], rtol=0, atol=1e-15)
    N, ratio = oracle.allocate_nm([2.0] * 32, 0.5)
    assert len(set(N)) == 1 and N[0] == 4 and np.allclose(ratio.mean(), 0.5 + 0.5 / 32)
    g = np.random.default_rng(3)
    w = g.random(40) + 0.1
    for R in (0.375, 0.5, 0.625, 0.75):
        N, ratio = oracle.allocate_nm(w, R)
        assert (ratio >= R).all() and (ratio < 1).all() and np.isclose(ratio.mean(), R + (1 - R) / 40)
        assert (np.argsort(ratio, kind="stable") == np.argsort(w, kind="stable")).all()      # monotone in the norm
        assert ((N >= 1) & (N <= 8)).all() and (np.abs(N - 8 * ratio) <= 0.5).all()
    N, ratio = oracle.allocate_nm([5.0, 0.0, 0.0], 0.5)
    assert list(N) == [8, 4, 4] and ratio[0] == 1.0
