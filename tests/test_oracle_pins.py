"""Pins the CPU oracle to what the paper and the mathematics fix (no GPU).

Each test names the passage it checks.  None of them re-uses the oracle's own
binary32 formula: the references are a hand-worked fixture, exact rational or
binary64 true-division restatements of Eq. 1 / Eq. 3, library rounding, and the
closed forms Eq. 2, 5, 9, 10 and Lemma 2.
"""
import math

import numpy as np
import pytest
from scipy import stats

from conftest import read_golden
from paper_2002_00104_b200 import workloads as W


def bits_of(mask, total):
    return np.unpackbits(np.asarray(mask, dtype=np.uint8), bitorder="little")[:total]


# ---------------------------------------------------------------- worked example (Eq. 1, Eq. 3)
def test_worked_example_b3(oracle):
    g = read_golden("worked_example_b3.txt")
    bits = int(g["bits"][0])
    x = np.array([float(v) for v in g["x"]], dtype=np.float32)
    ratios = np.array([float(v) for v in g["ratios"]], dtype=np.float32)
    m = oracle.absmax(x)
    assert m.tolist() == [float(g["m"][0])]
    res = oracle.search(x, bits, ratios)
    assert res["idx"].tolist() == [int(g["argmin"][0])]
    assert res["p"].tolist() == [float(g["p_star"][0])]
    assert res["err"].tolist() == [float(g["err_star"][0])]
    for k, p in enumerate(float(v) for v in g["p"]):
        assert res["sse64"][0, k] == float(g[f"sse.{k}"][0])
        assert res["sse"][0, k] == np.float32(float(g[f"sse.{k}"][0]))
        pk = np.array([p], dtype=np.float32)
        codes, mask, fake = oracle.quantize(x, bits, m, pk, layout=0)
        assert codes.tolist() == [int(v) for v in g[f"code.{k}"]]
        assert bits_of(mask, x.size).tolist() == [int(v) for v in g[f"region.{k}"]]
        want_y = np.array([float(v) for v in g[f"y.{k}"]], dtype=np.float32)
        assert fake.tobytes() == want_y.tobytes()          # also pins the sign of zero
        y = oracle.dequantize(codes, mask, bits, m, pk, C=1, n=x.size)
        assert y.tobytes() == want_y.tobytes()
        if f"q.{k}" in g:
            for xi, qi in zip(x, g[f"q.{k}"]):
                assert oracle.elem(xi, m[0], p, bits)[2] == int(qi)
    packed, mask, _ = oracle.quantize(x, bits, m, np.array([3.0], np.float32), layout=1)
    assert packed.tolist() == [int(v, 16) for v in g["packed.0"]]
    assert mask.tolist() == [int(v, 16) for v in g["mask.0"]]
    y = oracle.dequantize(packed, mask, bits, m, np.array([3.0], np.float32), C=1, n=16, layout=1)
    assert y.tobytes() == np.array([float(v) for v in g["y.0"]], np.float32).tobytes()


def test_absmax_rows_and_sign(oracle):
    x = np.array([[1.0, -7.5, 3.0], [0.0, -0.0, 0.0], [-2.0, 1.0, 1.5]], dtype=np.float32)
    assert oracle.absmax(x).tolist() == [7.5, 0.0, 2.0]
    ro = np.array([0, 1, 1, 4, 9], dtype=np.int64)      # ragged, with an empty row
    assert oracle.absmax(x.reshape(-1), ro).tolist() == [1.0, 0.0, 7.5, 2.0]
    with pytest.raises(oracle.OracleError):
        oracle.absmax(np.array([1.0, np.inf], dtype=np.float32))
    with pytest.raises(oracle.OracleError):
        oracle.absmax(np.array([np.nan, 1.0], dtype=np.float32))


# ---------------------------------------------------------------- Eq. 1: step and level count
@pytest.mark.parametrize("bits", [2, 3, 4, 6, 8])
def test_params_step_is_range_over_levels(oracle, bits):
    """s = Delta / (N - 1) with N = 2^(b-1) levels in each of the four pieces (Eq. 1, Sec. 3.2)."""
    m, p = np.float32(1.75), np.float32(0.4375)
    L, s1, inv1, s2, inv2 = oracle.params(m, p, bits)
    assert L == 2 ** (bits - 1) - 1
    assert s1 == np.float32(p) / np.float32(L) and inv1 == np.float32(L) / np.float32(p)
    d = np.float32(m - p)
    assert s2 == d / np.float32(L) and inv2 == np.float32(L) / d
    # Sec. 3.2: as many reconstruction levels in total as a (b+1)-bit uniform quantizer
    xs = np.linspace(-m, m, 20001).astype(np.float32)
    _, _, fake = oracle.quantize(xs, bits, [m], [p])
    assert np.unique(fake).size <= 2 ** (bits + 1)
    assert np.unique(fake).size >= 2 ** (bits + 1) - 3   # +-0 merge; level p reachable from both sides


# ---------------------------------------------------------------- invariants implied by Eq. 1-3
@pytest.mark.parametrize("bits", [2, 3, 4, 5, 8])
def test_levels_regions_and_half_step_bound(oracle, bits):
    rng = np.random.default_rng(100 + bits)
    L = 2 ** (bits - 1) - 1
    for trial in range(60):
        n = int(rng.integers(1, 400))
        x = (rng.laplace(0, 1, n) * 10.0 ** rng.uniform(-3, 2)).astype(np.float32)
        m = oracle.absmax(x)
        p = np.float32(m[0] * rng.uniform(0.02, 1.0))
        codes, mask, fake = oracle.quantize(x, bits, m, [p])
        region = bits_of(mask, n)
        q = codes & L
        neg = codes >> (bits - 1)
        a = np.abs(x)
        assert q.max() <= L and neg.max() <= 1
        assert np.array_equal(region == 1, a > p)                     # R1 closed, R2 open at p
        assert np.array_equal(neg == 1, x < 0)
        step = np.where(region == 1, (np.float64(m[0]) - np.float64(p)) / L, np.float64(p) / L)
        err = np.abs(np.abs(fake.astype(np.float64)) - a)
        slack = 4 * np.spacing(np.float32(m[0]))
        assert np.all(err <= step / 2 + slack)                        # rounding: at most half a step
        assert np.all(np.sign(fake) * np.sign(x) >= 0)
        y = oracle.dequantize(codes, mask, bits, m, [p], C=1, n=n)
        assert y.tobytes() == fake.tobytes()
        res = oracle.search(x, bits, [p / m[0]], m=m)
        if np.float32(m[0] * np.float32(p / m[0])) == p:
            sse = np.sum((np.abs(fake.astype(np.float64)) - a.astype(np.float64)) ** 2)
            assert math.isclose(res["sse64"][0, 0], sse, rel_tol=1e-12)


@pytest.mark.parametrize("bits", [2, 3, 4, 6, 8])
def test_p_equals_m_is_symmetric_uniform(oracle, bits):
    """p = m: no tail, pw(x) = sign(x) * uni(|x|; b-1, 0, m, 0)  (Eq. 3 with R2 empty)."""
    rng = np.random.default_rng(bits)
    x = rng.normal(0, 0.3, 5000).astype(np.float32)
    m = oracle.absmax(x)
    L = np.float32(2 ** (bits - 1) - 1)
    codes, mask, fake = oracle.quantize(x, bits, m, m)
    assert not mask.any()
    inv = L / m[0]
    s = m[0] / L
    q = np.minimum(np.rint((np.abs(x) * inv).astype(np.float32)), L)   # library half-even rounding
    want = np.copysign((q * s).astype(np.float32), np.where(x < 0, -1.0, 1.0)).astype(np.float32)
    assert np.array_equal(fake, want)
    assert np.array_equal(codes & int(L), q.astype(np.uint8))


@pytest.mark.parametrize("bits", [3, 4, 8])
def test_p_half_m_has_equal_steps(oracle, bits):
    """p = m/2: the four pieces have equal ranges and steps (Sec. 3.3)."""
    m = np.float32(3.1415927)
    p = np.float32(m * np.float32(0.5))
    L, s1, inv1, s2, inv2 = oracle.params(m, p, bits)
    assert s1 == s2 and inv1 == inv2
    xs = np.linspace(0, m, 4001).astype(np.float32)
    _, _, fake = oracle.quantize(xs, bits, [m], [p])
    lv = np.unique(fake)
    gaps = np.diff(lv.astype(np.float64))
    assert np.allclose(gaps, float(s1), rtol=0, atol=4 * float(np.spacing(m)))


# ---------------------------------------------------------------- brute force (Eq. 3, Eq. 6)
def pw_double(x, m, p, bits):
    """Independent binary64 restatement of Eq. 3 with true division."""
    L = 2 ** (bits - 1) - 1
    a = np.minimum(np.abs(x.astype(np.float64)), m)
    tail = a > p
    with np.errstate(divide="ignore", invalid="ignore"):
        s = np.where(tail, (m - p) / L, p / L)
        z = np.where(tail, p, 0.0)
        t = np.where(s > 0, (a - z) / s, 0.0)
    q = np.minimum(np.rint(t), L)
    return q, tail, q * s + z, t


@pytest.mark.parametrize("bits,K", [(2, 16), (3, 32), (4, 64), (8, 64)])
def test_bruteforce_dense_grid_tiny_rows(oracle, bits, K):
    rng = np.random.default_rng(bits * 1000 + K)
    dense = 4096
    for trial in range(12):
        n = int(rng.integers(2, 65))
        x = (rng.standard_normal(n) if trial % 2 else rng.laplace(0, 1, n)).astype(np.float32)
        x *= np.float32(10.0 ** rng.uniform(-2, 1))
        m = float(oracle.absmax(x)[0])
        ratios = W.ratio_grid(K)
        res = oracle.search(x, bits, ratios)
        # dense curve in binary64 contains the K-grid points exactly (dense % K == 0)
        dr = (np.arange(1, dense + 1, dtype=np.float64)) / dense
        curve = np.array([np.sum((pw_double(x, m, m * r, bits)[2] - np.abs(x.astype(np.float64))) ** 2)
                          for r in dr])
        on_grid = curve[dense // K - 1::dense // K]
        assert on_grid.size == K
        # oracle SSE (binary32 element arithmetic) follows the binary64 curve on the grid
        p32 = (np.float32(m) * ratios).astype(np.float64)
        exact = np.array([np.sum((pw_double(x, m, pk, bits)[2] - np.abs(x.astype(np.float64))) ** 2)
                          for pk in p32])
        flips = 0
        for k in range(K):
            q64, tail64, _, t = pw_double(x, m, p32[k], bits)
            codes, mask, _ = oracle.quantize(x, bits, [m], [np.float32(p32[k])])
            q32 = codes & (2 ** (bits - 1) - 1)
            assert np.array_equal(bits_of(mask, n) == 1, tail64)
            diff = q32 != q64
            # levels may differ only where t sits on a rounding tie up to binary32 noise
            frac = np.abs(t - np.floor(t) - 0.5)
            assert np.all(frac[diff] < 1e-4), (k, t[diff])
            flips += int(diff.sum())
        if flips == 0:
            # binary32 rounding moves each reconstructed value by at most d = 2 ulp(m); an error
            # e <= step/2 <= m/(2L) then changes e^2 by at most 2|e|d + d^2
            L = 2 ** (bits - 1) - 1
            d = 2.0 * float(np.spacing(np.float32(m)))
            assert np.allclose(res["sse64"][0], exact, rtol=1e-6, atol=n * (m / L * d + d * d))
        noise = n * (m / (2 ** (bits - 1) - 1) * 2.0 * float(np.spacing(np.float32(m))))
        # the chosen candidate is the best grid point of the dense curve (up to noise-level ties)
        best = int(np.argmin(exact))
        chosen = int(res["idx"][0])
        assert exact[chosen] <= exact[best] * (1 + 1e-6) + 2 * noise
        assert res["p"][0] == np.float32(m) * ratios[chosen]
        # and no K-grid point of the dense curve beats it by more than grid-rounding noise
        assert on_grid.min() >= exact[chosen] * (1 - 2e-2) - 2 * noise


# ---------------------------------------------------------------- argmin and tie-break (Eq. 6)
def test_lowest_index_wins_ties(oracle):
    x = np.array([2.5, -2.5, 2.5], dtype=np.float32)              # all |x| = m: every SSE is 0
    res = oracle.search(x, 4, W.ratio_grid(10))
    assert res["idx"][0] == 0 and res["err"][0] == 0.0
    rng = np.random.default_rng(5)
    x = rng.laplace(0, 1, 300).astype(np.float32)
    ratios = np.array([0.5, 0.2, 0.2, 0.9, 0.2], dtype=np.float32)   # duplicated best ratio
    res = oracle.search(x, 4, ratios)
    assert res["sse64"][0, 1] == res["sse64"][0, 2] == res["sse64"][0, 4]
    assert res["idx"][0] == int(np.argmin(res["sse64"][0]))           # numpy: first minimum
    assert res["idx"][0] == 1


def test_zero_rows_and_single_values(oracle):
    x = np.zeros((2, 5), dtype=np.float32)
    x[1, 2] = -3.0
    res = oracle.search(x, 4, W.ratio_grid(8))
    assert res["idx"].tolist() == [0, 0] and res["p"][0] == 0.0 and res["err"].tolist() == [0.0, 0.0]
    assert not res["sse64"].any()                # a lone value sits on the top level for any p
    codes, mask, fake = oracle.quantize(x, 4, [0.0, 3.0], [0.0, res["p"][1]])
    assert codes[:5].tolist() == [0] * 5 and fake[:5].tobytes() == np.zeros(5, np.float32).tobytes()
    assert fake[7] == -3.0 and codes[7] == 8 + 7


def test_ragged_rows_equal_dense_rows(oracle):
    w = W.small_mixed(seed=3, bits=4, K=16)
    ratios = W.ratio_grid(w.K)
    res = oracle.search(w.x, w.bits, ratios, row_offsets=w.row_offsets)
    m = oracle.absmax(w.x, w.row_offsets)
    codes, mask, fake = oracle.quantize(w.x, w.bits, m, res["p"], layout=1, row_offsets=w.row_offsets)
    y = oracle.dequantize(codes, mask, w.bits, m, res["p"], layout=1, row_offsets=w.row_offsets)
    assert y.tobytes() == fake.tobytes()
    for c in range(w.C):
        b, e = w.row_offsets[c], w.row_offsets[c + 1]
        one = oracle.search(w.x[b:e], w.bits, ratios)
        assert one["idx"][0] == res["idx"][c] and one["p"][0] == res["p"][c]
        assert np.array_equal(one["sse64"][0], res["sse64"][c])
        _, _, f1 = oracle.quantize(w.x[b:e], w.bits, m[c:c + 1], res["p"][c:c + 1])
        assert f1.tobytes() == fake[b:e].tobytes()


# ---------------------------------------------------------------- closed forms (Eq. 2, 5, 9, 10, Lemma 2)
def C_of(b):
    return 1.0 / (12.0 * (2 ** b - 1) ** 2)


def eq5(dist, b, m, p):
    """Expected squared error, Eq. 5: C(b-1) { (m-p)^2 + m (2p - m) [2F(p) - 1] }."""
    return C_of(b - 1) * ((m - p) ** 2 + m * (2 * p - m) * (2 * dist.cdf(p) - 1))


def eq9_root(dist, m):
    """p* solving Eq. 9: 2 m F(p) = 2m - p + m (m - 2p) f(p), by bisection on (0, m/2)."""
    g = lambda p: 2 * m * dist.cdf(p) - (2 * m - p + m * (m - 2 * p) * dist.pdf(p))
    lo, hi = 1e-9 * m, 0.5 * m
    assert g(lo) < 0 < g(hi)
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        lo, hi = (mid, hi) if g(mid) < 0 else (lo, mid)
    return 0.5 * (lo + hi)


def test_uniform_data_matches_eq2(oracle):
    """On uniformly distributed data every piece has error s^2/12 (Eq. 2); with p = m/2 the mean
    squared error is C(b-1) (m/2)^2, the quantity Lemma 2's proof compares against."""
    rng = np.random.default_rng(11)
    x = rng.uniform(-1, 1, 400000).astype(np.float32)
    x[0] = 1.0
    for b in (3, 4, 6):
        res = oracle.search(x, b, [0.5])
        mse = res["sse64"][0, 0] / x.size
        assert math.isclose(mse, C_of(b - 1) * 0.25, rel_tol=0.02)


@pytest.mark.parametrize("name,dist,scale,n", [("gauss", stats.norm, 1.0, 200000),
                                               ("laplace", stats.laplace, 1.0, 200000)])
@pytest.mark.parametrize("bits", [3, 4, 6])
def test_empirical_curve_follows_eq5_and_eq9(oracle, name, dist, scale, n, bits):
    rng = np.random.default_rng(42)
    x = (rng.standard_normal(n) if name == "gauss" else rng.laplace(0, 1, n)).astype(np.float32)
    m = float(oracle.absmax(x)[0])
    K = 200
    ratios = W.ratio_grid(K)
    res = oracle.search(x, bits, ratios)
    mse = res["sse64"][0] / n
    d = dist(0, scale)
    # Eq. 5 over the analysed range (0, m/2).  Eq. 5 assumes a flat density inside every cell
    # (Eq. 2), so the agreement tightens as the step shrinks: tolerances fall with b, and the
    # 3-bit Laplacian (tail step of 4 scale units at small p) is only compared for p >= m/4.
    tol = {("gauss", 3): 0.10, ("gauss", 4): 0.03, ("gauss", 6): 0.015,
           ("laplace", 3): 0.15, ("laplace", 4): 0.10, ("laplace", 6): 0.02}[(name, bits)]
    for k in range(9, K // 2, 10):
        p = m * float(ratios[k])
        if (name, bits) == ("laplace", 3) and k < 49:
            continue
        assert math.isclose(mse[k], eq5(d, bits, m, p), rel_tol=tol), k
    # Eq. 9: stationary point; Eq. 6: argmin lies in (0, m/2) for bell-shaped data
    p_star = eq9_root(d, m)
    assert abs(res["p"][0] / m - p_star / m) < 0.03
    assert 0 < res["p"][0] < m / 2
    # Eq. 10 gives the expected error at the optimum
    e10 = C_of(bits - 1) * (-p_star ** 2 + m * p_star - m * (m - 2 * p_star) ** 2 * d.pdf(p_star))
    assert math.isclose(eq5(d, bits, m, p_star), e10, rel_tol=1e-6)
    assert math.isclose(res["sse64"][0].min() / n, e10, rel_tol={3: 0.15, 4: 0.04, 6: 0.015}[bits])
    # Lemma 2: below C(b-1)/(16 C(b)) <= 9/16 of the b-bit uniform error 4 C(b) m^2
    uni = 4 * C_of(bits) * m * m
    assert res["sse64"][0].min() / n < C_of(bits - 1) / (16 * C_of(bits)) * uni
    assert C_of(bits - 1) / (16 * C_of(bits)) <= 9 / 16 + 1e-12
    # Lemma 1: convex, hence unimodal, on (0, m/2) up to sampling noise
    half = mse[:K // 2]
    kmin = int(np.argmin(half))
    sm = np.convolve(half, np.ones(5) / 5, mode="valid")
    kk = int(np.argmin(sm))
    assert np.all(np.diff(sm[:kk]) < 1e-3 * sm[kk]) and np.all(np.diff(sm[kk:]) > -1e-3 * sm[kk])
    assert abs(kmin - (kk + 2)) <= 6
    # Sec. 4 footnote: the bulk of the values (about 90 %) sits in the center region at p*
    _, mask, _ = oracle.quantize(x, bits, [m], res["p"])
    frac_center = 1.0 - bits_of(mask, n).mean()
    assert 0.75 < frac_center < 0.97


def test_ln_approximation_reading(oracle):
    """Sec. 5.1 prints p*/m = ln(0.8614 m + 0.6079) 'for normalized Gaussian'.  Taken literally it
    exceeds 1 at m = 3; read as p*/sigma = ln(0.8614 m/sigma + 0.6079) it reproduces the root of
    Eq. 9 to about 1 % and the empirical argmin of the oracle's curve."""
    for m in (3.0, 4.0, 5.0, 6.0, 8.0):
        root = eq9_root(stats.norm(0, 1), m)
        assert abs(math.log(0.8614 * m + 0.6079) - root) / root < 0.012
    assert math.log(0.8614 * 3 + 0.6079) > 1.0
    rng = np.random.default_rng(8)
    x = rng.standard_normal(300000).astype(np.float32)
    m = float(oracle.absmax(x)[0])
    res = oracle.search(x, 4, W.ratio_grid(400))
    assert abs(res["p"][0] - math.log(0.8614 * m + 0.6079)) < 0.12


# ---------------------------------------------------------------- analytic selection (Eq. 9, Sec. 5.1)
@pytest.mark.parametrize("model,dist", [(1, stats.norm), (2, stats.laplace)])
def test_analytic_root_matches_an_independent_solver(oracle, model, dist):
    """The oracle's bisection on Eq. 9 against scipy's Brent solver on the same equation written
    with scipy's CDF / PDF."""
    from scipy.optimize import brentq
    for m, scale in ((4.0, 1.0), (6.5, 1.0), (0.31, 0.05), (12.0, 1.3), (3.0, 0.4)):
        d = dist(0, scale)
        g = lambda p: 2 * m * d.cdf(p) - (2 * m - p + m * (m - 2 * p) * d.pdf(p))
        if g(0.5 * m) <= 0:
            assert oracle.analytic_p(m, scale, model) == 0.5 * m
            continue
        want = brentq(g, 1e-12 * m, 0.5 * m, xtol=1e-15, rtol=1e-14)
        assert math.isclose(oracle.analytic_p(m, scale, model), want, rel_tol=1e-9)
    # a row much flatter than the model: no stationary point inside (0, m/2), the bound is taken
    assert oracle.analytic_p(1.0, 5.0, 1) == 0.5


def test_analytic_approximation_and_scales(oracle):
    # Sec. 5.1 closed form in units of sigma, clamped to (0, m/2]
    assert math.isclose(oracle.analytic_p(5.0, 1.0, 0), math.log(0.8614 * 5.0 + 0.6079), rel_tol=1e-12)
    assert math.isclose(oracle.analytic_p(0.5, 0.1, 0), 0.1 * math.log(0.8614 * 5.0 + 0.6079), rel_tol=1e-12)
    assert oracle.analytic_p(2.0, 1.0, 0) == min(math.log(0.8614 * 2.0 + 0.6079), 1.0)
    assert oracle.analytic_p(0.0, 1.0, 0) == 0.0 and oracle.analytic_p(1.0, 0.0, 1) == 0.0
    rng = np.random.default_rng(17)
    x = rng.normal(0, 0.05, (3, 5000)).astype(np.float32)
    m = oracle.absmax(x)
    for model in (0, 1, 2):
        p, scale = oracle.select_analytic(x, m, model)
        ref = np.mean(np.abs(x.astype(np.float64)), axis=1) if model == 2 else \
            np.sqrt(np.mean(x.astype(np.float64) ** 2, axis=1))
        assert np.allclose(scale, ref, rtol=1e-12)
        want = [oracle.analytic_p(float(m[c]), float(scale[c]), model) for c in range(3)]
        assert np.array_equal(p, np.array(want, dtype=np.float32))


@pytest.mark.parametrize("name,model", [("gauss", 0), ("gauss", 1), ("laplace", 2)])
def test_analytic_choice_is_close_to_the_searched_optimum(oracle, name, model):
    """Sec. 5.1: the analytic breakpoint gives almost the same error as the minimiser.  Here: its
    squared error on the sample is within 3 % of the best grid candidate's (b = 4)."""
    rng = np.random.default_rng(23)
    n = 100000
    x = (rng.standard_normal(n) if name == "gauss" else rng.laplace(0, 1, n)).astype(np.float32)
    m = oracle.absmax(x)
    p, _ = oracle.select_analytic(x, m, model)
    grid = oracle.search(x, 4, W.ratio_grid(400))
    at_p = oracle.search(x, 4, [p[0] / m[0]])
    assert at_p["sse64"][0, 0] <= grid["sse64"][0].min() * 1.03
    assert 0 < p[0] <= m[0] / 2
