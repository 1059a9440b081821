"""Pins the oracle's two-breakpoint quantizer and pair search (no GPU).

References: a hand-worked dyadic fixture; the already pinned one-breakpoint oracle (p2 = m makes
the third region empty); a binary64 true-division restatement; the half-step bound per region;
the ordering of the pair search.
"""
import numpy as np
import pytest

from conftest import read_golden
from paper_2002_00104_b200 import workloads as W


def regions_of(region2, total):
    b = np.asarray(region2, dtype=np.uint8)
    r = np.stack([(b >> (2 * t)) & 3 for t in range(4)], axis=1).reshape(-1)
    return r[:total]


def test_worked_example_two_breakpoints(oracle):
    g = read_golden("worked_example_two_breakpoints_b3.txt")
    bits = int(g["bits"][0])
    x = np.array([float(v) for v in g["x"]], dtype=np.float32)
    ratios = np.array([float(v) for v in g["ratios"]], dtype=np.float32)
    m = np.array([float(g["m"][0])], np.float32)
    assert oracle.absmax(x).tolist() == m.tolist()
    res = oracle.search2(x, bits, ratios, m)
    assert [int(res["idx1"][0]), int(res["idx2"][0])] == [int(v) for v in g["argmin"]]
    assert [float(res["p1"][0]), float(res["p2"][0])] == [float(v) for v in g["p_star"]]
    assert float(res["err"][0]) == float(g["err_star"][0])
    K = ratios.size
    for i in range(K):
        for j in range(i + 1, K):
            assert res["sse64"][0, i, j] == float(g[f"sse.{i}.{j}"][0]), (i, j)
            if f"code.{i}.{j}" not in g:
                continue
            p1 = m * ratios[i]
            p2 = m * ratios[j]
            codes, reg, fake = oracle.quantize2(x, bits, m, p1, p2)
            assert codes.tolist() == [int(v) for v in g[f"code.{i}.{j}"]]
            assert regions_of(reg, x.size).tolist() == [int(v) for v in g[f"region.{i}.{j}"]]
            want_y = np.array([float(v) for v in g[f"y.{i}.{j}"]], np.float32)
            assert fake.tobytes() == want_y.tobytes()
            y = oracle.dequantize2(codes, reg, bits, m, p1, p2, C=1, n=x.size)
            assert y.tobytes() == want_y.tobytes()
    _, reg, _ = oracle.quantize2(x, bits, m, m * ratios[0], m * ratios[1])
    assert reg.tolist() == [int(v, 16) for v in g["region_bytes.0.1"]]


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_second_breakpoint_at_m_is_the_one_breakpoint_scheme(oracle, bits):
    rng = np.random.default_rng(bits)
    x = rng.laplace(0, 0.03, (5, 301)).astype(np.float32)
    m = oracle.absmax(x)
    ratios = np.append(W.ratio_grid(16)[:-1] * np.float32(0.9), np.float32(1.0)).astype(np.float32)
    K = ratios.size
    one = oracle.search(x, bits, ratios, m=m)
    two = oracle.search2(x, bits, ratios, m)
    assert np.array_equal(two["sse64"][:, :K - 1, K - 1], one["sse64"][:, :K - 1])
    for i in (0, 5, K - 2):
        p1 = (m * ratios[i]).astype(np.float32)
        c2, r2, f2 = oracle.quantize2(x, bits, m, p1, m)
        c1, r1, f1 = oracle.quantize(x, bits, m, p1)
        assert np.array_equal(c1, c2) and f1.tobytes() == f2.tobytes()
        tail = np.unpackbits(r1, bitorder="little")[:x.size]
        assert np.array_equal(regions_of(r2, x.size), tail)
    # the pair search can only improve on the one-breakpoint search over the same grid
    assert np.all(two["err"] <= one["sse64"][:, :K - 1].min(axis=1).astype(np.float32))


def pw2_double(x, m, p1, p2, bits):
    L = 2.0 ** (bits - 1) - 1.0
    a = np.minimum(np.abs(x.astype(np.float64)), m)
    r = (a > p1).astype(int) + (a > p2).astype(int)
    z = np.choose(r, [0.0, p1, p2])
    d = np.choose(r, [p1, p2 - p1, m - p2])
    s = d / L
    with np.errstate(divide="ignore", invalid="ignore"):
        t = np.where(s > 0, (a - z) / s, 0.0)
    q = np.minimum(np.rint(t), L)
    return q, r, q * s + z, a, t


@pytest.mark.parametrize("bits,K", [(2, 8), (4, 12), (8, 8)])
def test_bruteforce_true_division_two_breakpoints(oracle, bits, K):
    rng = np.random.default_rng(50 * bits + K)
    for trial in range(8):
        n = int(rng.integers(3, 65))
        x = (rng.standard_normal(n) * 10.0 ** rng.uniform(-2, 1)).astype(np.float32)
        m = oracle.absmax(x)
        m32 = np.float32(m[0])
        ratios = W.ratio_grid(K)
        res = oracle.search2(x, bits, ratios, m)
        exact = np.full((K, K), np.inf)
        flips = 0
        for i in range(K):
            for j in range(i + 1, K):
                p1, p2 = float(m32 * ratios[i]), float(m32 * ratios[j])
                q64, r64, v64, a64, t = pw2_double(x, float(m32), p1, p2, bits)
                exact[i, j] = np.sum((v64 - a64) ** 2)
                codes, reg, _ = oracle.quantize2(x, bits, m, [np.float32(p1)], [np.float32(p2)])
                assert np.array_equal(regions_of(reg, n), r64)
                q32 = codes & (2 ** (bits - 1) - 1)
                diff = q32 != q64
                frac = np.abs(t - np.floor(t) - 0.5)
                assert np.all(frac[diff] < 1e-4), (i, j, t[diff])
                flips += int(diff.sum())
        L = 2 ** (bits - 1) - 1
        d = 2.0 * float(np.spacing(m32))
        noise = n * (float(m32) / L * d + d * d)
        iu = np.triu_indices(K, 1)
        if flips == 0:
            assert np.allclose(res["sse64"][0][iu], exact[iu], rtol=1e-6, atol=noise)
        ci, cj = int(res["idx1"][0]), int(res["idx2"][0])
        assert ci < cj
        assert exact[ci, cj] <= exact[iu].min() * (1 + 1e-6) + 2 * noise + (flips > 0) * 0.05 * exact[iu].min()
        assert res["p1"][0] == m32 * ratios[ci] and res["p2"][0] == m32 * ratios[cj]


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_half_step_bound_per_region(oracle, bits):
    rng = np.random.default_rng(bits + 70)
    L = 2 ** (bits - 1) - 1
    x = rng.laplace(0, 1.0, (4, 400)).astype(np.float32)
    m = oracle.absmax(x)
    for r1, r2 in ((0.1, 0.4), (0.25, 0.5), (0.3, 1.0), (0.05, 0.06)):
        p1 = (m * np.float32(r1)).astype(np.float32)
        p2 = (m * np.float32(r2)).astype(np.float32)
        codes, reg, fake = oracle.quantize2(x, bits, m, p1, p2)
        r = regions_of(reg, x.size).reshape(4, 400)
        a = np.abs(x)
        assert np.array_equal(r, (a > p1[:, None]).astype(int) + (a > p2[:, None]).astype(int))
        q = (codes & (2 ** (bits - 1) - 1)).reshape(4, 400)
        assert q.max() <= L
        assert np.array_equal((codes >> (bits - 1)).reshape(4, 400) == 1, x < 0)
        step = np.choose(r, [(p1 / L)[:, None], ((p2 - p1) / L)[:, None], ((m - p2) / L)[:, None]])
        v = np.abs(fake.reshape(4, 400)).astype(np.float64)
        assert np.all(np.abs(v - a) <= step / 2 + 2 * np.spacing(m)[:, None])
        y = oracle.dequantize2(codes, reg, bits, m, p1, p2, C=4, n=400)
        assert y.tobytes() == fake.tobytes()


def test_pair_order_and_degenerate_rows(oracle):
    # all |x| = m: every pair reproduces every value exactly -> the first pair (0, 1) wins
    x = np.array([[2.0, -2.0, 2.0], [0.0, 0.0, -0.0]], np.float32)
    m = oracle.absmax(x)
    res = oracle.search2(x, 4, W.ratio_grid(6), m)
    assert res["idx1"].tolist() == [0, 0] and res["idx2"].tolist() == [1, 1]
    assert res["err"].tolist() == [0.0, 0.0]
    # entries that are not a pair i < j stay 0
    y = np.array([[0.3, -1.0, 0.77, 0.1]], np.float32)
    full = oracle.search2(y, 3, W.ratio_grid(6), oracle.absmax(y))["sse64"][0]
    assert np.all(full[np.tril_indices(6)] == 0.0) and np.all(full[np.triu_indices(6, 1)] > 0.0)
    assert res["p1"].tolist()[1] == 0.0 and res["p2"].tolist()[1] == 0.0
    codes, reg, fake = oracle.quantize2(x, 4, m, res["p1"], res["p2"])
    assert codes.reshape(2, 3)[1].tolist() == [0, 0, 0] and fake[3:].tolist() == [0.0, 0.0, 0.0]
    # ragged rows give the same result as the same rows one by one
    rng = np.random.default_rng(2)
    parts = [rng.standard_normal(n).astype(np.float32) for n in (5, 33, 1, 64)]
    flat = np.concatenate(parts)
    ro = np.concatenate([[0], np.cumsum([p.size for p in parts])]).astype(np.int64)
    mm = oracle.absmax(flat, ro)
    rr = oracle.search2(flat, 3, W.ratio_grid(8), mm, row_offsets=ro)
    for c, part in enumerate(parts):
        one = oracle.search2(part, 3, W.ratio_grid(8), mm[c:c + 1])
        assert one["idx1"][0] == rr["idx1"][c] and one["idx2"][0] == rr["idx2"][c]
        assert np.array_equal(one["sse64"][0], rr["sse64"][c])


def test_two_breakpoints_reduce_the_error_on_bell_shaped_data(oracle):
    """More regions, more levels (Sec. 5.1): on Gaussian and Laplacian samples the best pair must
    beat the best single breakpoint of the same grid clearly."""
    rng = np.random.default_rng(9)
    for x in (rng.standard_normal(20000), rng.laplace(0, 1, 20000)):
        x = x.astype(np.float32).reshape(1, -1)
        m = oracle.absmax(x)
        ratios = W.ratio_grid(24)
        one = oracle.search(x, 4, ratios, m=m)["err"][0]
        two = oracle.search2(x, 4, ratios, m, want_sse=False)["err"][0]
        assert two < 0.75 * one, (one, two)
