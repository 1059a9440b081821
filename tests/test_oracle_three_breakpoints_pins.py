"""Pins the oracle's three-breakpoint quantizer and triple search (no GPU).

References: a hand-worked dyadic fixture; the already pinned two-breakpoint oracle (p3 = m makes
the fourth region empty); a binary64 true-division restatement; the half-step bound per region;
the ordering of the triple search.
"""
import itertools

import numpy as np
import pytest

from conftest import read_golden
from paper_2002_00104_b200 import workloads as W
from test_oracle_two_breakpoints_pins import regions_of


def test_worked_example_three_breakpoints(oracle):
    g = read_golden("worked_example_three_breakpoints_b3.txt")
    bits = int(g["bits"][0])
    x = np.array([float(v) for v in g["x"]], dtype=np.float32)
    ratios = np.array([float(v) for v in g["ratios"]], dtype=np.float32)
    m = np.array([float(g["m"][0])], np.float32)
    assert oracle.absmax(x).tolist() == m.tolist()
    res = oracle.search3(x, bits, ratios, m)
    assert res["idx"][0].tolist() == [int(v) for v in g["argmin"]]
    assert res["p"][0].tolist() == [float(v) for v in g["p_star"]]
    assert float(res["err"][0]) == float(g["err_star"][0])
    K = ratios.size
    for i, j, k in itertools.combinations(range(K), 3):
        assert res["sse64"][0, i, j, k] == float(g[f"sse.{i}.{j}.{k}"][0]), (i, j, k)
    p = (m[0] * ratios[[0, 1, 2]]).reshape(1, 3)
    codes, reg, fake = oracle.quantize3(x, bits, m, p)
    assert codes.tolist() == [int(v) for v in g["code.0.1.2"]]
    assert regions_of(reg, x.size).tolist() == [int(v) for v in g["region.0.1.2"]]
    want_y = np.array([float(v) for v in g["y.0.1.2"]], np.float32)
    assert fake.tobytes() == want_y.tobytes()
    assert reg.tolist() == [int(v, 16) for v in g["region_bytes.0.1.2"]]
    assert oracle.dequantize3(codes, reg, bits, m, p, C=1, n=x.size).tobytes() == want_y.tobytes()
    packed, reg_p, _ = oracle.quantize3(x, bits, m, p, layout=1)
    assert packed.tolist() == [int(v, 16) for v in g["packed.0.1.2"]]
    assert oracle.dequantize3(packed, reg_p, bits, m, p, C=1, n=x.size,
                              layout=1).tobytes() == want_y.tobytes()


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_third_breakpoint_at_m_is_the_two_breakpoint_scheme(oracle, bits):
    rng = np.random.default_rng(bits)
    x = rng.laplace(0, 0.03, (4, 203)).astype(np.float32)
    m = oracle.absmax(x)
    ratios = np.append(W.ratio_grid(10)[:-1] * np.float32(0.9), np.float32(1.0)).astype(np.float32)
    K = ratios.size
    two = oracle.search2(x, bits, ratios, m)
    three = oracle.search3(x, bits, ratios, m)
    for i, j in itertools.combinations(range(K - 1), 2):
        assert np.array_equal(three["sse64"][:, i, j, K - 1], two["sse64"][:, i, j]), (i, j)
    for i, j in ((0, 1), (2, 7), (K - 3, K - 2)):
        p1, p2 = (m * ratios[i]).astype(np.float32), (m * ratios[j]).astype(np.float32)
        c3, r3, f3 = oracle.quantize3(x, bits, m, np.stack([p1, p2, m], axis=1))
        c2, r2, f2 = oracle.quantize2(x, bits, m, p1, p2)
        assert np.array_equal(c2, c3) and np.array_equal(r2, r3) and f2.tobytes() == f3.tobytes()
    # the triple search can only improve on the pair search over the same grid
    iu = np.triu_indices(K - 1, 1)
    best_two = np.array([two["sse64"][c][:K - 1, :K - 1][iu].min() for c in range(4)])
    assert np.all(three["err"] <= best_two.astype(np.float32))


def pw3_double(x, m, p, bits):
    L = 2.0 ** (bits - 1) - 1.0
    a = np.minimum(np.abs(x.astype(np.float64)), m)
    r = (a > p[0]).astype(int) + (a > p[1]).astype(int) + (a > p[2]).astype(int)
    z = np.choose(r, [0.0, p[0], p[1], p[2]])
    d = np.choose(r, [p[0], p[1] - p[0], p[2] - p[1], m - p[2]])
    s = d / L
    with np.errstate(divide="ignore", invalid="ignore"):
        t = np.where(s > 0, (a - z) / s, 0.0)
    q = np.minimum(np.rint(t), L)
    return q, r, q * s + z, a, t


@pytest.mark.parametrize("bits,K", [(2, 6), (4, 8), (8, 6)])
def test_bruteforce_true_division_three_breakpoints(oracle, bits, K):
    rng = np.random.default_rng(60 * bits + K)
    for trial in range(6):
        n = int(rng.integers(3, 65))
        x = (rng.standard_normal(n) * 10.0 ** rng.uniform(-2, 1)).astype(np.float32)
        m = oracle.absmax(x)
        m32 = np.float32(m[0])
        ratios = W.ratio_grid(K)
        res = oracle.search3(x, bits, ratios, m)
        triples = list(itertools.combinations(range(K), 3))
        exact = {}
        flips = 0
        for t3 in triples:
            p = [float(m32 * ratios[i]) for i in t3]
            q64, r64, v64, a64, t = pw3_double(x, float(m32), p, bits)
            exact[t3] = np.sum((v64 - a64) ** 2)
            codes, reg, _ = oracle.quantize3(x, bits, m, np.array([p], np.float32))
            assert np.array_equal(regions_of(reg, n), r64)
            q32 = codes & (2 ** (bits - 1) - 1)
            diff = q32 != q64
            frac = np.abs(t - np.floor(t) - 0.5)
            assert np.all(frac[diff] < 1e-4), (t3, t[diff])
            flips += int(diff.sum())
        L = 2 ** (bits - 1) - 1
        d = 2.0 * float(np.spacing(m32))
        noise = n * (float(m32) / L * d + d * d)
        lowest = min(exact.values())
        if flips == 0:
            for t3 in triples:
                assert np.isclose(res["sse64"][0][t3], exact[t3], rtol=1e-6, atol=noise), t3
        chosen = tuple(int(v) for v in res["idx"][0])
        assert chosen[0] < chosen[1] < chosen[2]
        assert exact[chosen] <= lowest * (1 + 1e-6) + 2 * noise + (flips > 0) * 0.05 * lowest
        assert res["p"][0].tolist() == [float(m32 * ratios[i]) for i in chosen]


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_half_step_bound_per_region_three_breakpoints(oracle, bits):
    rng = np.random.default_rng(bits + 90)
    L = 2 ** (bits - 1) - 1
    x = rng.laplace(0, 1.0, (4, 400)).astype(np.float32)
    m = oracle.absmax(x)
    for rr in ((0.1, 0.3, 0.6), (0.25, 0.5, 0.75), (0.2, 0.4, 1.0), (0.05, 0.06, 0.07)):
        p = np.stack([(m * np.float32(r)).astype(np.float32) for r in rr], axis=1)
        codes, reg, fake = oracle.quantize3(x, bits, m, p)
        r = regions_of(reg, x.size).reshape(4, 400)
        a = np.abs(x)
        assert np.array_equal(r, sum((a > p[:, t:t + 1]).astype(int) for t in range(3)))
        assert (codes & (2 ** (bits - 1) - 1)).max() <= L
        assert np.array_equal((codes >> (bits - 1)).reshape(4, 400) == 1, x < 0)
        edges = np.concatenate([np.zeros((4, 1), np.float32), p, m[:, None]], axis=1)
        step = np.take_along_axis(np.diff(edges, axis=1) / L, r, axis=1)
        v = np.abs(fake.reshape(4, 400)).astype(np.float64)
        assert np.all(np.abs(v - a) <= step / 2 + 2 * np.spacing(m)[:, None])
        y = oracle.dequantize3(codes, reg, bits, m, p, C=4, n=400)
        assert y.tobytes() == fake.tobytes()


def test_triple_order_and_degenerate_rows(oracle):
    # all |x| = m: every triple reproduces every value exactly -> the first triple (0, 1, 2) wins
    x = np.array([[2.0, -2.0, 2.0], [0.0, 0.0, -0.0]], np.float32)
    m = oracle.absmax(x)
    res = oracle.search3(x, 4, W.ratio_grid(6), m)
    assert res["idx"].tolist() == [[0, 1, 2], [0, 1, 2]]
    assert res["err"].tolist() == [0.0, 0.0] and res["p"][1].tolist() == [0.0, 0.0, 0.0]
    # entries that are not a triple i < j < k stay 0
    y = np.array([[0.3, -1.0, 0.77, 0.1]], np.float32)
    full = oracle.search3(y, 3, W.ratio_grid(5), oracle.absmax(y))["sse64"][0]
    for i, j, k in itertools.product(range(5), repeat=3):
        assert (full[i, j, k] > 0.0) == (i < j < k), (i, j, k)
    # ragged rows give the same result as the same rows one by one
    rng = np.random.default_rng(3)
    parts = [rng.standard_normal(n).astype(np.float32) for n in (5, 33, 1, 64)]
    flat = np.concatenate(parts)
    ro = np.concatenate([[0], np.cumsum([p.size for p in parts])]).astype(np.int64)
    mm = oracle.absmax(flat, ro)
    rr = oracle.search3(flat, 3, W.ratio_grid(7), mm, row_offsets=ro)
    for c, part in enumerate(parts):
        one = oracle.search3(part, 3, W.ratio_grid(7), mm[c:c + 1])
        assert one["idx"][0].tolist() == rr["idx"][c].tolist()
        assert np.array_equal(one["sse64"][0], rr["sse64"][c])


def test_three_breakpoints_reduce_the_error_further(oracle):
    """Sec. 5.1 / Table 1: each added breakpoint lowers the error on bell-shaped data."""
    rng = np.random.default_rng(10)
    for x in (rng.standard_normal(6000), rng.laplace(0, 1, 6000)):
        x = x.astype(np.float32).reshape(1, -1)
        m = oracle.absmax(x)
        ratios = W.ratio_grid(16)
        two = oracle.search2(x, 4, ratios, m, want_sse=False)["err"][0]
        three = oracle.search3(x, 4, ratios, m, want_sse=False)["err"][0]
        assert three < 0.8 * two, (two, three)
