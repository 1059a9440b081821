"""Pins the oracle's one-sided (unsigned / asymmetric range) quantizer (no GPU).

References used: a hand-worked dyadic fixture; the already pinned signed oracle (with x >= 0 and
lo = 0 the one-sided scheme at b bits is the positive half of the signed scheme at b + 1 bits);
exact shifts; a binary64 true-division restatement of Eq. 1 with z = r_l; the half-step bound.
"""
import numpy as np
import pytest

from conftest import read_golden
from paper_2002_00104_b200 import workloads as W


def bits_of(mask, total):
    return np.unpackbits(np.asarray(mask, dtype=np.uint8), bitorder="little")[:total]


def test_worked_example_unsigned_b2(oracle):
    g = read_golden("worked_example_unsigned_b2.txt")
    bits = int(g["bits"][0])
    x = np.array([float(v) for v in g["x"]], dtype=np.float32)
    lo = np.array([float(g["lo"][0])], np.float32)
    hi = np.array([float(g["hi"][0])], np.float32)
    ratios = np.array([float(v) for v in g["ratios"]], dtype=np.float32)
    res = oracle.search_u(x, bits, ratios, lo, hi)
    assert res["idx"].tolist() == [int(g["argmin"][0])]
    assert res["p"].tolist() == [float(g["p_star"][0])]
    assert res["err"].tolist() == [float(g["err_star"][0])]
    for k, p in enumerate(float(v) for v in g["p"]):
        assert res["sse64"][0, k] == float(g[f"sse.{k}"][0])
        pk = np.array([p], np.float32)
        codes, mask, fake = oracle.quantize_u(x, bits, lo, hi, pk, layout=0)
        assert codes.tolist() == [int(v) for v in g[f"code.{k}"]]
        assert bits_of(mask, x.size).tolist() == [int(v) for v in g[f"region.{k}"]]
        want_y = np.array([float(v) for v in g[f"y.{k}"]], np.float32)
        assert fake.tobytes() == want_y.tobytes()
        y = oracle.dequantize_u(codes, mask, bits, lo, hi, pk, C=1, n=x.size)
        assert y.tobytes() == want_y.tobytes()
        for xi, ci, ri, yi in zip(x, codes, bits_of(mask, x.size), want_y):
            assert oracle.elem_u(xi, lo[0], hi[0], p, bits) == (int(ci), int(ri), float(yi))
    packed, mask, _ = oracle.quantize_u(x, bits, lo, hi, np.array([3.0], np.float32), layout=1)
    assert packed.tolist() == [int(v, 16) for v in g["packed.0"]]
    assert mask.tolist() == [int(v, 16) for v in g["mask.0"]]
    y = oracle.dequantize_u(packed, mask, bits, lo, hi, np.array([3.0], np.float32), C=1,
                            n=x.size, layout=1)
    assert y.tobytes() == np.array([float(v) for v in g["y.0"]], np.float32).tobytes()


def test_minmax_rows(oracle):
    x = np.array([[1.0, -7.5, 3.0], [0.0, -0.0, 0.0], [2.0, 1.0, 1.5]], dtype=np.float32)
    lo, hi = oracle.minmax(x)
    assert lo.tolist() == [-7.5, 0.0, 1.0] and hi.tolist() == [3.0, 0.0, 2.0]
    ro = np.array([0, 1, 1, 4, 9], dtype=np.int64)      # ragged, with an empty row
    lo, hi = oracle.minmax(x.reshape(-1), ro)
    assert lo.tolist() == [1.0, 0.0, -7.5, 0.0] and hi.tolist() == [1.0, 0.0, 3.0, 2.0]
    rng = np.random.default_rng(5)
    y = rng.standard_normal((7, 33)).astype(np.float32)
    lo, hi = oracle.minmax(y)
    assert np.array_equal(lo, y.min(axis=1)) and np.array_equal(hi, y.max(axis=1))
    with pytest.raises(oracle.OracleError):
        oracle.minmax(np.array([1.0, np.inf], np.float32))


@pytest.mark.parametrize("bits", [2, 3, 4, 7])
def test_nonnegative_rows_equal_the_signed_scheme_with_one_more_bit(oracle, bits):
    """x >= 0, lo = 0, hi = max: L = 2^b - 1 is the signed scheme's L at b + 1 bits, whose sign
    bit stays 0 (Sec. 3.2: (b-1)-bit pieces plus sign; Eq. 1: unsigned domain for one-sided data)."""
    rng = np.random.default_rng(bits)
    x = np.maximum(rng.standard_normal((6, 257)), 0).astype(np.float32)
    x[:, 0] = 0.0
    lo = np.zeros(6, np.float32)
    hi = x.max(axis=1)
    ratios = W.ratio_grid(32)
    ru = oracle.search_u(x, bits, ratios, lo, hi)
    rs = oracle.search(x, bits + 1, ratios, m=hi)
    for key in ("idx", "p", "err", "sse64"):
        assert np.array_equal(ru[key], rs[key]), key
    cu, mu, fu = oracle.quantize_u(x, bits, lo, hi, ru["p"])
    cs, ms, fs = oracle.quantize(x, bits + 1, hi, ru["p"])
    assert np.array_equal(cu, cs) and np.array_equal(mu, ms) and fu.tobytes() == fs.tobytes()
    assert cu.max() <= 2 ** bits - 1
    yu = oracle.dequantize_u(cu, mu, bits, lo, hi, ru["p"], C=6, n=257)
    assert yu.tobytes() == fu.tobytes()


@pytest.mark.parametrize("shift", [16.0, -64.0])
def test_exact_shift_moves_nothing_but_the_offset(oracle, shift):
    """Dyadic data shifted by an exactly representable amount: same a = x - lo, hence the same
    codes, regions, errors and breakpoint; the delivered values move by the shift."""
    rng = np.random.default_rng(3)
    x = (rng.integers(0, 513, size=(4, 96)) / 64.0).astype(np.float32)       # k/64 in [0, 8]
    lo, hi = oracle.minmax(x)
    xs = (x + np.float32(shift)).astype(np.float32)
    assert np.array_equal(xs - np.float32(shift), x)
    los, his = oracle.minmax(xs)
    ratios = W.ratio_grid(16)
    r0 = oracle.search_u(x, 3, ratios, lo, hi)
    r1 = oracle.search_u(xs, 3, ratios, los, his)
    for key in ("idx", "p", "err", "sse64"):
        assert np.array_equal(r0[key], r1[key]), key
    c0, m0, f0 = oracle.quantize_u(x, 3, lo, hi, r0["p"])
    c1, m1, f1 = oracle.quantize_u(xs, 3, los, his, r0["p"])
    assert np.array_equal(c0, c1) and np.array_equal(m0, m1)
    # v + lo in binary32; with these magnitudes the sum is exact only up to one rounding
    assert np.allclose(f1.astype(np.float64), f0.astype(np.float64) + shift, rtol=0, atol=2 ** -17)


def pw_u_double(x, lo, hi, p, bits):
    """Eq. 1 with z = r_l per region in binary64 with a true division."""
    L = 2.0 ** bits - 1.0
    m = hi - lo
    a = np.minimum(np.maximum(x.astype(np.float64) - lo, 0.0), m)
    tail = a > p
    z = np.where(tail, p, 0.0)
    s = np.where(tail, (m - p) / L, p / L)
    with np.errstate(divide="ignore", invalid="ignore"):
        t = np.where(s > 0, (a - z) / s, 0.0)
    q = np.minimum(np.rint(t), L)
    return q, tail, q * s + z, a, t


@pytest.mark.parametrize("bits,K", [(2, 16), (4, 32), (8, 32)])
def test_bruteforce_true_division_tiny_rows(oracle, bits, K):
    rng = np.random.default_rng(100 * bits + K)
    for trial in range(10):
        n = int(rng.integers(2, 65))
        x = np.maximum(rng.standard_normal(n), -0.3).astype(np.float32) * np.float32(10.0 ** rng.uniform(-2, 1))
        x += np.float32(rng.uniform(-1, 1))
        lo, hi = oracle.minmax(x)
        m32 = np.float32(hi[0]) - np.float32(lo[0])
        ratios = W.ratio_grid(K)
        res = oracle.search_u(x, bits, ratios, lo, hi)
        p32 = (m32 * ratios).astype(np.float64)
        exact = np.empty(K)
        flips = 0
        for k in range(K):
            q64, tail64, v64, a64, t = pw_u_double(x, float(lo[0]), float(lo[0]) + float(m32), p32[k], bits)
            exact[k] = np.sum((v64 - a64) ** 2)
            codes, mask, _ = oracle.quantize_u(x, bits, lo, hi, [np.float32(p32[k])])
            tail32 = bits_of(mask, n) == 1
            # the subtraction x - lo rounds in binary32: regions and levels may differ only at
            # binary32-noise distance from a boundary or a tie
            near_p = np.abs(a64 - p32[k]) <= 4 * np.spacing(np.float32(m32))
            assert np.all((tail32 == tail64) | near_p)
            same = tail32 == tail64
            diff = (codes != q64) & same
            frac = np.abs(t - np.floor(t) - 0.5)
            assert np.all(frac[diff] < 1e-3 * max(1.0, 2.0 ** bits / 16)), (k, t[diff])
            flips += int(diff.sum()) + int((~same).sum())
        L = 2 ** bits - 1
        d = 4.0 * float(np.spacing(np.float32(max(abs(float(lo[0])), abs(float(hi[0])), float(m32)))))
        noise = n * (float(m32) / L * d + d * d)
        if flips == 0:
            assert np.allclose(res["sse64"][0], exact, rtol=1e-6, atol=noise)
        chosen = int(res["idx"][0])
        assert exact[chosen] <= exact.min() * (1 + 1e-6) + 2 * noise + (flips > 0) * exact.min() * 0.05
        assert res["p"][0] == m32 * ratios[chosen]


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_levels_regions_and_half_step_bound_unsigned(oracle, bits):
    rng = np.random.default_rng(bits + 40)
    L = 2 ** bits - 1
    x = (rng.laplace(0.5, 1.0, size=(5, 300))).astype(np.float32)
    lo, hi = oracle.minmax(x)
    m = hi - lo
    for ratio in (0.1, 0.37, 0.5, 1.0):
        p = (m * np.float32(ratio)).astype(np.float32)
        codes, mask, fake = oracle.quantize_u(x, bits, lo, hi, p)
        codes = codes.reshape(5, 300)
        tail = bits_of(mask, x.size).reshape(5, 300) == 1
        assert codes.max() <= L
        a = np.minimum(np.maximum(x - lo[:, None], 0), m[:, None]).astype(np.float32)
        assert np.array_equal(tail, a > p[:, None])
        step = np.where(tail, ((m - p) / L)[:, None], (p / L)[:, None]).astype(np.float64)
        v = fake.reshape(5, 300).astype(np.float64) - lo[:, None]
        slack = 4 * np.spacing(np.maximum(np.abs(lo), np.abs(hi)).astype(np.float32))[:, None]
        assert np.all(np.abs(v - a) <= step / 2 + slack)
        y = oracle.dequantize_u(codes.reshape(-1), mask, bits, lo, hi, p, C=5, n=300)
        assert y.tobytes() == fake.tobytes()
    # the extremes of the range are reproduced: a = 0 -> level 0, a = m -> level L of its region
    codes, mask, fake = oracle.quantize_u(x, bits, lo, hi, (m * np.float32(0.25)).astype(np.float32))
    codes = codes.reshape(5, 300)
    for c in range(5):
        assert codes[c, np.argmin(x[c])] == 0 and codes[c, np.argmax(x[c])] == L


def test_constant_and_empty_rows_unsigned(oracle):
    x = np.array([2.5, 2.5, 2.5, 1.0, 4.0], np.float32)
    ro = np.array([0, 3, 3, 5], np.int64)
    lo, hi = oracle.minmax(x, ro)
    assert lo.tolist() == [2.5, 0.0, 1.0] and hi.tolist() == [2.5, 0.0, 4.0]
    res = oracle.search_u(x, 4, W.ratio_grid(8), lo, hi, row_offsets=ro)
    assert res["idx"].tolist()[:2] == [0, 0] and res["p"].tolist()[:2] == [0.0, 0.0]
    assert res["err"].tolist()[:2] == [0.0, 0.0]
    codes, mask, fake = oracle.quantize_u(x, 4, lo, hi, res["p"], row_offsets=ro)
    assert codes[:3].tolist() == [0, 0, 0] and fake[:3].tolist() == [2.5, 2.5, 2.5]
    y = oracle.dequantize_u(codes, mask, 4, lo, hi, res["p"], row_offsets=ro)
    assert y.tobytes() == fake.tobytes()


def test_unsigned_beats_signed_on_relu_data(oracle):
    """The reason for the one-sided form: on non-negative data the sign bit is wasted, so b-bit
    unsigned levels must give about a quarter of the b-bit signed scheme's squared error
    (Eq. 2: the error of a uniform piece scales with 1 / (N - 1)^2)."""
    w = W.relu_activation(shape=(1, 16, 64, 64))
    x = w.x.reshape(1, -1)
    x = np.minimum(x, np.float32(6.0))            # keep the range tame: a clipped ReLU
    lo, hi = oracle.minmax(x)
    ratios = W.ratio_grid(64)
    for bits in (3, 4):
        eu = oracle.search_u(x, bits, ratios, lo, hi)["err"][0]
        es = oracle.search(x, bits, ratios, m=hi)["err"][0]
        ratio = es / eu
        assert 3.0 < ratio < 6.5, ratio
