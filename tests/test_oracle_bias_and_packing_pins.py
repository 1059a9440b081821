"""Pins the oracle's bias correction and dense (b+1)-bit storage (no GPU).

Bias correction is pinned by its defining property (the corrected row has the mean and the centred
norm of the original row), by a hand-computed row, by exactly representable rows (xi = 1, beta = 0)
and by its behaviour under exact rescaling.  The bit stream is pinned by a hand-written example and
by a bit-by-bit reference in Python.
"""
import numpy as np
import pytest

from paper_2002_00104_b200 import workloads as W


@pytest.mark.parametrize("bits", [3, 4, 6])
def test_corrected_rows_keep_mean_and_centred_norm(oracle, bits):
    rng = np.random.default_rng(bits)
    x = (rng.laplace(0.01, 0.05, (6, 700))).astype(np.float32)
    m = oracle.absmax(x)
    p = oracle.search(x, bits, W.ratio_grid(32), m=m)["p"]
    xi, beta = oracle.bias_correction(x, bits, m, p)
    _, _, y = oracle.quantize(x, bits, m, p)
    y = y.reshape(6, 700).astype(np.float64)
    x64 = x.astype(np.float64)
    yc = xi.astype(np.float64)[:, None] * y + beta.astype(np.float64)[:, None]
    assert np.allclose(yc.mean(axis=1), x64.mean(axis=1), rtol=0, atol=3e-7 * np.abs(x64).max())
    nx = np.sqrt(((x64 - x64.mean(axis=1, keepdims=True)) ** 2).sum(axis=1))
    ny = np.sqrt(((yc - yc.mean(axis=1, keepdims=True)) ** 2).sum(axis=1))
    assert np.allclose(ny, nx, rtol=3e-7)
    # quantization shrinks or stretches rows only slightly: the folded scale stays near 1
    assert np.all(np.abs(xi - 1) < 0.2) and np.any(xi != 1)


def test_hand_computed_row(oracle):
    """b = 3 (L = 3), m = 6, p = 3: both steps are 1, so y = round-half-even(x) here:
    x = [0.25, 1, -2, 4.5, 6, -0.25, 3, 5.25] gives y = [0, 1, -2, 5, 6, -0, 3, 5] (4.5 lies in the
    tail: (4.5 - 3) / 1 = 1.5 -> 2, y = 5).  Means and centred sums are worked out below."""
    x = np.array([0.25, 1.0, -2.0, 4.5, 6.0, -0.25, 3.0, 5.25], np.float32)
    m = np.array([6.0], np.float32)
    p = np.array([3.0], np.float32)
    _, _, y = oracle.quantize(x, 3, m, p)
    want_y = np.array([0.0, 1.0, -2.0, 5.0, 6.0, -0.0, 3.0, 5.0], np.float32)
    assert y.tobytes() == want_y.tobytes()
    # mean x = 17.75 / 8, mean y = 18 / 8; centred sums by hand
    mx, my = 17.75 / 8, 18.0 / 8
    vx = sum((v - mx) ** 2 for v in x.astype(np.float64))
    vy = sum((v - my) ** 2 for v in want_y.astype(np.float64))
    xi_want = (vx / vy) ** 0.5
    xi, beta = oracle.bias_correction(x, 3, m, p)
    assert xi[0] == np.float32(xi_want)
    assert beta[0] == np.float32(mx - xi_want * my)


def test_exact_rows_need_no_correction_and_degenerate_rows(oracle):
    # every value is a level of its region: y = x, so xi = 1 and beta = 0
    x = np.array([[0.0, 1.0, -2.0, 3.0, 4.0, -5.0, 6.0, 0.0]], np.float32)
    xi, beta = oracle.bias_correction(x, 3, [6.0], [3.0])
    assert xi.tolist() == [1.0] and beta.tolist() == [0.0]
    # a constant row: no spread to match, the offset alone restores the mean
    c = np.full((1, 5), 0.3, np.float32)
    xi, beta = oracle.bias_correction(c, 3, [0.3], [0.1])
    _, _, y = oracle.quantize(c, 3, [0.3], [0.1])
    assert xi.tolist() == [1.0] and abs(float(beta[0]) - (0.3 - float(y[0]))) < 1e-7
    # empty and all-zero rows
    ro = np.array([0, 0, 4], np.int64)
    xi, beta = oracle.bias_correction(np.zeros(4, np.float32), 4, [0.0, 0.0], [0.0, 0.0], row_offsets=ro)
    assert xi.tolist() == [1.0, 1.0] and beta.tolist() == [0.0, 0.0]


def test_rescaling_by_a_power_of_two(oracle):
    rng = np.random.default_rng(4)
    x = rng.standard_normal((3, 200)).astype(np.float32)
    m = oracle.absmax(x)
    p = (m * np.float32(0.3)).astype(np.float32)
    xi1, b1 = oracle.bias_correction(x, 4, m, p)
    xi2, b2 = oracle.bias_correction(x * np.float32(4), 4, m * np.float32(4), p * np.float32(4))
    assert np.array_equal(xi1, xi2) and np.array_equal(b1 * np.float32(4), b2)


def test_dequantize_with_correction_applies_scale_then_offset(oracle):
    rng = np.random.default_rng(6)
    x = rng.laplace(0, 0.1, (4, 99)).astype(np.float32)
    m = oracle.absmax(x)
    p = (m * np.float32(0.25)).astype(np.float32)
    xi, beta = oracle.bias_correction(x, 4, m, p)
    codes, mask, y = oracle.quantize(x, 4, m, p, layout=1)
    got = oracle.dequantize_bc(codes, mask, 4, m, p, xi, beta, C=4, n=99, layout=1)
    want = (xi[:, None] * y.reshape(4, 99)).astype(np.float32) + beta[:, None]
    assert got.tobytes() == want.astype(np.float32).reshape(-1).tobytes()


# --------------------------------------------------------------------------------- bit stream
def test_dense_stream_hand_example(oracle):
    # b = 3: four bits per value = code | region << 3; two values per byte, first in the low nibble
    codes = np.array([5, 2, 7, 0, 1], np.uint8)
    mask = np.array([0b10110], np.uint8)              # regions 0 1 1 0 1
    s = oracle.pack_dense(codes, mask, 3)
    assert s.tolist() == [0x5 | (0xA << 4), 0xF | (0x0 << 4), 0x9]
    # b = 6: seven bits per value, crossing byte borders: fields 0x41, 0x3F, 0x00 | region
    codes = np.array([0x01, 0x3F, 0x00], np.uint8)
    mask = np.array([0b101], np.uint8)
    s = oracle.pack_dense(codes, mask, 6)
    fields = [0x41, 0x3F, 0x40]
    word = fields[0] | (fields[1] << 7) | (fields[2] << 14)
    assert s.tolist() == [word & 0xFF, (word >> 8) & 0xFF, (word >> 16) & 0xFF]


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8])
def test_dense_stream_against_a_bitwise_reference_and_back(oracle, bits):
    rng = np.random.default_rng(bits)
    total = 1003
    codes = rng.integers(0, 2 ** bits, total).astype(np.uint8)
    reg = rng.integers(0, 2, total).astype(np.uint8)
    mask = np.packbits(reg, bitorder="little")
    s = oracle.pack_dense(codes, mask, bits)
    ref_bits = np.zeros(((total * (bits + 1) + 7) // 8) * 8, np.uint8)
    for i in range(total):
        field = int(codes[i]) | (int(reg[i]) << bits)
        for k in range(bits + 1):
            ref_bits[i * (bits + 1) + k] = (field >> k) & 1
    assert np.array_equal(s, np.packbits(ref_bits, bitorder="little"))
    c2, m2 = oracle.unpack_dense(s, total, bits)
    assert np.array_equal(c2, codes) and np.array_equal(m2, mask)
