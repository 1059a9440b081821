"""GPU parity of the one-sided (unsigned / asymmetric range) calls against the CPU oracle."""
import numpy as np
import pytest
import torch

from gpu_util import check_search, dev
from paper_2002_00104_b200 import workloads as W

pytestmark = [pytest.mark.gpu,
              pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]


@pytest.fixture(scope="module")
def pwlq():
    from paper_2002_00104_b200 import pwlq as _p
    _p.load_library()
    return _p


def np_(t):
    return None if t is None else t.cpu().numpy()


def relu_like(rng, shape, offset=0.0):
    """Non-negative bell-shaped data with a long tail, optionally moved off zero."""
    x = np.maximum(rng.standard_normal(shape), 0.0) + 0.05 * np.abs(rng.standard_cauchy(shape))
    return (np.minimum(x, 40.0) + offset).astype(np.float32)


# ------------------------------------------------------------------------------------ min / max
@pytest.mark.parametrize("C,n", [(1, 1), (3, 9), (5, 147), (64, 64), (7, 4607), (2, 100003), (1, 1 << 20)])
def test_minmax_dense(pwlq, oracle, C, n):
    rng = np.random.default_rng(C * 1000 + n)
    x = (rng.laplace(0, 0.02, (C, n)) + rng.uniform(-1, 1, (C, 1))).astype(np.float32)
    lo, hi = pwlq.minmax(dev(x))
    olo, ohi = oracle.minmax(x)
    assert np.array_equal(np_(lo), olo) and np.array_equal(np_(hi), ohi)
    assert pwlq.device_status() == 0


def test_minmax_ragged_unaligned_empty_rows(pwlq, oracle):
    w = W.small_mixed(seed=21)
    x = w.x + np.float32(0.25)
    lo, hi = pwlq.minmax(dev(x), row_offsets=dev(w.row_offsets))
    olo, ohi = oracle.minmax(x, w.row_offsets)
    assert np.array_equal(np_(lo), olo) and np.array_equal(np_(hi), ohi)
    buf = dev(np.concatenate([[0.0], x]).astype(np.float32))      # base 4 bytes off 16
    lo2, hi2 = pwlq.minmax(buf[1:], row_offsets=dev(w.row_offsets))
    assert np.array_equal(np_(lo2), olo) and np.array_equal(np_(hi2), ohi)
    ro = np.array([0, 0, 3, 3, 3, 10, 10], np.int64)               # empty rows everywhere
    y = np.array([-1.5, 2.0, 0.5, -0.0, 0.0, -3.0, 7.0, 7.0, 1.0, -2.5], np.float32)
    lo, hi = pwlq.minmax(dev(y), row_offsets=dev(ro))
    olo, ohi = oracle.minmax(y, ro)
    assert np.array_equal(np_(lo), olo) and np.array_equal(np_(hi), ohi)
    assert np_(lo).tolist() == [0.0, -1.5, 0.0, 0.0, -3.0, 0.0]


# --------------------------------------------------------------------------------------- search
def run_search_u(pwlq, x, bits, ratios, lo, hi, row_offsets=None, max_n=None):
    out = pwlq.search_unsigned(dev(x), bits, dev(ratios), dev(lo), dev(hi),
                               row_offsets=None if row_offsets is None else dev(row_offsets),
                               max_n=max_n, want_sse=True)
    torch.cuda.synchronize()
    return {k: np_(out[k]) for k in ("p", "err", "idx", "sse")}, pwlq.search_status(out["workspace"])


@pytest.mark.parametrize("bits,K", [(2, 16), (3, 100), (4, 256), (8, 64)])
@pytest.mark.parametrize("C,n", [(6, 9), (4, 256), (3, 4097), (1, 20000)])
def test_search_unsigned_dense(pwlq, oracle, bits, K, C, n):
    rng = np.random.default_rng(bits * 100 + K + n)
    x = relu_like(rng, (C, n), offset=float(rng.uniform(-0.5, 0.5)))
    lo, hi = oracle.minmax(x)
    ratios = W.ratio_grid(K)
    got, status = run_search_u(pwlq, x, bits, ratios, lo, hi)
    assert status == 0
    ora = oracle.search_u(x, bits, ratios, lo, hi)
    check_search(got, ora, ratios, (hi - lo).astype(np.float32), n)


def test_search_unsigned_rows_of_a_hundred_values_at_eight_bits(pwlq, oracle):
    """Many levels, few values: 255 levels per piece over rows of 65 .. 200 values.  Here a
    single value that lands on the other of two neighbouring levels shows in the row's sum at the
    1e-5 level, so the level has to be decided as Eq. 3 is evaluated operation by operation: the
    product u * L / range rounded first, then rounded to the nearest level.  (A product that rounds
    to an exact tie, x.5, while its unrounded value does not, goes to the other level when product
    and rounding are fused; a randomized run met that case in a row of 116 values.)"""
    rng = np.random.default_rng(424201)
    lens = rng.integers(65, 201, 3000).astype(np.int64)
    row_offsets = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    x = (np.maximum(rng.standard_normal(int(lens.sum())), 0) + rng.uniform(-0.5, 0.5)).astype(np.float32)
    lo, hi = oracle.minmax(x, row_offsets)
    ratios = W.ratio_grid(64)
    got, status = run_search_u(pwlq, x, 8, ratios, lo, hi, row_offsets=row_offsets,
                               max_n=int(lens.max()))
    assert status == 0
    ora = oracle.search_u(x, 8, ratios, lo, hi, row_offsets=row_offsets)
    check_search(got, ora, ratios, (hi - lo).astype(np.float32), lens)


def test_search_unsigned_ragged_with_given_ranges(pwlq, oracle):
    w = W.small_mixed(seed=5, bits=4, K=64)
    x = np.abs(w.x).astype(np.float32)
    n_rows = np.diff(w.row_offsets)
    lo, hi = oracle.minmax(x, w.row_offsets)
    lo = (lo * np.float32(1.5)).astype(np.float32)     # ranges narrower than the data: values clamp
    hi = (hi * np.float32(0.75)).astype(np.float32)
    hi = np.maximum(hi, lo)
    ratios = W.ratio_grid(64)
    got, status = run_search_u(pwlq, x, 4, ratios, lo, hi, row_offsets=w.row_offsets,
                               max_n=int(n_rows.max()))
    assert status == 0
    ora = oracle.search_u(x, 4, ratios, lo, hi, row_offsets=w.row_offsets)
    check_search(got, ora, ratios, (hi - lo).astype(np.float32), n_rows)


def test_search_unsigned_matches_signed_one_more_bit(pwlq):
    """Non-negative data, lo = 0: the one-sided search at b bits is the signed search at b + 1."""
    rng = np.random.default_rng(8)
    x = relu_like(rng, (5, 3000))
    x[:, 0] = 0.0
    xd = dev(x)
    lo, hi = pwlq.minmax(xd)
    assert np_(lo).tolist() == [0.0] * 5
    ratios = dev(W.ratio_grid(128))
    u = pwlq.search_unsigned(xd, 3, ratios, lo, hi, want_sse=True)
    s = pwlq.search(xd, 4, ratios, m=hi, want_sse=True)
    for k in ("p", "err", "idx", "sse"):
        assert torch.equal(u[k], s[k]), k


# ------------------------------------------------------------------------- quantize / dequantize
@pytest.mark.parametrize("bits,layout", [(2, 1), (4, 1), (4, 0), (6, 1), (8, 0)])
@pytest.mark.parametrize("C,n", [(1, 7), (5, 147), (3, 4096), (2, 9001), (300, 27)])
def test_quantize_dequantize_unsigned_dense(pwlq, oracle, bits, layout, C, n):
    rng = np.random.default_rng(bits + 10 * layout + n)
    x = relu_like(rng, (C, n), offset=float(rng.uniform(-2, 2)))
    lo, hi = oracle.minmax(x)
    if C > 1:
        lo[1] = hi[1]                                  # a constant range: code 0, y = lo
    p = ((hi - lo) * rng.uniform(0.05, 1.0, C)).astype(np.float32)
    codes, mask, fake = pwlq.quantize_unsigned(dev(x), bits, dev(lo), dev(hi), dev(p),
                                               layout=layout, want_fake=True)
    oc, om, of = oracle.quantize_u(x, bits, lo, hi, p, layout=layout)
    assert np.array_equal(np_(codes), oc)
    assert np.array_equal(np_(mask), om)
    assert np_(fake).tobytes() == of.tobytes()
    y = pwlq.dequantize_unsigned(codes, mask, bits, dev(lo), dev(hi), dev(p), C=C, n=n,
                                 layout=layout)
    assert np_(y).tobytes() == oracle.dequantize_u(oc, om, bits, lo, hi, p, C=C, n=n,
                                                   layout=layout).tobytes()
    assert np_(y).tobytes() == of.tobytes()
    assert pwlq.device_status() == 0


@pytest.mark.parametrize("bits,layout", [(3, 1), (8, 0)])
def test_quantize_dequantize_unsigned_ragged(pwlq, oracle, bits, layout):
    w = W.small_mixed(seed=13)
    x = (np.abs(w.x) - np.float32(0.01)).astype(np.float32)
    ro = w.row_offsets
    lo, hi = oracle.minmax(x, ro)
    p = ((hi - lo) * np.float32(0.3)).astype(np.float32)
    codes, mask, fake = pwlq.quantize_unsigned(dev(x), bits, dev(lo), dev(hi), dev(p),
                                               layout=layout, row_offsets=dev(ro), want_fake=True)
    oc, om, of = oracle.quantize_u(x, bits, lo, hi, p, layout=layout, row_offsets=ro)
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(mask), om)
    assert np_(fake).tobytes() == of.tobytes()
    y = pwlq.dequantize_unsigned(codes, mask, bits, dev(lo), dev(hi), dev(p), layout=layout,
                                 row_offsets=dev(ro))
    assert np_(y).tobytes() == of.tobytes()


def test_whole_unsigned_path_on_an_activation_tensor(pwlq, oracle):
    """min/max -> search -> quantize -> dequantize on a ReLU-like tensor of a few tiles, every step
    on the device, against the oracle run the same way."""
    w = W.relu_activation(shape=(1, 8, 56, 56))
    x = w.x
    xd = dev(x).view(1, -1)
    ratios = W.ratio_grid(256)
    lo, hi = pwlq.minmax(xd)
    out = pwlq.search_unsigned(xd, 4, dev(ratios), lo, hi, want_sse=True)
    codes, mask, fake = pwlq.quantize_unsigned(xd, 4, lo, hi, out["p"], layout=1, want_fake=True)
    y = pwlq.dequantize_unsigned(codes, mask, 4, lo, hi, out["p"], C=1, n=x.size, layout=1)
    torch.cuda.synchronize()
    olo, ohi = oracle.minmax(x)
    assert np.array_equal(np_(lo), olo) and np.array_equal(np_(hi), ohi)
    ora = oracle.search_u(x, 4, ratios, olo, ohi)
    got = {k: np_(out[k]) for k in ("p", "err", "idx", "sse")}
    check_search(got, ora, ratios, (ohi - olo).astype(np.float32), x.size)
    oc, om, of = oracle.quantize_u(x, 4, olo, ohi, got["p"], layout=1)
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(mask), om)
    assert np_(fake).tobytes() == of.tobytes() and np_(y).tobytes() == of.tobytes()
    assert pwlq.device_status() == 0


def test_unsigned_argument_errors(pwlq):
    x = torch.zeros(4, 8, device="cuda")
    lo, hi = pwlq.minmax(x)
    with pytest.raises(pwlq.PwlqError):
        pwlq.minmax(x, out=(lo, lo))
    with pytest.raises(pwlq.PwlqError):
        pwlq.search_unsigned(x, 9, dev(W.ratio_grid(4)), lo, hi)
    with pytest.raises(pwlq.PwlqError):
        pwlq.search_unsigned(x, 4, dev(W.ratio_grid(4)), None, hi)
    with pytest.raises(pwlq.PwlqError):
        pwlq.quantize_unsigned(x, 4, None, hi, hi)


@pytest.mark.parametrize("ragged", [False, True])
def test_encode_host_unsigned_matches_oracle(pwlq, oracle, ragged):
    """The one-sided form of the host-buffer entry point: min/max, search, quantize and
    dequantize from pinned host buffers, against the oracle run step by step."""
    rng = np.random.default_rng(77)
    if ragged:
        w = W.small_mixed(seed=29, bits=4, K=64)
        x = (np.abs(w.x) + np.float32(0.25)).astype(np.float32)
        ro, C = w.row_offsets, w.C
    else:
        x = relu_like(rng, (9, 500), offset=-0.5).reshape(-1)
        ro, C = None, 9
    total = x.size
    max_n = int(np.diff(ro).max()) if ragged else 500
    ratios = W.ratio_grid(64)
    hx = torch.from_numpy(x).pin_memory()
    hro = torch.from_numpy(ro).pin_memory() if ragged else None
    f32 = lambda n: torch.empty(n, dtype=torch.float32).pin_memory()
    out = {"lo": f32(C), "hi": f32(C), "p": f32(C), "err": f32(C),
           "idx": torch.empty(C, dtype=torch.int32).pin_memory(),
           "codes": torch.empty((total + 1) // 2, dtype=torch.uint8).pin_memory(),
           "mask": torch.empty((total + 7) // 8, dtype=torch.uint8).pin_memory()}
    scratch = torch.empty(pwlq.encode_host_scratch_bytes(C, total, max_n, 64), dtype=torch.uint8,
                          device="cuda")
    pwlq.encode_host_unsigned(hx, hro, C, max_n, 4, torch.from_numpy(ratios).pin_memory(), out,
                              pwlq.CODES_PACKED, scratch)
    torch.cuda.synchronize()
    xo = x if ragged else x.reshape(C, -1)
    olo, ohi = oracle.minmax(xo, ro)
    assert np.array_equal(out["lo"].numpy(), olo) and np.array_equal(out["hi"].numpy(), ohi)
    ora = oracle.search_u(xo, 4, ratios, olo, ohi, row_offsets=ro)
    rows = np.arange(C)
    gi = out["idx"].numpy()
    gap = np.abs(ora["sse64"][rows, gi] - ora["sse64"][rows, ora["idx"]])
    assert np.all(gap <= 1e-5 * ora["sse64"][rows, ora["idx"]] + 1e-30)
    oc, ok, _ = oracle.quantize_u(xo, 4, olo, ohi, out["p"].numpy(), layout=1, row_offsets=ro)
    assert np.array_equal(out["codes"].numpy(), oc) and np.array_equal(out["mask"].numpy(), ok)
    assert pwlq.device_status() == 0


@pytest.mark.parametrize("bits", [2, 3])
def test_search_unsigned_short_rows_whose_values_mostly_sit_on_levels(pwlq, oracle, bits):
    """Thousands of rows of 5 ... 31 values of a ReLU output moved off zero: most values of a row
    equal its lower bound (error 0 under every candidate), so a sum is carried by a few small
    errors and shows any rounding the search adds to the operation-by-operation sequence."""
    rng = np.random.default_rng(40 + bits)
    lens = rng.integers(5, 32, 6000).astype(np.int64)
    ro = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    total = int(ro[-1])
    off = np.repeat(rng.uniform(-0.5, 0.5, lens.size), lens)
    x = (np.maximum(rng.standard_normal(total), 0.0) + off).astype(np.float32)
    lo, hi = oracle.minmax(x, ro)
    ratios = W.ratio_grid(64)
    got, status = run_search_u(pwlq, x, bits, ratios, lo, hi, row_offsets=ro, max_n=int(lens.max()))
    assert status == 0
    ora = oracle.search_u(x, bits, ratios, lo, hi, row_offsets=ro)
    check_search(got, ora, ratios, (hi - lo).astype(np.float32), lens)
