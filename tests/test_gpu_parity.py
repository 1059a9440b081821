"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element."""
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


def run_search(pwlq, x, bits, ratios, row_offsets=None, max_n=None, m=None):
    out = pwlq.search(dev(x), bits, dev(ratios), m=None if m is None else dev(m),
                      row_offsets=None if row_offsets is None else dev(row_offsets),
                      max_n=max_n, want_sse=True)
    torch.cuda.synchronize()
    return {k: np_(out[k]) for k in ("p", "err", "idx", "sse")}, pwlq.search_status(out["workspace"])


# ------------------------------------------------------------------------------------ abs-max
@pytest.mark.parametrize("C,n", [(1, 1), (3, 9), (5, 147), (64, 64), (7, 4607), (2, 100003), (1, 1 << 20)])
def test_absmax_dense(pwlq, oracle, C, n):
    rng = np.random.default_rng(C * 1000 + n)
    x = rng.laplace(0, 0.02, (C, n)).astype(np.float32)
    x[0, 0] = -x.max() * 3 if n > 1 else x[0, 0]
    m = np_(pwlq.absmax(dev(x)))
    assert np.array_equal(m, oracle.absmax(x))


def test_absmax_ragged_and_unaligned(pwlq, oracle):
    w = W.small_mixed(seed=11)
    m = np_(pwlq.absmax(dev(w.x), row_offsets=dev(w.row_offsets)))
    assert np.array_equal(m, oracle.absmax(w.x, w.row_offsets))
    # base pointer 4 bytes off a 16-byte boundary: vector loads must not be used
    buf = dev(np.concatenate([[0.0], w.x]).astype(np.float32))
    m2 = np_(pwlq.absmax(buf[1:], row_offsets=dev(w.row_offsets)))
    assert np.array_equal(m2, m)
    z = np.zeros((4, 33), dtype=np.float32)
    z[2, 5] = -0.0
    assert np.array_equal(np_(pwlq.absmax(dev(z))), np.zeros(4, np.float32))


# ------------------------------------------------------------------------- quantize / dequantize
def canary(nbytes, dtype=torch.uint8):
    """Output buffer with a guard band on both sides."""
    pad = 64
    buf = torch.full((nbytes + 2 * pad,), 0xA5, dtype=torch.uint8, device="cuda")
    return buf, buf[pad:pad + nbytes]


def guards_intact(buf, nbytes):
    b = buf.cpu().numpy()
    return np.all(b[:64] == 0xA5) and np.all(b[64 + nbytes:] == 0xA5)


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 8])
@pytest.mark.parametrize("layout", [0, 1])
def test_quantize_dequantize_ragged_bit_exact(pwlq, oracle, bits, layout):
    w = W.small_mixed(seed=20 + bits, bits=bits)
    ratios = W.ratio_grid(16)
    ora = oracle.search(w.x, bits, ratios, row_offsets=w.row_offsets)
    m = oracle.absmax(w.x, w.row_offsets)
    p = ora["p"]
    oc, om, of = oracle.quantize(w.x, bits, m, p, layout=layout, row_offsets=w.row_offsets)
    total = w.total
    cbuf, codes = canary(pwlq.code_bytes(total, bits, layout))
    mbuf, mask = canary((total + 7) // 8)
    fbuf, fake8 = canary(total * 4)
    fake = fake8.view(torch.float32)
    pwlq.quantize(dev(w.x), bits, dev(m), dev(p), layout=layout, row_offsets=dev(w.row_offsets),
                  out=(codes, mask, fake))
    torch.cuda.synchronize()
    assert np.array_equal(np_(codes), oc)
    assert np.array_equal(np_(mask), om)
    assert np_(fake).tobytes() == of.tobytes()
    assert guards_intact(cbuf, codes.numel()) and guards_intact(mbuf, mask.numel())
    assert guards_intact(fbuf, total * 4)
    ybuf, y8 = canary(total * 4)
    y = y8.view(torch.float32)
    pwlq.dequantize(codes, mask, bits, dev(m), dev(p), layout=layout,
                    row_offsets=dev(w.row_offsets), out=y)
    torch.cuda.synchronize()
    assert np_(y).tobytes() == of.tobytes()
    assert guards_intact(ybuf, total * 4)


@pytest.mark.parametrize("C,n,bits,layout", [(1, 1, 4, 1), (3, 9, 3, 1), (5, 147, 4, 1), (4, 4607, 8, 0),
                                             (2, 100003, 4, 1), (64, 64, 6, 1), (16, 4096, 3, 1)])
def test_quantize_dequantize_dense_bit_exact(pwlq, oracle, C, n, bits, layout):
    rng = np.random.default_rng(C + n + bits)
    x = (rng.standard_normal((C, n)) * 0.05).astype(np.float32)
    if n > 4:
        x[0, :3] = [0.0, -0.0, -1e-30]
    m = oracle.absmax(x)
    p = (m * rng.uniform(0.05, 1.0, C).astype(np.float32)).astype(np.float32)
    if C > 1:
        p[-1] = m[-1]                                # p = m: empty tail
    oc, om, of = oracle.quantize(x, bits, m, p, layout=layout)
    codes, mask, fake = pwlq.quantize(dev(x), bits, dev(m), dev(p), layout=layout, want_fake=True)
    y = pwlq.dequantize(codes, mask, bits, dev(m), dev(p), C=C, n=n, layout=layout)
    torch.cuda.synchronize()
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(mask), om)
    assert np_(fake).tobytes() == of.tobytes() and np_(y).tobytes() == of.tobytes()
    assert np.array_equal(np_(y), oracle.dequantize(oc, om, bits, m, p, C=C, n=n, layout=layout))


def test_quantize_worked_example(pwlq):
    from conftest import read_golden
    g = read_golden("worked_example_b3.txt")
    x = np.array([float(v) for v in g["x"]], dtype=np.float32)[None]
    m = np.array([12.0], np.float32)
    for k, p in enumerate(float(v) for v in g["p"]):
        codes, mask, fake = pwlq.quantize(dev(x), 3, dev(m), dev(np.array([p], np.float32)),
                                          want_fake=True)
        assert np_(codes).tolist() == [int(v) for v in g[f"code.{k}"]]
        bits_ = np.unpackbits(np_(mask), bitorder="little")[:16]
        assert bits_.tolist() == [int(v) for v in g[f"region.{k}"]]
        assert np_(fake).tobytes() == np.array([float(v) for v in g[f"y.{k}"]], np.float32).tobytes()
    out, _ = run_search(pwlq, x, 3, np.array([float(v) for v in g["ratios"]], np.float32))
    assert out["idx"].tolist() == [1] and out["p"].tolist() == [6.0]
    assert out["sse"][0].tolist() == [float(g[f"sse.{k}"][0]) for k in range(4)]


def test_zero_rows_quantize_to_zero(pwlq, oracle):
    x = np.zeros((3, 40), dtype=np.float32)
    x[1] = np.linspace(-1, 1, 40)
    m = oracle.absmax(x)
    p = np.array([0.0, 0.25, 0.0], np.float32)
    oc, om, of = oracle.quantize(x, 4, m, p, layout=1)
    codes, mask, fake = pwlq.quantize(dev(x), 4, dev(m), dev(p), layout=1, want_fake=True)
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(mask), om)
    assert np_(fake).tobytes() == of.tobytes()


# ------------------------------------------------------------------------------------- search
@pytest.mark.parametrize("bits,K", [(4, 64), (3, 100), (4, 256), (8, 256), (2, 33), (6, 1024), (4, 1)])
def test_search_ragged_small(pwlq, oracle, bits, K):
    w = W.small_mixed(seed=bits * 7 + K, bits=bits, K=K)
    ratios = W.ratio_grid(K)
    ora = oracle.search(w.x, bits, ratios, row_offsets=w.row_offsets)
    gpu, status = run_search(pwlq, w.x, bits, ratios, row_offsets=w.row_offsets,
                             max_n=int(np.diff(w.row_offsets).max()))
    assert status == 0
    m = oracle.absmax(w.x, w.row_offsets)
    check_search(gpu, ora, ratios, m, np.diff(w.row_offsets))


@pytest.mark.parametrize("C,n,bits,K", [(1, 36864, 4, 100), (3, 20001, 4, 64), (2, 8192, 3, 256),
                                        (5, 8193, 4, 40), (40, 147, 4, 256), (300, 9, 3, 256)])
def test_search_dense_tiles_and_tails(pwlq, oracle, C, n, bits, K):
    rng = np.random.default_rng(C * 31 + n)
    x = rng.laplace(0, 0.02, (C, n)).astype(np.float32)
    ratios = W.ratio_grid(K)
    ora = oracle.search(x, bits, ratios)
    gpu, status = run_search(pwlq, x, bits, ratios)
    assert status == 0
    check_search(gpu, ora, ratios, oracle.absmax(x), n)


@pytest.mark.parametrize("n", [1, 2, 9, 31, 32, 33, 63, 64, 65])
@pytest.mark.parametrize("bits,K", [(3, 256), (4, 100), (8, 300), (2, 1), (4, 1024)])
def test_search_tiny_rows(pwlq, oracle, n, bits, K):
    """Rows around the limit of the one-warp-per-row kernel (64 values), with candidate counts that
    are not multiples of its batch, bit-widths on both sides of the fused / unfused switch, a zero
    row and an exact-tie row."""
    rng = np.random.default_rng(n * 100 + K)
    x = (rng.laplace(0, 0.02, (37, n)) * 10.0 ** rng.uniform(-2, 1, (37, 1))).astype(np.float32)
    x[5] = 0.0
    x[6] = np.float32(0.75) * np.where(np.arange(n) % 2, -1, 1)      # all |x| = m
    ratios = W.ratio_grid(K)
    ora = oracle.search(x, bits, ratios)
    gpu, status = run_search(pwlq, x, bits, ratios)
    assert status == 0
    check_search(gpu, ora, ratios, oracle.absmax(x), n)
    assert gpu["idx"][5] == 0 and gpu["p"][5] == 0.0 and gpu["err"][5] == 0.0


def test_search_tiny_rows_unsorted_grid_and_ties(pwlq, oracle):
    rng = np.random.default_rng(8)
    x = rng.standard_normal((50, 9)).astype(np.float32)
    ratios = np.array([0.5, 0.2, 0.2, 0.9, 0.35, 1.0, 0.05, 0.2], dtype=np.float32)
    ora = oracle.search(x, 4, ratios)
    gpu, _ = run_search(pwlq, x, 4, ratios)
    check_search(gpu, ora, ratios, oracle.absmax(x), 9)
    assert np.all(gpu["idx"] != 2) and np.all(gpu["idx"] != 7)        # duplicates: lowest index wins
    assert np.array_equal(gpu["sse"][:, 1], gpu["sse"][:, 2])


def test_search_with_given_range_and_unsorted_grid(pwlq, oracle):
    rng = np.random.default_rng(77)
    x = rng.standard_normal((6, 700)).astype(np.float32)
    m = (oracle.absmax(x) * np.float32(1.25)).astype(np.float32)      # caller-chosen wider range
    ratios = np.array([0.5, 0.2, 0.2, 0.9, 0.35, 1.0, 0.05], dtype=np.float32)
    ora = oracle.search(x, 4, ratios, m=m)
    gpu, _ = run_search(pwlq, x, 4, ratios, m=m)
    check_search(gpu, ora, ratios, m, 700)


def test_search_ties_take_lowest_index(pwlq):
    x = np.array([[2.5, -2.5, 2.5, 2.5], [0.0, 0.0, 0.0, 0.0]], dtype=np.float32)
    gpu, status = run_search(pwlq, x, 4, W.ratio_grid(10))
    assert gpu["idx"].tolist() == [0, 0] and gpu["err"].tolist() == [0.0, 0.0]
    assert gpu["p"].tolist() == [np.float32(2.5) * W.ratio_grid(10)[0], 0.0] and status == 0
    rng = np.random.default_rng(5)
    x = rng.laplace(0, 1, (1, 300)).astype(np.float32)
    ratios = np.array([0.5, 0.2, 0.2, 0.9, 0.2], dtype=np.float32)
    gpu, _ = run_search(pwlq, x, 4, ratios)
    assert gpu["idx"].tolist() == [1]
    assert gpu["sse"][0, 1] == gpu["sse"][0, 2] == gpu["sse"][0, 4]


def test_search_reports_nonfinite_range(pwlq):
    x = np.ones((3, 50), dtype=np.float32)
    x[1, 7] = np.inf
    gpu, status = run_search(pwlq, x, 4, W.ratio_grid(8))
    assert status == 1 << pwlq.ERR_NONFINITE
    assert gpu["idx"].tolist() == [0, 0, 0] and gpu["p"][1] == 0.0


def test_search_is_reproducible(pwlq):
    w = W.small_mixed(seed=1, K=256)
    ratios = W.ratio_grid(256)
    a, _ = run_search(pwlq, w.x, 4, ratios, row_offsets=w.row_offsets, max_n=9001)
    b, _ = run_search(pwlq, w.x, 4, ratios, row_offsets=w.row_offsets, max_n=9001)
    assert all(a[k].tobytes() == b[k].tobytes() for k in a)


# ---------------------------------------------------------------------- argument errors (host)
def test_argument_errors_launch_nothing(pwlq):
    x = dev(np.ones((2, 8), np.float32))
    r = dev(W.ratio_grid(4))
    with pytest.raises(pwlq.PwlqError) as e:
        pwlq.search(x, 1, r)
    assert e.value.status == pwlq.ERR_INVALID_ARG
    with pytest.raises(pwlq.PwlqError) as e:
        pwlq.search(x, 4, r, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == pwlq.ERR_WORKSPACE
    with pytest.raises(pwlq.PwlqError) as e:
        pwlq.search(x, 4, dev(W.ratio_grid(pwlq.MAX_K + 1)))
    assert e.value.status == pwlq.ERR_UNSUPPORTED
    torch.cuda.synchronize()


def test_no_bounded_wait_expired(pwlq):
    """Runs after the parity tests of this file: none of their kernels gave up on a wait."""
    assert pwlq.device_status() == 0


# ------------------------------------------------------------------ awkward layouts, host entry
def awkward_rows(seed=3):
    """Ragged rows with empty rows, single values, lengths that straddle every vector width, one
    all-zero row and one row longer than a search tile."""
    lengths = [0, 1, 0, 3, 7, 8, 9, 0, 15, 16, 17, 31, 33, 100, 0, 255, 257, 1000, 4097, 8193, 5, 0]
    rng = np.random.default_rng(seed)
    parts = [rng.laplace(0, 0.03, n).astype(np.float32) for n in lengths]
    parts[13][:] = 0.0
    ro = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
    return np.concatenate(parts), ro


@pytest.mark.parametrize("misalign", [0, 1, 2, 3])
@pytest.mark.parametrize("bits,layout", [(4, 1), (8, 0)])
def test_whole_path_on_awkward_rows_and_unaligned_buffers(pwlq, oracle, misalign, bits, layout):
    """Empty rows, tiny rows, a ragged tail, and every buffer shifted off its natural vector
    alignment by `misalign` elements: the vector and bulk-copy fast paths must step aside."""
    x, ro = awkward_rows()
    total = x.size
    ratios = W.ratio_grid(32)
    xb = dev(np.concatenate([np.zeros(misalign, np.float32), x]))[misalign:]
    m = pwlq.absmax(xb, row_offsets=dev(ro))
    om = oracle.absmax(x, ro)
    assert np.array_equal(np_(m), om)
    s = pwlq.search(xb, bits, dev(ratios), m=m, row_offsets=dev(ro), max_n=8193, want_sse=True)
    ora = oracle.search(x, bits, ratios, row_offsets=ro)
    check_search({k: np_(s[k]) for k in ("p", "err", "idx", "sse")}, ora, ratios, om, np.diff(ro))
    p = s["p"]
    nbytes = pwlq.code_bytes(total, bits, layout)
    cbuf = torch.zeros(nbytes + 16, dtype=torch.uint8, device="cuda")
    mbuf = torch.zeros((total + 7) // 8 + 16, dtype=torch.uint8, device="cuda")
    fbuf = torch.zeros(total + 16, dtype=torch.float32, device="cuda")
    codes, mask, fake = cbuf[misalign:misalign + nbytes], mbuf[misalign:misalign + (total + 7) // 8], \
        fbuf[misalign:misalign + total]
    pwlq.quantize(xb, bits, m, p, layout=layout, row_offsets=dev(ro), out=(codes, mask, fake))
    oc, ok, of = oracle.quantize(x, bits, om, np_(p), layout=layout, row_offsets=ro)
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(mask), ok)
    assert np_(fake).tobytes() == of.tobytes()
    ybuf = torch.zeros(total + 16, dtype=torch.float32, device="cuda")
    y = ybuf[misalign:misalign + total]
    pwlq.dequantize(codes, mask, bits, m, p, layout=layout, row_offsets=dev(ro), out=y)
    assert np_(y).tobytes() == of.tobytes()
    assert float(ybuf[:misalign].abs().sum()) == 0 and float(ybuf[misalign + total:].abs().sum()) == 0
    assert pwlq.device_status() == 0


@pytest.mark.parametrize("ragged", [False, True])
def test_encode_host_matches_oracle(pwlq, oracle, ragged):
    """The host-buffer entry point (copies in, abs-max, search, quantize, dequantize, copies out)."""
    if ragged:
        w = W.small_mixed(seed=41, bits=4, K=64)
        x, ro, C = w.x, w.row_offsets, w.C
    else:
        rng = np.random.default_rng(2)
        x = rng.normal(0, 0.05, (12, 300)).astype(np.float32).reshape(-1)
        ro, C = None, 12
    total = x.size
    max_n = int(np.diff(ro).max()) if ragged else 300
    ratios = W.ratio_grid(64)
    hx = torch.from_numpy(x).pin_memory()
    hro = torch.from_numpy(ro).pin_memory() if ragged else None
    out = {"m": torch.empty(C, dtype=torch.float32).pin_memory(),
           "p": torch.empty(C, dtype=torch.float32).pin_memory(),
           "err": torch.empty(C, dtype=torch.float32).pin_memory(),
           "idx": torch.empty(C, dtype=torch.int32).pin_memory(),
           "codes": torch.empty((total + 1) // 2, dtype=torch.uint8).pin_memory(),
           "mask": torch.empty((total + 7) // 8, dtype=torch.uint8).pin_memory()}
    scratch = torch.empty(pwlq.encode_host_scratch_bytes(C, total, max_n, 64), dtype=torch.uint8,
                          device="cuda")
    pwlq.encode_host(hx, hro, C, max_n, 4, torch.from_numpy(ratios).pin_memory(), out,
                     pwlq.CODES_PACKED, scratch)
    torch.cuda.synchronize()
    xo = x if ragged else x.reshape(C, -1)
    om = oracle.absmax(xo, ro)
    assert np.array_equal(out["m"].numpy(), om)
    ora = oracle.search(xo, 4, ratios, row_offsets=ro)
    rows = np.arange(C)
    gi = out["idx"].numpy()
    gap = np.abs(ora["sse64"][rows, gi] - ora["sse64"][rows, ora["idx"]])
    assert np.all(gap <= 1e-5 * ora["sse64"][rows, ora["idx"]] + 1e-30)
    oc, ok, _ = oracle.quantize(xo, 4, om, out["p"].numpy(), layout=1, row_offsets=ro)
    assert np.array_equal(out["codes"].numpy(), oc) and np.array_equal(out["mask"].numpy(), ok)
    assert pwlq.encode_host_status(scratch, C, total, max_n, 64) == 0
    # a non-finite value makes its row's range non-finite: reported in the status word
    hx[total // 2] = float("inf")
    pwlq.encode_host(hx, hro, C, max_n, 4, torch.from_numpy(ratios).pin_memory(), out,
                     pwlq.CODES_PACKED, scratch)
    torch.cuda.synchronize()
    assert pwlq.encode_host_status(scratch, C, total, max_n, 64) == 1 << pwlq.ERR_NONFINITE


def test_a_bounded_wait_that_runs_out_is_reported_once(pwlq):
    """Failure detection without a fault: a one-warp kernel polls a barrier that nobody arrives on
    through the streaming kernels' own wait helper, with a limit of a few dozen polls; the wait
    runs out, the kernel sets the expiry flag and returns.  pwlq_device_status reports it once
    (reading clears it), and the library works as before afterwards."""
    torch.cuda.synchronize()
    assert pwlq.device_status() == 0
    pwlq.selftest_expire_wait(48)
    torch.cuda.synchronize()
    assert pwlq.device_status() == 1 << pwlq.ERR_TIMEOUT
    assert pwlq.device_status() == 0
    x = torch.arange(-2000, 2000, dtype=torch.float32, device="cuda").reshape(4, 1000)
    m = pwlq.absmax(x)
    torch.cuda.synchronize()
    assert m.cpu().tolist() == [2000.0, 1000.0, 999.0, 1999.0]
    assert pwlq.device_status() == 0


@pytest.mark.parametrize("layout,bits", [(1, 4), (0, 8), (1, 3)])
def test_quantize_nan_values_and_ranges_near_the_smallest_magnitudes(pwlq, oracle, layout, bits):
    """Values outside the precondition (NaN of either sign: quantized like +m by both sides) and
    rows whose range is so small that L / p or L / (m - p) overflows: every path of the kernel
    (whole passes inside a row, passes with row starts, the tensor's tail) must give the oracle's
    bytes."""
    rng = np.random.default_rng(5 + bits)
    lengths = np.array([512, 147, 40, 1024, 9, 300, 4096 + 24, 77], np.int64)
    ro = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
    x = rng.laplace(0, 0.03, int(ro[-1])).astype(np.float32)
    tiny = [1, 3, 6]                                         # rows scaled into the subnormal range
    for c, scale in zip(tiny, (1e-38, 3e-39, 1e-41)):
        x[ro[c]:ro[c + 1]] *= np.float32(scale) / np.float32(0.03)
    m = oracle.absmax(x, ro)
    p = (m * rng.uniform(0.2, 0.9, lengths.size).astype(np.float32)).astype(np.float32)
    p[6] = m[6] * np.float32(1 - 2.0 ** -20)                 # a tail range of a few subnormal steps
    nan_pos = np.frombuffer(np.array([0x7FC00000], np.uint32).tobytes(), np.float32)[0]
    nan_neg = np.frombuffer(np.array([0xFFC00000], np.uint32).tobytes(), np.float32)[0]
    for c in (0, 2, 3, 5):
        b, e = int(ro[c]), int(ro[c + 1])
        x[b] = nan_pos; x[b + 1] = nan_neg; x[e - 1] = nan_neg; x[(b + e) // 2] = nan_pos
    oc, om, of = oracle.quantize(x, bits, m, p, layout=layout, row_offsets=ro)
    codes, mask, fake = pwlq.quantize(dev(x), bits, dev(m), dev(p), layout=layout,
                                      row_offsets=dev(ro), want_fake=True)
    y = pwlq.dequantize(codes, mask, bits, dev(m), dev(p), layout=layout, row_offsets=dev(ro))
    torch.cuda.synchronize()
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(mask), om)
    assert np_(fake).tobytes() == of.tobytes() and np_(y).tobytes() == of.tobytes()


@pytest.mark.parametrize("K", [64, 256])
def test_search_many_ragged_rows_of_every_class_with_full_tiles(pwlq, oracle, K):
    """Enough rows that long rows keep full tiles (no finer cut), rows of every row-length class
    and rows of several tiles in one call: every class launch writes its rows' partial sums and
    the combine kernels read them all.  Repeated: the result must not change from run to run."""
    rng = np.random.default_rng(K)
    lengths = np.concatenate([rng.integers(1, 3001, 400), [9001, 20000, 8192, 8193, 64, 65, 512,
                                                           513, 2304, 2305]]).astype(np.int64)
    rng.shuffle(lengths)
    ro = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
    x = (rng.standard_normal(int(ro[-1])) * rng.choice([0.01, 1.0, 30.0], 1)).astype(np.float32)
    ratios = W.ratio_grid(K)
    first = None
    for rep in range(3):
        out, status = run_search(pwlq, x, 4, ratios, row_offsets=ro, max_n=int(lengths.max()))
        assert status == 0
        if first is None:
            first = out
            m = oracle.absmax(x, ro)
            ora = oracle.search(x, 4, ratios, m=m, row_offsets=ro)
            check_search(out, ora, ratios, m, lengths)
        else:
            for k in ("p", "err", "idx", "sse"):
                assert out[k].tobytes() == first[k].tobytes(), (rep, k)


@pytest.mark.parametrize("kind", ["sparse", "relu_sparse", "on_a_grid"])
@pytest.mark.parametrize("bits", [3, 4, 7, 8])
def test_search_sums_carried_by_a_few_small_errors(pwlq, oracle, kind, bits):
    """Pruned, ReLU-ed or already quantized values: under some candidates almost every value sits
    on a level, and a sum is then orders of magnitude below n * step^2 / 12 and made of a few
    small errors e_i.  Each e_i is a difference of two binary32 numbers of the size of m, known
    to about one ulp of m on either side (the oracle rounds q * s and + z, the search rounds the
    fused form once), so two correct evaluations may differ by sum 2 |e_i| ulp(m) <=
    2 sqrt(n * SSE) * 2^-23 m in first order.  The 1e-5 relative bar holds where the sums have
    their usual size; this test holds the search to the first-order bound elsewhere."""
    rng = np.random.default_rng(bits * 7 + len(kind))
    lens = rng.choice([32, 40, 64, 147, 512, 1000, 4096, 4608, 9000], 120).astype(np.int64)
    ro = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    total = int(ro[-1])
    x = rng.laplace(0, 0.05, total).astype(np.float32)
    if kind == "relu_sparse":
        x = np.maximum(x, 0)
    if kind == "on_a_grid":
        x = (np.round(x * 64) / 64).astype(np.float32)
    else:
        x[rng.random(total) < np.repeat(rng.choice([0.5, 0.9, 0.99], lens.size), lens)] = 0.0
    om = oracle.absmax(x, ro)
    ratios = W.ratio_grid(64)
    s = pwlq.search(dev(x), bits, dev(ratios), m=dev(om), row_offsets=dev(ro), max_n=int(lens.max()),
                    want_sse=True)
    ora = oracle.search(x, bits, ratios, row_offsets=ro)
    sse = np_(s["sse"]).astype(np.float64)
    o = ora["sse64"]
    ulp_m = 2.0 ** -23 * om.astype(np.float64)[:, None]
    n = lens[:, None].astype(np.float64)
    bound = 1e-5 * o + 2.0 * np.sqrt(n * o) * ulp_m + n * ulp_m ** 2 + 2.0 ** -23 * o
    assert np.all(np.abs(sse - o) <= bound)
    # the chosen candidate is the oracle's, or as good within the same bound
    rows = np.arange(lens.size)
    gi, oi = np_(s["idx"]).astype(np.int64), ora["idx"].astype(np.int64)
    assert np.all(np.abs(o[rows, gi] - o[rows, oi]) <= bound[rows, oi])
    assert pwlq.device_status() == 0
