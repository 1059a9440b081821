"""GPU parity of the three-breakpoint calls (triple search, quantize, dequantize) against the
oracle's plain definition (every triple evaluated value by value)."""
import itertools

import numpy as np
import pytest
import torch

from gpu_util import SSE_RTOL, dev, sse_atol
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


def check_triples(got, ora, ratios, m, row_len):
    """Sum of every triple within the parity tolerance; the chosen triple equal to the oracle's
    unless the oracle's own sums are a near-tie; breakpoints and error consistent with it."""
    C, K = ora["idx"].shape[0], ratios.size
    row_len = np.broadcast_to(np.asarray(row_len), (C,))
    valid = np.zeros((K, K, K), bool)
    for t3 in itertools.combinations(range(K), 3):
        valid[t3] = True
    for c in range(C):
        o = ora["sse64"][c]
        atol = sse_atol(row_len[c], m[c])
        if got["sse"] is not None:
            g = got["sse"][c].astype(np.float64)
            assert np.all(g[~valid] == 0.0)
            d = np.abs(g[valid] - o[valid])
            assert np.all(d <= SSE_RTOL * o[valid] + atol + 2.0 ** -23 * o[valid]), (c, d.max())
        gt = tuple(int(v) for v in got["idx"][c])
        ot = tuple(int(v) for v in ora["idx"][c])
        assert 0 <= gt[0] < gt[1] < gt[2] < K
        if gt != ot:
            assert abs(o[gt] - o[ot]) <= SSE_RTOL * o[ot] + atol, (c, gt, ot)
        if m[c] > 0:
            assert got["p"][c].tolist() == [float(np.float32(m[c]) * ratios[i]) for i in gt]
        else:
            assert got["p"][c].tolist() == [0.0, 0.0, 0.0]
        assert abs(float(got["err"][c]) - o[gt]) <= SSE_RTOL * o[gt] + atol + 2.0 ** -23 * o[gt]


def run_search3(pwlq, x, bits, ratios, m, row_offsets=None, max_n=None, want_sse=True):
    out = pwlq.search3(dev(x), bits, dev(ratios), dev(m),
                       row_offsets=None if row_offsets is None else dev(row_offsets), max_n=max_n,
                       want_sse=want_sse)
    torch.cuda.synchronize()
    status = int(out["workspace"][:4].view(torch.int32).item())
    return {k: np_(out[k]) for k in ("p", "err", "idx", "sse")}, status


def test_search3_worked_example(pwlq):
    """The hand-worked fixture: triples of (3, 6, 12, 24) on sixteen dyadic values."""
    from conftest import read_golden
    g = read_golden("worked_example_three_breakpoints_b3.txt")
    x = np.array([float(v) for v in g["x"]], np.float32).reshape(1, -1)
    ratios = np.array([float(v) for v in g["ratios"]], np.float32)
    got, status = run_search3(pwlq, x, 3, ratios, np.array([24.0], np.float32))
    assert status == 0
    assert got["idx"][0].tolist() == [0, 1, 2] and got["p"][0].tolist() == [3.0, 6.0, 12.0]
    for t3 in itertools.combinations(range(4), 3):
        assert got["sse"][0][t3] == float(g["sse.%d.%d.%d" % t3][0])
    assert float(got["err"][0]) == 16.25
    xd, md, pd = dev(x), dev(np.array([24.0], np.float32)), dev(got["p"])
    codes, reg, fake = pwlq.quantize3(xd, 3, md, pd, layout=1, want_fake=True)
    assert np_(codes).tolist() == [int(v, 16) for v in g["packed.0.1.2"]]
    assert np_(reg).tolist() == [int(v, 16) for v in g["region_bytes.0.1.2"]]
    assert np_(fake).tolist() == [float(v) for v in g["y.0.1.2"]]


@pytest.mark.parametrize("bits,K", [(2, 6), (3, 10), (4, 12), (8, 7)])
@pytest.mark.parametrize("C,n", [(5, 9), (4, 300), (3, 4097), (2, 8192)])
def test_search3_dense(pwlq, oracle, bits, K, C, n):
    rng = np.random.default_rng(bits * 100 + K + n)
    x = (rng.laplace(0, 0.02, (C, n)) if n % 2 else rng.standard_normal((C, n))).astype(np.float32)
    m = oracle.absmax(x)
    ratios = W.ratio_grid(K)
    got, status = run_search3(pwlq, x, bits, ratios, m)
    assert status == 0
    check_triples(got, oracle.search3(x, bits, ratios, m), ratios, m, n)


@pytest.mark.parametrize("bits,K,C,n", [(4, 8, 2, 8193), (3, 6, 1, 40000)])
def test_search3_rows_longer_than_a_tile(pwlq, oracle, bits, K, C, n):
    rng = np.random.default_rng(n + K)
    x = rng.laplace(0, 0.02, (C, n)).astype(np.float32)
    m = oracle.absmax(x)
    ratios = W.ratio_grid(K)
    got, status = run_search3(pwlq, x, bits, ratios, m)
    assert status == 0
    check_triples(got, oracle.search3(x, bits, ratios, m), ratios, m, n)
    again, _ = run_search3(pwlq, x, bits, ratios, m)
    assert all(np.array_equal(got[k], again[k]) for k in got)


def test_search3_ragged_rows_ties_and_degenerate_rows(pwlq, oracle):
    rng = np.random.default_rng(8)
    lengths = [33, 0, 11, 9001, 3, 700, 16400]
    x = rng.standard_normal(sum(lengths)).astype(np.float32)
    ro = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
    x[ro[2]:ro[3]] = 0.0                                        # a row of zeros
    x[ro[4]:ro[5]] = [1.5, -1.5, 1.5]                           # all |x| = m: every triple exact
    m = oracle.absmax(x, ro)
    ratios = W.ratio_grid(8)
    got, status = run_search3(pwlq, x, 4, ratios, m, row_offsets=ro, max_n=max(lengths))
    assert status == 0
    check_triples(got, oracle.search3(x, 4, ratios, m, row_offsets=ro), ratios, m, np.diff(ro))
    for c in (1, 2, 4):
        assert got["idx"][c].tolist() == [0, 1, 2] and got["err"][c] == 0.0


def test_search3_contains_the_pair_search_and_improves_on_it(pwlq):
    """Triples (i, j, K-1) with ratios[K-1] = 1 are the pairs (i, j)."""
    rng = np.random.default_rng(13)
    x = dev(rng.standard_normal((4, 3000)).astype(np.float32))
    m = pwlq.absmax(x)
    ratios = dev(W.ratio_grid(12))
    three = pwlq.search3(x, 4, ratios, m, want_sse=True)
    two = pwlq.search2(x, 4, ratios, m, want_sse=True)
    a, b = three["sse"][:, :11, :11, 11].double(), two["sse"][:, :11, :11].double()
    assert torch.all((a - b).abs() <= 2e-6 * b)
    assert torch.all(three["err"] <= two["err"] * (1 + 1e-6))


def test_search3_limits_and_bad_grid(pwlq):
    x = torch.zeros(2, 16, device="cuda") + 1.0
    m = pwlq.absmax(x)
    with pytest.raises(pwlq.PwlqError) as e:
        pwlq.search3(x, 4, dev(W.ratio_grid(65)), m)
    assert e.value.status == pwlq.ERR_UNSUPPORTED
    with pytest.raises(pwlq.PwlqError):
        pwlq.search3(x, 4, dev(W.ratio_grid(2)), m)
    out = pwlq.search3(x, 4, dev(np.array([0.5, 0.25, 0.75, 1.0], np.float32)), m)   # not ascending
    torch.cuda.synchronize()
    assert int(out["workspace"][:4].view(torch.int32).item()) == 1 << pwlq.ERR_INVALID_ARG


@pytest.mark.parametrize("bits,layout", [(2, 1), (4, 1), (4, 0), (8, 0)])
@pytest.mark.parametrize("C,n", [(1, 7), (5, 147), (3, 4096), (300, 27)])
def test_quantize3_dequantize3_dense(pwlq, oracle, bits, layout, C, n):
    rng = np.random.default_rng(bits + 10 * layout + n)
    x = rng.laplace(0, 0.05, (C, n)).astype(np.float32)
    m = oracle.absmax(x)
    if C > 1:
        x[1] = 0.0
        m[1] = 0.0
    r = np.sort(rng.uniform(0.03, 1.0, (C, 3)), axis=1)
    r[::4, 2] = 1.0                                             # p3 = m: the fourth region is empty
    p = (m[:, None] * r).astype(np.float32)
    codes, reg, fake = pwlq.quantize3(dev(x), bits, dev(m), dev(p), layout=layout, want_fake=True)
    oc, orr, of = oracle.quantize3(x, bits, m, p, layout=layout)
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(reg), orr)
    assert np_(fake).tobytes() == of.tobytes()
    y = pwlq.dequantize3(codes, reg, bits, dev(m), dev(p), C=C, n=n, layout=layout)
    assert np_(y).tobytes() == oracle.dequantize3(oc, orr, bits, m, p, C=C, n=n,
                                                  layout=layout).tobytes()
    assert np_(y).tobytes() == of.tobytes()


def test_quantize3_dequantize3_ragged_after_search(pwlq, oracle):
    w = W.small_mixed(seed=19)
    x, ro = w.x, w.row_offsets
    xd, rod = dev(x), dev(ro)
    m = pwlq.absmax(xd, row_offsets=rod)
    out = pwlq.search3(xd, 3, dev(W.ratio_grid(10)), m, row_offsets=rod,
                       max_n=int(np.diff(ro).max()))
    codes, reg, fake = pwlq.quantize3(xd, 3, m, out["p"], layout=1, row_offsets=rod, want_fake=True)
    y = pwlq.dequantize3(codes, reg, 3, m, out["p"], layout=1, row_offsets=rod)
    torch.cuda.synchronize()
    oc, orr, of = oracle.quantize3(x, 3, np_(m), np_(out["p"]), layout=1, row_offsets=ro)
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(reg), orr)
    assert np_(fake).tobytes() == of.tobytes() and np_(y).tobytes() == of.tobytes()


@pytest.mark.parametrize("misalign", [0, 1, 4])
def test_quantize3_dequantize3_with_buffers_off_their_vector_alignment(pwlq, oracle, misalign):
    """Aligned buffers take the producer / consumer kernels, anything else the element-wise ones:
    the same bytes either way, and nothing written outside the outputs."""
    rng = np.random.default_rng(31 + misalign)
    lengths = [5000, 13, 4096, 700, 701, 702, 9000, 3]
    ro = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
    total = int(ro[-1])
    x = rng.laplace(0, 0.05, total).astype(np.float32)
    m = oracle.absmax(x, ro)
    p = (m[:, None] * np.array([0.15, 0.4, 0.8], dtype=np.float32)[None, :]).astype(np.float32)
    bits, layout = 4, 1
    xb = dev(np.concatenate([np.zeros(misalign, np.float32), x]))[misalign:]
    nbytes = pwlq.code_bytes(total, bits, layout)
    nreg = (total + 3) // 4
    cbuf = torch.zeros(nbytes + 32, dtype=torch.uint8, device="cuda")
    rbuf = torch.zeros(nreg + 32, dtype=torch.uint8, device="cuda")
    fbuf = torch.zeros(total + 32, dtype=torch.float32, device="cuda")
    ybuf = torch.zeros(total + 32, dtype=torch.float32, device="cuda")
    codes, reg = cbuf[misalign:misalign + nbytes], rbuf[misalign:misalign + nreg]
    fake, y = fbuf[misalign:misalign + total], ybuf[misalign:misalign + total]
    pwlq.quantize3(xb, bits, dev(m), dev(p), layout=layout, row_offsets=dev(ro), out=(codes, reg, fake))
    pwlq.dequantize3(codes, reg, bits, dev(m), dev(p), layout=layout, row_offsets=dev(ro), out=y)
    torch.cuda.synchronize()
    oc, orr, of = oracle.quantize3(x, bits, m, p, layout=layout, row_offsets=ro)
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(reg), orr)
    assert np_(fake).tobytes() == of.tobytes() and np_(y).tobytes() == of.tobytes()
    for buf, n in ((cbuf, nbytes), (rbuf, nreg), (fbuf, total), (ybuf, total)):
        assert float(buf[:misalign].float().abs().sum()) == 0
        assert float(buf[misalign + n:].float().abs().sum()) == 0
    assert pwlq.device_status() == 0
