"""GPU parity of the two-breakpoint calls (pair search, quantize, dequantize) against the oracle."""
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


def check_pairs(got, ora, ratios, m, row_len):
    """SSE of every pair within the parity tolerance; the chosen pair equal to the oracle's unless
    the oracle's own sums are a near-tie; p1, p2 and the error consistent with the chosen pair."""
    C, K = ora["idx1"].size, ratios.size
    iu = np.triu_indices(K, 1)
    row_len = np.broadcast_to(np.asarray(row_len), (C,))
    for c in range(C):
        o = ora["sse64"][c]
        atol = sse_atol(row_len[c], m[c])
        if got["sse"] is not None:
            g = got["sse"][c].astype(np.float64)
            assert np.all(g[np.tril_indices(K)] == 0.0)
            d = np.abs(g[iu] - o[iu])
            assert np.all(d <= SSE_RTOL * o[iu] + atol + 2.0 ** -23 * o[iu]), (c, d.max())
        gi, gj = int(got["idx1"][c]), int(got["idx2"][c])
        oi, oj = int(ora["idx1"][c]), int(ora["idx2"][c])
        assert 0 <= gi < gj < K
        if (gi, gj) != (oi, oj):
            assert abs(o[gi, gj] - o[oi, oj]) <= SSE_RTOL * o[oi, oj] + atol, (c, (gi, gj), (oi, oj))
        if m[c] > 0:
            assert got["p1"][c] == np.float32(m[c]) * ratios[gi]
            assert got["p2"][c] == np.float32(m[c]) * ratios[gj]
        else:
            assert got["p1"][c] == 0 and got["p2"][c] == 0
        assert abs(float(got["err"][c]) - o[gi, gj]) <= SSE_RTOL * o[gi, gj] + atol + 2.0 ** -23 * o[gi, gj]


def run_search2(pwlq, x, bits, ratios, m, row_offsets=None, max_n=None, want_sse=True):
    out = pwlq.search2(dev(x), bits, dev(ratios), dev(m),
                       row_offsets=None if row_offsets is None else dev(row_offsets), max_n=max_n,
                       want_sse=want_sse)
    torch.cuda.synchronize()
    status = int(out["workspace"][:4].view(torch.int32).item())
    return {k: np_(out[k]) for k in ("p1", "p2", "err", "idx1", "idx2", "sse")}, status


@pytest.mark.parametrize("bits,K", [(2, 8), (3, 16), (4, 24), (8, 12)])
@pytest.mark.parametrize("C,n", [(5, 9), (4, 300), (3, 4097), (2, 8192)])
def test_search2_dense(pwlq, oracle, bits, K, C, n):
    rng = np.random.default_rng(bits * 100 + K + n)
    x = (rng.laplace(0, 0.02, (C, n)) if n % 2 else rng.standard_normal((C, n))).astype(np.float32)
    m = oracle.absmax(x)
    ratios = W.ratio_grid(K)
    got, status = run_search2(pwlq, x, bits, ratios, m)
    assert status == 0
    check_pairs(got, oracle.search2(x, bits, ratios, m), ratios, m, n)


def test_search2_ragged_mixed_rows(pwlq, oracle):
    w = W.small_mixed(seed=3)
    keep = np.diff(w.row_offsets) <= 8192
    rows = [w.x[w.row_offsets[c]:w.row_offsets[c + 1]] for c in range(w.C) if keep[c]]
    rows.insert(2, np.zeros(0, np.float32))                     # an empty row
    rows.insert(4, np.zeros(11, np.float32))                    # a row of zeros
    x = np.concatenate(rows).astype(np.float32)
    ro = np.concatenate([[0], np.cumsum([r.size for r in rows])]).astype(np.int64)
    m = oracle.absmax(x, ro)
    ratios = W.ratio_grid(20)
    got, status = run_search2(pwlq, x, 4, ratios, m, row_offsets=ro, max_n=int(np.diff(ro).max()))
    assert status == 0
    check_pairs(got, oracle.search2(x, 4, ratios, m, row_offsets=ro), ratios, m, np.diff(ro))
    assert (got["idx1"][2], got["idx2"][2], got["err"][2]) == (0, 1, 0.0)
    assert (got["idx1"][4], got["idx2"][4], got["p2"][4]) == (0, 1, 0.0)


@pytest.mark.parametrize("bits,K,C,n", [(4, 16, 3, 8193), (3, 12, 2, 20000), (8, 8, 1, 70001)])
def test_search2_rows_longer_than_a_tile(pwlq, oracle, bits, K, C, n):
    """Rows cut into tiles of 8192 values: the tiles' terms are added by the row-closing kernel."""
    rng = np.random.default_rng(n + K)
    x = rng.laplace(0, 0.02, (C, n)).astype(np.float32)
    m = oracle.absmax(x)
    ratios = W.ratio_grid(K)
    got, status = run_search2(pwlq, x, bits, ratios, m)
    assert status == 0
    check_pairs(got, oracle.search2(x, bits, ratios, m), ratios, m, n)
    again, _ = run_search2(pwlq, x, bits, ratios, m)
    assert all(np.array_equal(got[k], again[k]) for k in got)           # fixed order of the tiles


def test_search2_ragged_rows_with_and_without_tiles(pwlq, oracle):
    rng = np.random.default_rng(5)
    lengths = [9001, 0, 300, 8192, 16385, 1, 12000]
    x = rng.standard_normal(sum(lengths)).astype(np.float32)
    ro = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
    x[ro[2]:ro[3]] = 0.0                                        # a row of zeros among tiled rows
    m = oracle.absmax(x, ro)
    ratios = W.ratio_grid(10)
    got, status = run_search2(pwlq, x, 4, ratios, m, row_offsets=ro, max_n=max(lengths))
    assert status == 0
    check_pairs(got, oracle.search2(x, 4, ratios, m, row_offsets=ro), ratios, m, np.diff(ro))
    assert (got["idx1"][1], got["idx2"][1], got["err"][1]) == (0, 1, 0.0)
    assert (got["idx1"][2], got["idx2"][2], got["p2"][2]) == (0, 1, 0.0)


def test_search2_with_p2_at_m_contains_the_one_breakpoint_search(pwlq):
    """Pairs (i, K-1) with ratios[K-1] = 1 are the one-breakpoint candidates i (same arithmetic up
    to the summation order)."""
    rng = np.random.default_rng(12)
    x = dev(rng.standard_normal((6, 2000)).astype(np.float32))
    m = pwlq.absmax(x)
    ratios = dev(W.ratio_grid(32))
    two = pwlq.search2(x, 4, ratios, m, want_sse=True)
    one = pwlq.search(x, 4, ratios, m=m, want_sse=True)
    a, b = two["sse"][:, :31, 31].double(), one["sse"][:, :31].double()
    assert torch.all((a - b).abs() <= 2e-6 * b)
    assert torch.all(two["err"] <= one["err"] * (1 + 1e-6))


def test_search2_limits_and_bad_grid(pwlq):
    x = torch.zeros(2, 16, device="cuda") + 1.0
    m = pwlq.absmax(x)
    with pytest.raises(pwlq.PwlqError) as e:
        pwlq.search2(x, 4, dev(W.ratio_grid(65)), m)
    assert e.value.status == pwlq.ERR_UNSUPPORTED
    small = torch.empty(256, dtype=torch.uint8, device="cuda")           # a long row needs more
    with pytest.raises(pwlq.PwlqError) as e:
        pwlq.search2(torch.zeros(1, 8200, device="cuda"), 4, dev(W.ratio_grid(8)), m[:1],
                     workspace=small)
    assert e.value.status == pwlq.ERR_WORKSPACE
    with pytest.raises(pwlq.PwlqError):
        pwlq.search2(x, 4, dev(W.ratio_grid(1)), m)
    out = pwlq.search2(x, 4, dev(np.array([0.5, 0.25, 1.0], np.float32)), m)   # not ascending
    torch.cuda.synchronize()
    assert int(out["workspace"][:4].view(torch.int32).item()) == 1 << pwlq.ERR_INVALID_ARG


@pytest.mark.parametrize("bits,layout", [(2, 1), (4, 1), (4, 0), (8, 0)])
@pytest.mark.parametrize("C,n", [(1, 7), (5, 147), (3, 4096), (300, 27)])
def test_quantize2_dequantize2_dense(pwlq, oracle, bits, layout, C, n):
    rng = np.random.default_rng(bits + 10 * layout + n)
    x = rng.laplace(0, 0.05, (C, n)).astype(np.float32)
    m = oracle.absmax(x)
    if C > 1:
        x[1] = 0.0
        m[1] = 0.0
    r1 = rng.uniform(0.05, 0.5, C)
    p1 = (m * r1).astype(np.float32)
    p2 = (m * np.minimum(r1 + rng.uniform(0.0, 0.6, C), 1.0)).astype(np.float32)
    codes, reg, fake = pwlq.quantize2(dev(x), bits, dev(m), dev(p1), dev(p2), layout=layout,
                                      want_fake=True)
    oc, orr, of = oracle.quantize2(x, bits, m, p1, p2, layout=layout)
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(reg), orr)
    assert np_(fake).tobytes() == of.tobytes()
    y = pwlq.dequantize2(codes, reg, bits, dev(m), dev(p1), dev(p2), C=C, n=n, layout=layout)
    assert np_(y).tobytes() == oracle.dequantize2(oc, orr, bits, m, p1, p2, C=C, n=n,
                                                  layout=layout).tobytes()
    assert np_(y).tobytes() == of.tobytes()


def test_quantize2_dequantize2_ragged_after_search(pwlq, oracle):
    w = W.small_mixed(seed=17)
    keep = np.diff(w.row_offsets) <= 8192
    rows = [w.x[w.row_offsets[c]:w.row_offsets[c + 1]] for c in range(w.C) if keep[c]]
    rows.insert(1, np.zeros(0, np.float32))
    x = np.concatenate(rows).astype(np.float32)
    ro = np.concatenate([[0], np.cumsum([r.size for r in rows])]).astype(np.int64)
    xd, rod = dev(x), dev(ro)
    m = pwlq.absmax(xd, row_offsets=rod)
    out = pwlq.search2(xd, 3, dev(W.ratio_grid(16)), m, row_offsets=rod,
                       max_n=int(np.diff(ro).max()))
    codes, reg, fake = pwlq.quantize2(xd, 3, m, out["p1"], out["p2"], layout=1, row_offsets=rod,
                                      want_fake=True)
    y = pwlq.dequantize2(codes, reg, 3, m, out["p1"], out["p2"], layout=1, row_offsets=rod)
    torch.cuda.synchronize()
    mm, p1, p2 = np_(m), np_(out["p1"]), np_(out["p2"])
    oc, orr, of = oracle.quantize2(x, 3, mm, p1, p2, layout=1, row_offsets=ro)
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(reg), orr)
    assert np_(fake).tobytes() == of.tobytes() and np_(y).tobytes() == of.tobytes()
