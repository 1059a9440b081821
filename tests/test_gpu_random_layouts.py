"""Seeded random row layouts through every streaming call (abs-max, min/max, quantize, dequantize,
the same with row maps built ahead of time, and the two- / three-breakpoint quantizers), compared
with the CPU oracle bit for bit; the search's sums within its tolerance.  Layout kinds: tiny rows,
short rows, lengths around the span and tile sizes, many empty rows, long rows; buffers shifted
off their vector alignment in three cases out of four."""
import numpy as np
import pytest
import torch

from gpu_util import dev
from paper_2002_00104_b200 import workloads as W

pytestmark = [pytest.mark.gpu,
              pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]


@pytest.fixture(scope="module")
def pwlq():
    from paper_2002_00104_b200 import pwlq as _p
    _p.load_library()
    return _p


def np_(t):
    return t.cpu().numpy()


def random_layout(rng):
    nrows = int(rng.integers(1, 2500))
    kind = int(rng.integers(0, 5))
    if kind == 0:
        lens = rng.integers(0, 17, nrows)
    elif kind == 1:
        lens = rng.integers(0, 600, nrows)
    elif kind == 2:
        lens = rng.choice([0, 1, 7, 8, 9, 4095, 4096, 4097, 8192, 12288], nrows % 300 + 1)
    elif kind == 3:
        lens = np.where(rng.random(nrows) < 0.3, 0, rng.integers(1, 40, nrows))
    else:
        lens = rng.integers(1, 9000, nrows % 400 + 1)
    return lens.astype(np.int64)


@pytest.mark.parametrize("seed", range(24))
def test_random_layout(pwlq, oracle, seed):
    rng = np.random.default_rng(1000 + seed)
    lens = random_layout(rng)
    while lens.sum() == 0 or lens.sum() > 3_000_000:
        lens = random_layout(rng)
    total = int(lens.sum())
    ro = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    x = rng.laplace(0, 0.05, total).astype(np.float32)
    x[rng.random(total) < 0.01] = 0.0
    mis = int(rng.integers(0, 4))
    xb = dev(np.concatenate([np.zeros(mis, np.float32), x]))[mis:]
    rod = dev(ro)
    bits, layout = int(rng.integers(2, 9)), int(rng.integers(0, 2))

    # ranges
    om = oracle.absmax(x, ro)
    assert np.array_equal(np_(pwlq.absmax(xb, row_offsets=rod)), om)
    lo, hi = pwlq.minmax(xb, row_offsets=rod)
    olo, ohi = oracle.minmax(x, ro)
    assert np.array_equal(np_(lo), olo) and np.array_equal(np_(hi), ohi)

    # one breakpoint, plain and with row maps built ahead of time
    p = (om * rng.uniform(0.02, 1.0, om.size)).astype(np.float32)
    oc, ok, of = oracle.quantize(x, bits, om, p, layout=layout, row_offsets=ro)
    rmap = pwlq.rowmap_build(om.size, total, row_offsets=rod)
    assert np.array_equal(np_(pwlq.absmax(xb, row_offsets=rod, rowmap=rmap)), om)
    for kw in ({}, {"rowmap": rmap}):
        codes, mask, fake = pwlq.quantize(xb, bits, dev(om), dev(p), layout=layout, row_offsets=rod,
                                          want_fake=True, **kw)
        assert np.array_equal(np_(codes), oc) and np.array_equal(np_(mask), ok)
        assert np_(fake).tobytes() == of.tobytes()
        y = pwlq.dequantize(codes, mask, bits, dev(om), dev(p), layout=layout, row_offsets=rod, **kw)
        assert np_(y).tobytes() == of.tobytes()

    # two and three breakpoints; some rows delivered as zeros, some with an empty last region
    r3 = np.sort(rng.uniform(0.03, 1.0, (om.size, 3)), axis=1)
    r3[rng.random(om.size) < 0.2, 2] = 1.0
    p3 = (om[:, None] * r3).astype(np.float32)
    om0 = om.copy()
    om0[rng.random(om.size) < 0.05] = 0.0
    c3, g3, f3 = pwlq.quantize3(xb, bits, dev(om0), dev(p3), layout=layout, row_offsets=rod,
                                want_fake=True)
    oc3, og3, of3 = oracle.quantize3(x, bits, om0, p3, layout=layout, row_offsets=ro)
    assert np.array_equal(np_(c3), oc3) and np.array_equal(np_(g3), og3)
    assert np_(f3).tobytes() == of3.tobytes()
    y3 = pwlq.dequantize3(c3, g3, bits, dev(om0), dev(p3), layout=layout, row_offsets=rod)
    assert np_(y3).tobytes() == of3.tobytes()
    p1, p2 = np.ascontiguousarray(p3[:, 0]), np.ascontiguousarray(p3[:, 1])
    c2, g2, f2 = pwlq.quantize2(xb, bits, dev(om0), dev(p1), dev(p2), layout=layout, row_offsets=rod,
                                want_fake=True)
    oc2, og2, of2 = oracle.quantize2(x, bits, om0, p1, p2, layout=layout, row_offsets=ro)
    assert np.array_equal(np_(c2), oc2) and np.array_equal(np_(g2), og2)
    assert np_(f2).tobytes() == of2.tobytes()
    y2 = pwlq.dequantize2(c2, g2, bits, dev(om0), dev(p1), dev(p2), layout=layout, row_offsets=rod)
    assert np_(y2).tobytes() == of2.tobytes()

    # the search's sums
    K = int(rng.choice([1, 7, 64, 100]))
    ratios = W.ratio_grid(K)
    s = pwlq.search(xb, bits, dev(ratios), m=dev(om), row_offsets=rod, max_n=int(lens.max()),
                    want_sse=True)
    ora = oracle.search(x, bits, ratios, row_offsets=ro)
    sse = np_(s["sse"]).astype(np.float64)
    tol = 1e-5 * ora["sse64"] + lens[:, None] * (2.0 ** -23 * om[:, None]) ** 2 + 2.0 ** -23 * ora["sse64"]
    assert np.all(np.abs(sse - ora["sse64"]) <= tol)
    assert pwlq.device_status() == 0


@pytest.mark.parametrize("seed", range(8))
def test_random_layout_from_host_buffers(pwlq, oracle, seed):
    """The host-buffer entry points (signed and one-sided) cut the rows into runs of their own; the
    results must not depend on where the cuts fall."""
    rng = np.random.default_rng(2000 + seed)
    lens = random_layout(rng)
    while lens.sum() == 0 or lens.sum() > 3_000_000:
        lens = random_layout(rng)
    total, C, max_n = int(lens.sum()), lens.size, int(lens.max())
    ro = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    one_sided = bool(seed & 1)
    x = rng.laplace(0, 0.05, total).astype(np.float32)
    if one_sided:
        x = (np.maximum(x, 0) + np.float32(0.1)).astype(np.float32)
    bits, layout, K = int(rng.integers(2, 9)), int(rng.integers(0, 2)), int(rng.choice([7, 64, 100]))
    ratios = W.ratio_grid(K)

    def pin(a):
        return torch.from_numpy(np.ascontiguousarray(a)).pin_memory()

    out = {k: torch.empty(C, dtype=torch.float32).pin_memory() for k in ("m", "p", "err", "lo", "hi")}
    out["idx"] = torch.empty(C, dtype=torch.int32).pin_memory()
    out["codes"] = torch.empty(pwlq.code_bytes(total, bits, layout), dtype=torch.uint8).pin_memory()
    out["mask"] = torch.empty((total + 7) // 8, dtype=torch.uint8).pin_memory()
    scratch = torch.empty(pwlq.encode_host_scratch_bytes(C, total, max_n, K), dtype=torch.uint8,
                          device="cuda")
    call = pwlq.encode_host_unsigned if one_sided else pwlq.encode_host
    call(pin(x), pin(ro), C, max_n, bits, pin(ratios), out, layout, scratch)
    torch.cuda.synchronize()
    p = out["p"].numpy()
    if one_sided:
        olo, ohi = oracle.minmax(x, ro)
        assert np.array_equal(out["lo"].numpy(), olo) and np.array_equal(out["hi"].numpy(), ohi)
        ora = oracle.search_u(x, bits, ratios, olo, ohi, row_offsets=ro)
        width = (ohi - olo).astype(np.float64)
        oc, ok, _ = oracle.quantize_u(x, bits, olo, ohi, p, layout=layout, row_offsets=ro)
    else:
        om = oracle.absmax(x, ro)
        assert np.array_equal(out["m"].numpy(), om)
        ora = oracle.search(x, bits, ratios, row_offsets=ro)
        width = om.astype(np.float64)
        oc, ok, _ = oracle.quantize(x, bits, om, p, layout=layout, row_offsets=ro)
    o, rows = ora["sse64"], np.arange(C)
    gi, oi = out["idx"].numpy().astype(np.int64), ora["idx"].astype(np.int64)
    tol = 1e-5 * o[rows, oi] + lens * (2.0 ** -23 * width) ** 2
    assert np.all(np.abs(o[rows, gi] - o[rows, oi]) <= tol)      # the oracle's choice, or a near-tie
    assert np.array_equal(out["codes"].numpy(), oc) and np.array_equal(out["mask"].numpy(), ok)
    assert pwlq.encode_host_status(scratch, C, total, max_n, K) == 0
    assert pwlq.device_status() == 0
