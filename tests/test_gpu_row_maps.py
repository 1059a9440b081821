"""GPU parity of the streaming kernels (abs-max, min/max, quantize, dequantize) on row layouts
chosen around the limits of their row maps: a span of the flat storage is 4096 values, a map
describes up to about 510 rows of a span, rows may start exactly at span boundaries, be empty, be
shorter than the eight values a lane owns, or change length from span to span.  Everything is
compared with the CPU oracle bit for bit."""
import numpy as np
import pytest
import torch

from gpu_util import dev

pytestmark = [pytest.mark.gpu,
              pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]

SPAN = 4096


@pytest.fixture(scope="module")
def pwlq():
    from paper_2002_00104_b200 import pwlq as _p
    _p.load_library()
    return _p


def np_(t):
    return t.cpu().numpy()


def layouts():
    """name -> list of row lengths."""
    rng = np.random.default_rng(11)
    out = {
        # more rows per span than a map describes, then long rows again (slow spans and back)
        "tiny_then_long": [1] * 3000 + [2, 3] * 900 + [5000, 3, 4096, 8192, 1],
        # 455 / 512 / 585 rows per span: below, at and above the limit
        "rows_of_9": [9] * 2000,
        "rows_of_8": [8] * 2100,
        "rows_of_7": [7] * 2400,
        # starts exactly at span boundaries, with and without empty rows there
        "span_aligned": [SPAN, SPAN, 0, SPAN, 2 * SPAN, 0, 0, SPAN - 1, 1, SPAN + 1, SPAN - 1],
        # empty rows inside spans, in front and at the end
        "empties": [0, 0, 100, 0, 200, 0, 0, 0, 3000, 0, 5000, 0, 17, 0],
        # lengths that change between chunks of 32 rows (the producer's register chunks)
        "mixed": list(rng.integers(1, 700, 400)),
        # one start per lane group and odd lengths
        "odd": [147] * 300 + [27] * 500 + [1153] * 20,
        # more than 64 rows per span for many spans (rows beyond the two register chunks)
        "rows_of_24": [24] * 3000,
    }
    return out


def make(lengths, seed):
    rng = np.random.default_rng(seed)
    lengths = [int(v) for v in lengths]
    total = int(sum(lengths))
    x = rng.laplace(0, 0.05, total).astype(np.float32)
    scale = np.repeat(10.0 ** rng.uniform(-2, 1, len(lengths)), lengths).astype(np.float32)
    x *= scale
    ro = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
    return x, ro


@pytest.mark.parametrize("name", sorted(layouts()))
def test_absmax_and_minmax(pwlq, oracle, name):
    x, ro = make(layouts()[name], 5)
    m = pwlq.absmax(dev(x), row_offsets=dev(ro))
    assert np.array_equal(np_(m), oracle.absmax(x, ro))
    y = x + np.float32(0.125)
    lo, hi = pwlq.minmax(dev(y), row_offsets=dev(ro))
    olo, ohi = oracle.minmax(y, ro)
    assert np.array_equal(np_(lo), olo) and np.array_equal(np_(hi), ohi)
    assert pwlq.device_status() == 0


@pytest.mark.parametrize("bits,layout", [(3, 1), (4, 1), (8, 0)])
@pytest.mark.parametrize("name", sorted(layouts()))
def test_quantize_dequantize(pwlq, oracle, name, bits, layout):
    x, ro = make(layouts()[name], 7)
    total = x.size
    om = oracle.absmax(x, ro)
    rng = np.random.default_rng(3)
    p = (om * rng.uniform(0.05, 1.0, om.size)).astype(np.float32)
    p[::7] = om[::7]                                   # p = m: empty tail
    codes, mask, fake = pwlq.quantize(dev(x), bits, dev(om), dev(p), layout=layout,
                                      row_offsets=dev(ro), want_fake=True)
    oc, ok, of = oracle.quantize(x, bits, om, p, layout=layout, row_offsets=ro)
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(mask), ok)
    assert np_(fake).tobytes() == of.tobytes()
    codes2, mask2, none = pwlq.quantize(dev(x), bits, dev(om), dev(p), layout=layout,
                                        row_offsets=dev(ro), want_fake=False)
    assert none is None
    assert np.array_equal(np_(codes2), oc) and np.array_equal(np_(mask2), ok)
    y = pwlq.dequantize(codes, mask, bits, dev(om), dev(p), layout=layout, row_offsets=dev(ro))
    assert np_(y).tobytes() == of.tobytes()
    assert total == y.numel()
    assert pwlq.device_status() == 0


@pytest.mark.parametrize("C,n", [(5000, 1), (700, 7), (600, 8), (520, 9), (3, 4095), (3, 4096),
                                 (3, 4097), (2, 65535), (2, 65536), (2, 65537), (1, 300001)])
def test_dense_rows_around_the_span(pwlq, oracle, C, n):
    """Dense rows below, at and above one span and sixteen spans (where dequantize changes kernel)."""
    rng = np.random.default_rng(C + n)
    x = (rng.standard_normal((C, n)) * rng.uniform(0.01, 3.0, (C, 1))).astype(np.float32)
    m = pwlq.absmax(dev(x))
    om = oracle.absmax(x)
    assert np.array_equal(np_(m), om)
    p = (om * np.float32(0.3)).astype(np.float32)
    codes, mask, fake = pwlq.quantize(dev(x), 4, m, dev(p), layout=1, want_fake=True)
    oc, ok, of = oracle.quantize(x, 4, om, p, layout=1)
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(mask), ok)
    assert np_(fake).tobytes() == of.tobytes()
    y = pwlq.dequantize(codes, mask, 4, m, dev(p), C=C, n=n, layout=1)
    assert np_(y).tobytes() == of.tobytes()
    assert pwlq.device_status() == 0


# ---------------------------------------------------------------- maps built once per layout
@pytest.mark.parametrize("bits,layout", [(3, 1), (8, 0)])
@pytest.mark.parametrize("name", sorted(layouts()))
def test_calls_with_prebuilt_maps_match_the_oracle(pwlq, oracle, name, bits, layout):
    """pwlq_rowmap_build once, then abs-max, quantize (with and without the reconstructed
    values) and dequantize through the *_mapped entry points: bit for bit the oracle's results."""
    x, ro = make(layouts()[name], 9)
    total, C = x.size, ro.size - 1
    dro = dev(ro)
    rowmap = pwlq.rowmap_build(C, total, row_offsets=dro)
    assert rowmap.numel() >= pwlq.rowmap_bytes(total)
    m = pwlq.absmax(dev(x), row_offsets=dro, rowmap=rowmap)
    om = oracle.absmax(x, ro)
    assert np.array_equal(np_(m), om)
    rng = np.random.default_rng(4)
    p = (om * rng.uniform(0.05, 1.0, om.size)).astype(np.float32)
    p[::5] = om[::5]
    oc, ok, of = oracle.quantize(x, bits, om, p, layout=layout, row_offsets=ro)
    for want_fake in (True, False):
        codes, mask, fake = pwlq.quantize(dev(x), bits, m, dev(p), layout=layout, row_offsets=dro,
                                          want_fake=want_fake, rowmap=rowmap)
        assert np.array_equal(np_(codes), oc) and np.array_equal(np_(mask), ok)
        if want_fake:
            assert np_(fake).tobytes() == of.tobytes()
    y = pwlq.dequantize(codes, mask, bits, m, dev(p), layout=layout, row_offsets=dro, rowmap=rowmap)
    assert np_(y).tobytes() == of.tobytes()
    assert pwlq.device_status() == 0


@pytest.mark.parametrize("C,n", [(5000, 1), (700, 7), (520, 9), (300, 147), (3, 4095), (3, 4097)])
def test_prebuilt_maps_of_dense_rows(pwlq, oracle, C, n):
    rng = np.random.default_rng(C + n)
    x = (rng.standard_normal((C, n)) * rng.uniform(0.01, 3.0, (C, 1))).astype(np.float32)
    dx = dev(x)
    rowmap = pwlq.rowmap_build(C, C * n, n=n, device=dx.device)
    m = pwlq.absmax(dx, rowmap=rowmap)
    om = oracle.absmax(x)
    assert np.array_equal(np_(m), om)
    p = (om * np.float32(0.3)).astype(np.float32)
    codes, mask, fake = pwlq.quantize(dx, 4, m, dev(p), layout=1, want_fake=True, rowmap=rowmap)
    oc, ok, of = oracle.quantize(x, 4, om, p, layout=1)
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(mask), ok)
    assert np_(fake).tobytes() == of.tobytes()
    y = pwlq.dequantize(codes, mask, 4, m, dev(p), C=C, n=n, layout=1, rowmap=rowmap)
    assert np_(y).tobytes() == of.tobytes()
    assert pwlq.device_status() == 0


def test_maps_of_another_layout_are_reported(pwlq):
    """Maps built for other rows make the call a no-op that the device status names."""
    x, ro = make([300] * 40, 1)
    other = np.concatenate([[0], np.cumsum([200] * 40)]).astype(np.int64)
    rowmap = pwlq.rowmap_build(40, int(other[-1]), row_offsets=dev(other))
    assert pwlq.device_status() == 0
    m = torch.full((40,), -1.0, dtype=torch.float32, device="cuda")
    pwlq.absmax(dev(x), row_offsets=dev(ro), rowmap=rowmap, out=m)
    torch.cuda.synchronize()
    assert pwlq.device_status() == 1 << pwlq.ERR_INVALID_ARG
    assert pwlq.device_status() == 0                    # read and cleared
    # too small a buffer is refused on the host
    small = torch.empty(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(Exception):
        pwlq.rowmap_build(40, x.size, row_offsets=dev(ro), out=small)


# ------------------------------------------------- two and three breakpoints on the same layouts
def multi_layouts():
    out = dict(layouts())
    # (layouts whose rows average fewer than 32 values go through the element-wise kernels)
    # around the number of rows a span's stage holds constants for (160): 157 / 163 rows per
    # span, followed by long rows so that the producer / consumer kernels take the layout
    out["rows_of_26_then_long"] = [26] * 700 + [6000] * 30
    out["rows_of_25_then_long"] = [25] * 700 + [6000] * 30
    # spans without a usable map (too many rows, empty rows) between long rows
    out["slow_spans_between_long_rows"] = [1] * 300 + [9] * 400 + [4096 * 5] + [3] * 100 + [0, 0, 20000]
    # long rows with short ones in between, a tail that is not a multiple of anything
    out["long_and_short"] = [9000, 13, 4096 * 3, 40, 41, 42, 12289, 5]
    return out


def breakpoints(om, nbp, seed):
    rng = np.random.default_rng(seed)
    r = np.sort(rng.uniform(0.03, 1.0, (om.size, nbp)), axis=1)
    r[::4, nbp - 1] = 1.0                              # last breakpoint = m: the last region is empty
    return (om[:, None] * r).astype(np.float32)


@pytest.mark.parametrize("bits,layout", [(3, 1), (4, 0), (8, 0)])
@pytest.mark.parametrize("name", sorted(multi_layouts()))
def test_quantize2_dequantize2_layouts(pwlq, oracle, name, bits, layout):
    x, ro = make(multi_layouts()[name], 21)
    om = oracle.absmax(x, ro)
    om[3::11] = 0.0                                    # rows delivered as zeros
    p = breakpoints(om, 2, 5)
    p1, p2 = np.ascontiguousarray(p[:, 0]), np.ascontiguousarray(p[:, 1])
    oc, orr, of = oracle.quantize2(x, bits, om, p1, p2, layout=layout, row_offsets=ro)
    for want_fake in (True, False):
        codes, reg, fake = pwlq.quantize2(dev(x), bits, dev(om), dev(p1), dev(p2), layout=layout,
                                          row_offsets=dev(ro), want_fake=want_fake)
        assert np.array_equal(np_(codes), oc) and np.array_equal(np_(reg), orr)
        assert (fake is None) if not want_fake else np_(fake).tobytes() == of.tobytes()
    y = pwlq.dequantize2(codes, reg, bits, dev(om), dev(p1), dev(p2), layout=layout,
                         row_offsets=dev(ro))
    assert np_(y).tobytes() == of.tobytes()
    assert pwlq.device_status() == 0


@pytest.mark.parametrize("bits,layout", [(2, 1), (4, 1), (6, 0)])
@pytest.mark.parametrize("name", sorted(multi_layouts()))
def test_quantize3_dequantize3_layouts(pwlq, oracle, name, bits, layout):
    x, ro = make(multi_layouts()[name], 22)
    om = oracle.absmax(x, ro)
    om[5::13] = 0.0
    p = breakpoints(om, 3, 6)
    oc, orr, of = oracle.quantize3(x, bits, om, p, layout=layout, row_offsets=ro)
    for want_fake in (True, False):
        codes, reg, fake = pwlq.quantize3(dev(x), bits, dev(om), dev(p), layout=layout,
                                          row_offsets=dev(ro), want_fake=want_fake)
        assert np.array_equal(np_(codes), oc) and np.array_equal(np_(reg), orr)
        assert (fake is None) if not want_fake else np_(fake).tobytes() == of.tobytes()
    y = pwlq.dequantize3(codes, reg, bits, dev(om), dev(p), layout=layout, row_offsets=dev(ro))
    assert np_(y).tobytes() == of.tobytes()
    assert pwlq.device_status() == 0


@pytest.mark.parametrize("C,n", [(600, 8), (3, 4095), (3, 4097), (2, 65537), (1, 300001), (380, 11)])
def test_multi_breakpoint_dense_rows_around_the_span(pwlq, oracle, C, n):
    rng = np.random.default_rng(C + n)
    x = (rng.standard_normal((C, n)) * rng.uniform(0.01, 3.0, (C, 1))).astype(np.float32)
    om = oracle.absmax(x)
    p = breakpoints(om, 3, 7)
    oc, orr, of = oracle.quantize3(x, 4, om, p, layout=1)
    codes, reg, fake = pwlq.quantize3(dev(x), 4, dev(om), dev(p), layout=1, want_fake=True)
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(reg), orr)
    assert np_(fake).tobytes() == of.tobytes()
    y = pwlq.dequantize3(codes, reg, 4, dev(om), dev(p), C=C, n=n, layout=1)
    assert np_(y).tobytes() == of.tobytes()
    p1, p2 = np.ascontiguousarray(p[:, 0]), np.ascontiguousarray(p[:, 1])
    oc, orr, of = oracle.quantize2(x, 4, om, p1, p2, layout=1)
    codes, reg, fake = pwlq.quantize2(dev(x), 4, dev(om), dev(p1), dev(p2), layout=1, want_fake=True)
    assert np.array_equal(np_(codes), oc) and np.array_equal(np_(reg), orr)
    assert np_(fake).tobytes() == of.tobytes()
    y = pwlq.dequantize2(codes, reg, 4, dev(om), dev(p1), dev(p2), C=C, n=n, layout=1)
    assert np_(y).tobytes() == of.tobytes()
    assert pwlq.device_status() == 0
