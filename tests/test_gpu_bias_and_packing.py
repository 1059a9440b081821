"""GPU parity of bias correction, the corrected dequantize and the dense bit stream."""
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
    return None if t is None else t.cpu().numpy()


def check_bias(xi, beta, oxi, obeta, scale):
    """xi, beta are binary64 results rounded to binary32 on both sides; the one-pass and the
    two-pass variance differ by rounding noise only."""
    assert np.allclose(xi, oxi, rtol=2e-6, atol=0)
    assert np.allclose(beta, obeta, rtol=0, atol=2e-6 * scale)


@pytest.mark.parametrize("bits", [3, 4, 8])
@pytest.mark.parametrize("C,n", [(6, 9), (4, 700), (3, 8192), (2, 30001)])
def test_bias_correction_dense(pwlq, oracle, bits, C, n):
    rng = np.random.default_rng(bits * 10 + n)
    x = (rng.laplace(0, 0.05, (C, n)) + rng.uniform(-0.02, 0.02, (C, 1))).astype(np.float32)
    m = oracle.absmax(x)
    p = (m * rng.uniform(0.1, 0.5, C)).astype(np.float32)
    xi, beta = pwlq.bias_correction(dev(x), bits, dev(m), dev(p))
    oxi, obeta = oracle.bias_correction(x, bits, m, p)
    check_bias(np_(xi), np_(beta), oxi, obeta, float(np.abs(x).max()))


def test_bias_correction_ragged_and_degenerate_rows(pwlq, oracle):
    w = W.small_mixed(seed=23)
    rows = [w.x[w.row_offsets[c]:w.row_offsets[c + 1]] for c in range(w.C)]
    rows.insert(1, np.zeros(0, np.float32))                       # empty
    rows.insert(3, np.full(40, 0.3, np.float32))                  # constant
    rows.insert(5, np.zeros(17, np.float32))                      # zeros
    x = np.concatenate(rows).astype(np.float32)
    ro = np.concatenate([[0], np.cumsum([r.size for r in rows])]).astype(np.int64)
    m = oracle.absmax(x, ro)
    p = (m * np.float32(0.3)).astype(np.float32)
    xi, beta = pwlq.bias_correction(dev(x), 4, dev(m), dev(p), row_offsets=dev(ro),
                                    max_n=int(np.diff(ro).max()))
    oxi, obeta = oracle.bias_correction(x, 4, m, p, row_offsets=ro)
    check_bias(np_(xi), np_(beta), oxi, obeta, float(np.abs(x).max()))
    assert np_(xi)[[1, 3, 5]].tolist() == [1.0, 1.0, 1.0]
    assert np_(beta)[[1, 5]].tolist() == [0.0, 0.0]


@pytest.mark.parametrize("bits,layout", [(3, 1), (4, 0), (8, 0)])
def test_dequantize_bc_is_bit_exact(pwlq, oracle, bits, layout):
    w = W.small_mixed(seed=29)
    x, ro = w.x, w.row_offsets
    m = oracle.absmax(x, ro)
    p = (m * np.float32(0.25)).astype(np.float32)
    oxi, obeta = oracle.bias_correction(x, bits, m, p, row_offsets=ro)
    oc, om, _ = oracle.quantize(x, bits, m, p, layout=layout, row_offsets=ro)
    y = pwlq.dequantize_bc(dev(oc), dev(om), bits, dev(m), dev(p), dev(oxi), dev(obeta),
                           layout=layout, row_offsets=dev(ro))
    want = oracle.dequantize_bc(oc, om, bits, m, p, oxi, obeta, layout=layout, row_offsets=ro)
    assert np_(y).tobytes() == want.tobytes()
    # dense rows too
    xd = x[:4096].reshape(8, 512)
    md = oracle.absmax(xd)
    pd = (md * np.float32(0.4)).astype(np.float32)
    xi, beta = oracle.bias_correction(xd, bits, md, pd)
    oc, om, _ = oracle.quantize(xd, bits, md, pd, layout=layout)
    y = pwlq.dequantize_bc(dev(oc), dev(om), bits, dev(md), dev(pd), dev(xi), dev(beta), C=8, n=512,
                           layout=layout)
    assert np_(y).tobytes() == oracle.dequantize_bc(oc, om, bits, md, pd, xi, beta, C=8, n=512,
                                                    layout=layout).tobytes()


def test_corrected_rows_keep_mean_and_norm_on_the_device(pwlq):
    """The defining property, end to end on the GPU path."""
    rng = np.random.default_rng(31)
    x = dev(rng.laplace(0, 0.03, (64, 1152)).astype(np.float32))
    m = pwlq.absmax(x)
    out = pwlq.search(x, 4, dev(W.ratio_grid(64)), m=m)
    xi, beta = pwlq.bias_correction(x, 4, m, out["p"])
    codes, mask, _ = pwlq.quantize(x, 4, m, out["p"], layout=1)
    y = pwlq.dequantize_bc(codes, mask, 4, m, out["p"], xi, beta, C=64, n=1152, layout=1)
    y = y.view(64, 1152).double()
    xd = x.double()
    assert torch.allclose(y.mean(dim=1), xd.mean(dim=1), rtol=0, atol=1e-6)
    ny = (y - y.mean(dim=1, keepdim=True)).norm(dim=1)
    nx = (xd - xd.mean(dim=1, keepdim=True)).norm(dim=1)
    assert torch.allclose(ny, nx, rtol=1e-5)


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("total", [1, 8, 31, 32, 1003, 65536 + 5])
def test_dense_stream_pack_and_unpack(pwlq, oracle, bits, total):
    rng = np.random.default_rng(bits * 7 + total)
    codes = rng.integers(0, 2 ** bits, total).astype(np.uint8)
    mask = np.packbits(rng.integers(0, 2, total).astype(np.uint8), bitorder="little")
    s = pwlq.pack_dense(dev(codes), dev(mask), bits)
    want = oracle.pack_dense(codes, mask, bits)
    assert s.numel() == pwlq.dense_bytes(total, bits) == want.size
    assert np.array_equal(np_(s), want)
    c2, m2 = pwlq.unpack_dense(s, total, bits)
    assert np.array_equal(np_(c2), codes) and np.array_equal(np_(m2), mask)


@pytest.mark.parametrize("bits", [3, 4, 8])
def test_dense_stream_from_unaligned_buffers(pwlq, oracle, bits):
    """Buffers that start off the word boundaries take the byte-wise kernels: same stream."""
    total = 5000
    rng = np.random.default_rng(bits)
    codes = rng.integers(0, 2 ** bits, total).astype(np.uint8)
    mask = np.packbits(rng.integers(0, 2, total).astype(np.uint8), bitorder="little")
    cbuf = torch.zeros(total + 16, dtype=torch.uint8, device="cuda")
    mbuf = torch.zeros(mask.size + 16, dtype=torch.uint8, device="cuda")
    cbuf[3:3 + total] = dev(codes)
    mbuf[1:1 + mask.size] = dev(mask)
    want = oracle.pack_dense(codes, mask, bits)
    s = pwlq.pack_dense(cbuf[3:3 + total], mbuf[1:1 + mask.size], bits)
    assert np.array_equal(np_(s), want)
    sbuf = torch.zeros(want.size + 8, dtype=torch.uint8, device="cuda")
    sbuf[1:1 + want.size] = s
    c2, m2 = pwlq.unpack_dense(sbuf[1:1 + want.size], total, bits)
    assert np.array_equal(np_(c2), codes) and np.array_equal(np_(m2), mask)


def test_dense_stream_after_quantize(pwlq, oracle):
    """b = 3 and b = 6 (the cases where b + 1 bits do not fill a byte or a nibble pair evenly)."""
    rng = np.random.default_rng(41)
    x = rng.standard_normal((16, 1000)).astype(np.float32)
    for bits in (3, 6):
        xd = dev(x)
        m = pwlq.absmax(xd)
        p = (m * 0.3).contiguous()
        codes, mask, _ = pwlq.quantize(xd, bits, m, p, layout=0)
        s = pwlq.pack_dense(codes, mask, bits)
        assert s.numel() == (x.size * (bits + 1) + 7) // 8
        assert np.array_equal(np_(s), oracle.pack_dense(np_(codes), np_(mask), bits))
        c2, m2 = pwlq.unpack_dense(s, x.size, bits)
        y1 = pwlq.dequantize(c2, m2, bits, m, p, C=16, n=1000)
        y0 = pwlq.dequantize(codes, mask, bits, m, p, C=16, n=1000)
        assert torch.equal(y0, y1)
