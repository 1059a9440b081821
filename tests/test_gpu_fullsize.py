"""Parity at the full benchmark sizes, in the launch configuration bench.py times (ragged rows,
ranges passed in, packed codes).  Where the oracle cannot do everything in seconds, it checks a
stratified sample of rows (or of candidates) one by one, and properties that hold at any size
cover the rest: exact ranges, p = m * ratio[idx], err = SSE[idx] = min SSE, and codes / region
bits / reconstructed values of every single value against the oracle's quantizer."""
import numpy as np
import pytest
import torch

from gpu_util import check_search, dev, oracle_sse_over_candidates
from paper_2002_00104_b200 import workloads as W

pytestmark = [pytest.mark.gpu,
              pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]


@pytest.fixture(scope="module")
def pwlq():
    from paper_2002_00104_b200 import pwlq as _p
    _p.load_library()
    return _p


def run_path(pwlq, w, bits=None, K=None, want_sse=True):
    bits = bits or w.bits
    K = K or w.K
    ratios = W.ratio_grid(K)
    x = dev(w.x)
    n = w.uniform_n()
    if n is not None:
        x, ro = x.view(w.C, n), None
    else:
        ro = dev(w.row_offsets)
    max_n = int(np.diff(w.row_offsets).max())
    m = pwlq.absmax(x, row_offsets=ro)
    s = pwlq.search(x, bits, dev(ratios), m=m, row_offsets=ro, max_n=max_n, want_sse=want_sse)
    codes, mask, _ = pwlq.quantize(x, bits, m, s["p"], layout=pwlq.CODES_PACKED, row_offsets=ro)
    y = pwlq.dequantize(codes, mask, bits, m, s["p"], C=w.C, n=n, layout=pwlq.CODES_PACKED,
                        row_offsets=ro)
    torch.cuda.synchronize()
    assert pwlq.search_status(s["workspace"]) == 0 and pwlq.device_status() == 0
    out = {k: s[k].cpu().numpy() for k in ("p", "err", "idx")}
    out["sse"] = s["sse"].cpu().numpy() if want_sse else None
    out.update(m=m.cpu().numpy(), codes=codes.cpu().numpy(), mask=mask.cpu().numpy(),
               y=y.cpu().numpy(), ratios=ratios, bits=bits, K=K)
    return out


def check_all_rows(oracle, w, g):
    """Checks that need no per-candidate oracle work: every row, every value."""
    m = oracle.absmax(w.x, w.row_offsets)
    assert np.array_equal(g["m"], m)
    want_p = (m * g["ratios"][g["idx"]]).astype(np.float32)
    want_p[m == 0] = 0
    assert np.array_equal(g["p"], want_p)
    if g["sse"] is not None:
        rows = np.arange(w.C)
        mins = g["sse"].min(axis=1)
        assert np.array_equal(g["sse"][rows, g["idx"]], mins)          # the minimum ...
        assert np.array_equal(g["idx"], np.argmin(g["sse"], axis=1)) or \
            np.all(g["sse"][rows, np.argmin(g["sse"], axis=1)] == mins)
        assert np.allclose(g["err"], mins, rtol=2e-7, atol=0)          # ... is what err reports
    oc, om, of = oracle.quantize(w.x, g["bits"], m, g["p"], layout=1, row_offsets=w.row_offsets)
    assert np.array_equal(g["codes"], oc)
    assert np.array_equal(g["mask"], om)
    assert g["y"].tobytes() == of.tobytes()
    return m


def check_sampled_rows(oracle, w, g, rows, m):
    lens = np.diff(w.row_offsets)
    xs = np.concatenate([w.x[w.row_offsets[c]:w.row_offsets[c + 1]] for c in rows])
    ro = np.concatenate([[0], np.cumsum(lens[rows])]).astype(np.int64)
    ora = oracle.search(xs, g["bits"], g["ratios"], m=m[rows], row_offsets=ro)
    sub = {k: g[k][rows] for k in ("p", "err", "idx", "sse")}
    return check_search(sub, ora, g["ratios"], m[rows], lens[rows])


def stratified_rows(w, per_length, every):
    """Every `every`-th row plus the first `per_length` rows of each distinct length."""
    lens = np.diff(w.row_offsets)
    rows = set(range(0, w.C, every))
    for n in np.unique(lens):
        rows.update(np.nonzero(lens == n)[0][:per_length].tolist())
    return np.array(sorted(rows))


def test_single_conv_full(pwlq, oracle):
    w = W.single_conv()
    g = run_path(pwlq, w)
    m = check_all_rows(oracle, w, g)
    assert check_sampled_rows(oracle, w, g, np.array([0]), m) == 0


def test_resnet50_full(pwlq, oracle):
    w = W.resnet50()
    g = run_path(pwlq, w)
    m = check_all_rows(oracle, w, g)
    differ = check_sampled_rows(oracle, w, g, stratified_rows(w, 3, 60), m)
    assert differ <= 2          # near-ties only (check_search has already vetted each of them)


def test_mobilenetv2_full(pwlq, oracle):
    w = W.mobilenetv2()
    g = run_path(pwlq, w)
    m = check_all_rows(oracle, w, g)
    check_sampled_rows(oracle, w, g, stratified_rows(w, 4, 25), m)


def test_relu_activation_full(pwlq, oracle):
    """One row of 25.7 M values, K = 1024: every one of the 1024 per-candidate sums against the
    oracle's binary64 sums (the sum over 25.7 M terms with a range of 10^5 .. 10^6 is where
    accumulation error would show), the oracle fanned over the candidates on the host threads."""
    w = W.relu_activation()
    g = run_path(pwlq, w)
    m = check_all_rows(oracle, w, g)
    sse_o = oracle_sse_over_candidates(oracle, w.x, w.bits, g["ratios"], m)
    assert sse_o.shape == (w.K,)
    ora = {"sse64": sse_o[None, :], "idx": np.array([int(np.argmin(sse_o))])}
    sub = {k: g[k][:1] for k in ("p", "err", "idx", "sse")}
    check_search(sub, ora, g["ratios"], m[:1], w.total)


@pytest.mark.parametrize("bits", [3, 4, 6, 8])
@pytest.mark.parametrize("K", [64, 256, 1024])
def test_laplace_matrix_sweep(pwlq, oracle, bits, K):
    w = W.laplace_matrix()
    g = run_path(pwlq, w, bits=bits, K=K)
    m = check_all_rows(oracle, w, g)
    check_sampled_rows(oracle, w, g, np.arange(5, w.C, 64), m)          # 64 rows per (b, K)


# ------------------------------------------------------------ host-buffer entry point, pipelined
@pytest.mark.parametrize("layout,bits", [(1, 4), (0, 6)])
def test_encode_host_in_several_runs_equals_the_resident_path(pwlq, oracle, layout, bits):
    """A tensor large enough to be cut into runs of rows whose copies and kernels overlap, with row
    lengths that put most row starts off a multiple of 8: the outputs must equal those of the four
    device calls on the whole tensor, and sampled rows must equal the oracle."""
    rng = np.random.default_rng(77)
    lengths = np.tile(np.array([147, 1001, 64, 4608, 9, 2304, 33], np.int64), 1800)
    ro = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
    total, C, max_n, K = int(ro[-1]), lengths.size, int(lengths.max()), 32
    assert total > 8 * (1 << 20)
    x = rng.laplace(0, 0.03, total).astype(np.float32)
    ratios = W.ratio_grid(K)
    hx, hro = torch.from_numpy(x).pin_memory(), torch.from_numpy(ro).pin_memory()
    cb = (total + 1) // 2 if (layout == 1 and bits <= 4) else total
    out = {"m": torch.empty(C, dtype=torch.float32).pin_memory(),
           "p": torch.empty(C, dtype=torch.float32).pin_memory(),
           "err": torch.empty(C, dtype=torch.float32).pin_memory(),
           "idx": torch.empty(C, dtype=torch.int32).pin_memory(),
           "codes": torch.empty(cb, dtype=torch.uint8).pin_memory(),
           "mask": torch.empty((total + 7) // 8, dtype=torch.uint8).pin_memory()}
    scratch = torch.empty(pwlq.encode_host_scratch_bytes(C, total, max_n, K), dtype=torch.uint8,
                          device="cuda")
    for _ in range(2):                                # the second call reuses streams and scratch
        pwlq.encode_host(hx, hro, C, max_n, bits, torch.from_numpy(ratios).pin_memory(), out,
                         layout, scratch)
    torch.cuda.synchronize()
    xd, rod = hx.cuda(), hro.cuda()
    m = pwlq.absmax(xd, row_offsets=rod)
    s = pwlq.search(xd, bits, torch.from_numpy(ratios).cuda(), m=m, row_offsets=rod, max_n=max_n)
    codes, mask, _ = pwlq.quantize(xd, bits, m, s["p"], layout=layout, row_offsets=rod)
    torch.cuda.synchronize()
    assert torch.equal(out["m"], m.cpu()) and torch.equal(out["idx"], s["idx"].cpu())
    assert torch.equal(out["p"], s["p"].cpu()) and torch.equal(out["err"], s["err"].cpu())
    assert torch.equal(out["codes"], codes.cpu()) and torch.equal(out["mask"], mask.cpu())
    assert pwlq.device_status() == 0
    for c in rng.choice(C, 40, replace=False):
        xr = x[ro[c]:ro[c + 1]]
        om = oracle.absmax(xr)
        assert out["m"][c].item() == om[0]
        oc, _, _ = oracle.quantize(xr, bits, om, [out["p"][c].item()], layout=0)
        got = codes.cpu().numpy()
        if layout == 1 and bits <= 4:
            idx = np.arange(ro[c], ro[c + 1])
            got_row = (got[idx >> 1] >> ((idx & 1) * 4)) & 0xF
        else:
            got_row = got[ro[c]:ro[c + 1]]
        assert np.array_equal(got_row, oc)


@pytest.mark.parametrize("name", ["resnet50", "mobilenetv2"])
def test_prebuilt_row_maps_at_full_size(pwlq, oracle, name):
    """The *_mapped calls on the benchmark's ragged layouts, repeated as the streaming leg of the
    benchmark repeats them (two copies back to back): every range, code byte, region byte and
    reconstructed value against the oracle."""
    w = getattr(W, name)()
    copies = 2
    x = np.tile(w.x, copies)
    ro = np.concatenate([w.row_offsets[:-1] + k * w.total for k in range(copies)] +
                        [np.array([copies * w.total])]).astype(np.int64)
    C, total = ro.size - 1, x.size
    xd, rod = dev(x), dev(ro)
    rowmap = pwlq.rowmap_build(C, total, row_offsets=rod)
    m = pwlq.absmax(xd, row_offsets=rod, rowmap=rowmap)
    om = oracle.absmax(x, ro)
    assert np.array_equal(m.cpu().numpy(), om)
    p = (om * np.float32(0.3)).astype(np.float32)
    codes, mask, fake = pwlq.quantize(xd, w.bits, m, dev(p), layout=pwlq.CODES_PACKED,
                                      row_offsets=rod, want_fake=True, rowmap=rowmap)
    y = pwlq.dequantize(codes, mask, w.bits, m, dev(p), layout=pwlq.CODES_PACKED, row_offsets=rod,
                        rowmap=rowmap)
    torch.cuda.synchronize()
    assert pwlq.device_status() == 0
    oc, ok, of = oracle.quantize(x, w.bits, om, p, layout=1, row_offsets=ro)
    assert np.array_equal(codes.cpu().numpy(), oc) and np.array_equal(mask.cpu().numpy(), ok)
    assert fake.cpu().numpy().tobytes() == of.tobytes()
    assert y.cpu().numpy().tobytes() == of.tobytes()
