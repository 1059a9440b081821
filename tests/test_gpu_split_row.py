"""One row cut into pieces (the multi-GPU form of a per-layer tensor, run here piece by piece on
one GPU through the C ABI): ranges of the pieces -> their maximum; per-candidate binary64 sums of
every piece under the common range (pwlq_search_partial); the pieces' sums added in order and the
first minimum taken (pwlq_search_finish).  Checked against the oracle on the whole row and against
the one-call search."""
import numpy as np
import pytest
import torch

from gpu_util import check_search, dev
from paper_2002_00104_b200 import shard, workloads as W

pytestmark = [pytest.mark.gpu,
              pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]


@pytest.fixture(scope="module")
def pwlq():
    from paper_2002_00104_b200 import pwlq as _p
    _p.load_library()
    return _p


def split_search(pwlq, x, bits, ratios, world, unsigned=False):
    """x: numpy [C, n].  Returns (gpu result dict of numpy arrays, m, lo or None, sums [world,C,K])."""
    C, n = x.shape
    r = dev(ratios)
    pieces = [dev(np.ascontiguousarray(x[:, b:e])) for b, e in shard.partition_elements(n, world)
              if e > b]
    if unsigned:
        los, his = zip(*[pwlq.minmax(p) for p in pieces])
        lo = torch.stack(los).min(dim=0).values
        m = torch.stack(his).max(dim=0).values
    else:
        lo = None
        m = torch.stack([pwlq.absmax(p) for p in pieces]).max(dim=0).values   # the all-reduce(max)
    sums = torch.stack([pwlq.search_partial(p, bits, r, m, lo=lo)[0] for p in pieces])
    out = pwlq.search_finish(sums, m, r, lo=lo, want_sse=True)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    g = {k: out[k].cpu().numpy() for k in ("p", "err", "idx", "sse")}
    return g, m.cpu().numpy(), None if lo is None else lo.cpu().numpy(), sums.cpu().numpy()


@pytest.mark.parametrize("world", [2, 3, 8])
def test_single_conv_row_in_pieces(pwlq, oracle, world):
    w = W.single_conv()
    ratios = W.ratio_grid(w.K)
    g, m, _, sums = split_search(pwlq, w.x[None], w.bits, ratios, world)
    assert np.array_equal(m, oracle.absmax(w.x))
    ora = oracle.search(w.x, w.bits, ratios, m=m)
    assert check_search(g, ora, ratios, m, w.total) == 0
    # every piece's sums against the oracle on that piece under the common range
    for (b, e), s in zip(shard.partition_elements(w.total, world), sums):
        want = oracle.search(w.x[b:e], w.bits, ratios, m=m)["sse64"]
        assert np.allclose(s, want, rtol=1e-5, atol=(e - b) * (2.0 ** -23 * m[0]) ** 2)
    # the one-call search agrees (same index; sums equal up to the order of the binary64 adds)
    one = pwlq.search(dev(w.x[None]), w.bits, dev(ratios), want_sse=True)
    torch.cuda.synchronize()
    assert one["idx"].cpu().numpy().tolist() == g["idx"].tolist()
    assert np.allclose(one["sse"].cpu().numpy(), g["sse"], rtol=3e-7, atol=0)


@pytest.mark.parametrize("bits,K,C,n", [(4, 64, 3, 20001), (3, 256, 5, 777), (8, 100, 2, 50000),
                                        (4, 1024, 1, 9), (4, 33, 4, 64)])
def test_matrix_rows_in_column_pieces(pwlq, oracle, bits, K, C, n):
    rng = np.random.default_rng(bits * 100 + K)
    x = rng.laplace(0, 0.05, (C, n)).astype(np.float32)
    if C > 2:
        x[1] = 0.0                                        # an all-zero row
    ratios = W.ratio_grid(K)
    g, m, _, _ = split_search(pwlq, x, bits, ratios, 2)
    assert np.array_equal(m, oracle.absmax(x))
    ora = oracle.search(x, bits, ratios, m=m)
    check_search(g, ora, ratios, m, n)


def test_one_sided_row_in_pieces(pwlq, oracle):
    rng = np.random.default_rng(12)
    x = np.maximum(rng.standard_normal((2, 30000)), 0).astype(np.float32)
    ratios = W.ratio_grid(128)
    g, hi, lo, _ = split_search(pwlq, x, 4, ratios, 3, unsigned=True)
    olo, ohi = oracle.minmax(x)
    assert np.array_equal(lo, olo) and np.array_equal(hi, ohi)
    ora = oracle.search_u(x, 4, ratios, olo, ohi)
    check_search(g, ora, ratios, ohi - olo, 30000)


def test_finish_reports_a_nonfinite_range_and_is_reproducible(pwlq):
    x = dev(np.linspace(-1, 1, 4096, dtype=np.float32)[None])
    r = dev(W.ratio_grid(16))
    m = torch.tensor([float("inf")], device="cuda")
    sums, _ = pwlq.search_partial(x, 4, r, m)
    out = pwlq.search_finish(sums[None], m, r)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 1 << pwlq.ERR_NONFINITE and int(out["idx"].item()) == 0
    m = pwlq.absmax(x)
    a = pwlq.search_partial(x, 4, r, m)[0].clone()
    b = pwlq.search_partial(x, 4, r, m)[0]
    assert torch.equal(a, b)
