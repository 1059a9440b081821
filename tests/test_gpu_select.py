"""GPU parity of the analytic breakpoint selection (Sec. 3.3 / Sec. 5.1) against the oracle."""
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


def compare(pwlq, oracle, x, model, row_offsets=None, max_n=None):
    m = oracle.absmax(x, row_offsets)
    want_p, want_scale = oracle.select_analytic(x, m, model, row_offsets=row_offsets)
    p, scale = pwlq.select_analytic(dev(x), dev(m), model,
                                    row_offsets=None if row_offsets is None else dev(row_offsets),
                                    max_n=max_n, want_scale=True)
    torch.cuda.synchronize()
    p, scale = p.cpu().numpy(), scale.cpu().numpy()
    # binary64 sums in another order: a few ulps of binary64, invisible after rounding to binary32
    # except at a rounding boundary
    assert np.allclose(scale, want_scale.astype(np.float32), rtol=2e-7, atol=0)
    assert np.allclose(p, want_p, rtol=1e-6, atol=0)
    assert np.all((p > 0) | (m == 0)) and np.all(p <= m * np.float32(0.5) * (1 + 1e-6))


@pytest.mark.parametrize("model", [0, 1, 2])
def test_select_against_scipy_and_the_closed_form(pwlq, model):
    """The GPU's breakpoints against solvers that share nothing with it or with the oracle: SciPy's
    Brent root finder on Eq. 9 written with SciPy's CDF / PDF (models 1, 2), math.log for the
    Sec. 5.1 closed form (model 0); the scale against NumPy's binary64 moments."""
    import math
    from scipy.optimize import brentq
    from scipy.stats import laplace, norm
    rng = np.random.default_rng(91 + model)
    scales = np.array([0.003, 0.02, 0.05, 0.4, 1.0, 1.3, 7.0, 0.05])
    n = 6000
    gen = rng.laplace if model == 2 else rng.normal
    x = np.stack([gen(0, s, n) for s in scales]).astype(np.float32)
    x[-1] = rng.uniform(-1, 1, n).astype(np.float32)        # flatter than either model
    x64 = x.astype(np.float64)
    m = np.abs(x).max(axis=1)
    p, scale = pwlq.select_analytic(dev(x), dev(m), model, want_scale=True)
    torch.cuda.synchronize()
    p, scale = p.cpu().numpy().astype(np.float64), scale.cpu().numpy().astype(np.float64)
    fit = np.mean(np.abs(x64), axis=1) if model == 2 else np.sqrt(np.mean(x64 ** 2, axis=1))
    assert np.allclose(scale, fit, rtol=2e-7, atol=0)
    inside = 0
    for c in range(len(scales)):
        mc, sc = float(m[c]), float(fit[c])
        if model == 0:
            want = min(sc * math.log(0.8614 * mc / sc + 0.6079), 0.5 * mc)
        else:
            d = (laplace if model == 2 else norm)(0, sc)
            g = lambda t: 2 * mc * d.cdf(t) - (2 * mc - t + mc * (mc - 2 * t) * d.pdf(t))
            if g(0.5 * mc) <= 0:
                want = 0.5 * mc
            else:
                want = brentq(g, 1e-12 * mc, 0.5 * mc, xtol=1e-15, rtol=1e-14)
                inside += 1
        assert math.isclose(p[c], want, rel_tol=1e-6), (c, p[c], want)
    assert model == 0 or inside >= 5                        # real roots were compared, not only bounds


@pytest.mark.parametrize("model", [0, 1, 2])
def test_select_ragged_rows(pwlq, oracle, model):
    w = W.small_mixed(seed=31 + model)
    compare(pwlq, oracle, w.x, model, w.row_offsets, int(np.diff(w.row_offsets).max()))


@pytest.mark.parametrize("model", [0, 1, 2])
@pytest.mark.parametrize("C,n", [(1, 36864), (3, 20001), (300, 9), (7, 8192), (2, 1)])
def test_select_dense(pwlq, oracle, model, C, n):
    rng = np.random.default_rng(C * 7 + n + model)
    x = (rng.laplace(0, 0.02, (C, n)) if model == 2 else rng.normal(0, 0.05, (C, n))).astype(np.float32)
    if C > 1:
        x[-1] = 0.0                                   # an all-zero row: p = 0
    compare(pwlq, oracle, x, model)


def test_select_resnet50_feeds_the_quantizer(pwlq, oracle):
    """The analytic p of every ResNet-50-shaped row, then codes and reconstructed values from it
    against the oracle's quantizer with the same p."""
    w = W.resnet50()
    max_n = int(np.diff(w.row_offsets).max())
    compare(pwlq, oracle, w.x, 0, w.row_offsets, max_n)
    x, ro = dev(w.x), dev(w.row_offsets)
    m = pwlq.absmax(x, row_offsets=ro)
    p, _ = pwlq.select_analytic(x, m, pwlq.MODEL_GAUSS_ROOT, row_offsets=ro, max_n=max_n)
    codes, mask, fake = pwlq.quantize(x, 4, m, p, layout=pwlq.CODES_PACKED, row_offsets=ro,
                                      want_fake=True)
    torch.cuda.synchronize()
    oc, om, of = oracle.quantize(w.x, 4, m.cpu().numpy(), p.cpu().numpy(), layout=1,
                                 row_offsets=w.row_offsets)
    assert np.array_equal(codes.cpu().numpy(), oc) and np.array_equal(mask.cpu().numpy(), om)
    assert fake.cpu().numpy().tobytes() == of.tobytes()
