"""Two and three breakpoints at the benchmark's full size: the rows of the ResNet-50 workload
(ragged, packed codes), every code, region index and delivered value against the oracle."""
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


@pytest.mark.parametrize("name", ["resnet50", "mobilenetv2"])
def test_three_and_two_breakpoints_at_full_size(pwlq, oracle, name):
    w = getattr(W, name)()
    x, ro = w.x, w.row_offsets
    bits = w.bits
    m = oracle.absmax(x, ro)
    p = (m[:, None] * np.array([0.2, 0.45, 0.75], dtype=np.float32)[None, :]).astype(np.float32)
    xd, rod, md, pd = dev(x), dev(ro), dev(m), dev(p)
    codes, reg, fake = pwlq.quantize3(xd, bits, md, pd, layout=1, row_offsets=rod, want_fake=True)
    y = pwlq.dequantize3(codes, reg, bits, md, pd, layout=1, row_offsets=rod)
    torch.cuda.synchronize()
    oc, orr, of = oracle.quantize3(x, bits, m, p, layout=1, row_offsets=ro)
    assert np.array_equal(codes.cpu().numpy(), oc) and np.array_equal(reg.cpu().numpy(), orr)
    assert fake.cpu().numpy().tobytes() == of.tobytes()
    assert y.cpu().numpy().tobytes() == of.tobytes()
    p1, p2 = np.ascontiguousarray(p[:, 0]), np.ascontiguousarray(p[:, 2])
    codes, reg, _ = pwlq.quantize2(xd, bits, md, dev(p1), dev(p2), layout=1, row_offsets=rod)
    y = pwlq.dequantize2(codes, reg, bits, md, dev(p1), dev(p2), layout=1, row_offsets=rod)
    torch.cuda.synchronize()
    oc, orr, of = oracle.quantize2(x, bits, m, p1, p2, layout=1, row_offsets=ro)
    assert np.array_equal(codes.cpu().numpy(), oc) and np.array_equal(reg.cpu().numpy(), orr)
    assert y.cpu().numpy().tobytes() == of.tobytes()
    assert pwlq.device_status() == 0
