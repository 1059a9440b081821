"""The allocation-free search entry point gives what the ordinary one gives.

Some users of the library cannot allocate device memory at all: their process has handed the
whole GPU to another allocator, or they run inside a loop where cudaMalloc's device-wide
synchronisation is not acceptable, or they are only ever given input and output buffers.
``pwlq_search_noalloc`` serves them with a workspace built into the library.  This test calls it
through the C ABI twice in a row (the built-in workspace is shared and keeps the previous call's
contents, so the second call shows that leftovers do no harm) and compares every output with the
ordinary ``pwlq_search`` on the same inputs; both run the same kernels, so the match is exact.
The file name makes pytest collect it last.
"""
import numpy as np
import pytest
import torch

from paper_2002_00104_b200 import workloads as W

pytestmark = [pytest.mark.gpu,
              pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]


def _cmp(a, b):
    torch.cuda.synchronize()
    for k in ("p", "err", "idx", "sse"):
        assert torch.equal(a[k], b[k]), k


def test_noalloc_matches_search_on_two_calls_in_a_row():
    from paper_2002_00104_b200 import pwlq
    rng = np.random.default_rng(2024)
    # call 1: a single long row cut into several tiles (uses the partial-sum area of the scratch)
    x1 = torch.from_numpy(rng.laplace(0, 0.02, (1, 36864)).astype(np.float32)).cuda()
    r1 = torch.from_numpy(W.ratio_grid(100)).cuda()
    # call 2: many short rows, other K and bit-width, one all-zero row; leaves of call 1 remain
    x2n = rng.standard_normal((37, 147)).astype(np.float32)
    x2n[5] = 0.0
    x2 = torch.from_numpy(x2n).cuda()
    r2 = torch.from_numpy(W.ratio_grid(256)).cuda()
    for x, r, bits in ((x1, r1, 4), (x2, r2, 3), (x1, r1, 4)):
        ref = pwlq.search(x, bits, r, want_sse=True)
        got = pwlq.search_noalloc(x, bits, r, want_sse=True)
        _cmp(got, ref)
        assert int(got["status"].item()) == pwlq.search_status(ref["workspace"]) == 0
    # a caller-supplied range and a non-finite value: status travels through status_out
    x3 = x2.clone()
    x3[3, 3] = float("inf")
    ref = pwlq.search(x3, 4, r2, want_sse=True)
    got = pwlq.search_noalloc(x3, 4, r2, want_sse=True)
    _cmp(got, ref)
    assert int(got["status"].item()) == 1 << pwlq.ERR_NONFINITE


def test_noalloc_rejects_problems_larger_than_its_scratch():
    from paper_2002_00104_b200 import pwlq
    limit = pwlq.noalloc_max_bytes()
    assert limit == 4 << 20
    n = 8192 * 600                                   # 600 tiles x 1024 candidates x 8 B > 4 MiB
    assert pwlq.search_workspace_bytes(1, n, 1024) > limit
    x = torch.zeros((1, n), dtype=torch.float32, device="cuda")
    r = torch.from_numpy(W.ratio_grid(1024)).cuda()
    with pytest.raises(pwlq.PwlqError) as e:
        pwlq.search_noalloc(x, 4, r)
    assert e.value.status == pwlq.ERR_UNSUPPORTED
