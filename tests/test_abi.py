"""The C-ABI library loads without a GPU and exports every symbol the public header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2002_00104_b200 import build, pwlq
    build.build()
    return pwlq.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "pwlq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pwlq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    from paper_2002_00104_b200 import pwlq
    names = declared_symbols()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert names == pwlq.exported_symbols()


def test_status_strings_and_version(lib):
    from paper_2002_00104_b200 import pwlq
    assert pwlq.version().count(".") == 1
    assert pwlq.status_string(0) == "ok"
    assert len({pwlq.status_string(i) for i in range(7)}) == 7


def test_argument_validation_happens_before_any_cuda_call(lib):
    """Invalid arguments are rejected on the host (these calls never reach the CUDA runtime)."""
    from paper_2002_00104_b200 import pwlq
    null = ctypes.c_void_p(0)
    fake = ctypes.c_void_p(0x1000)
    assert lib.pwlq_absmax(null, 1, 1, fake, null) == pwlq.ERR_INVALID_ARG
    assert lib.pwlq_absmax(fake, 0, 1, fake, null) == pwlq.ERR_INVALID_ARG
    assert lib.pwlq_absmax(ctypes.c_void_p(0x1002), 1, 1, fake, null) == pwlq.ERR_INVALID_ARG
    ws = ctypes.c_void_p(0x10000)
    args = [fake, 4, 16, 4, fake, 8, null, fake, fake, fake, null, ws, 1 << 20, null]
    bad_bits = list(args); bad_bits[3] = 9
    assert lib.pwlq_search(*bad_bits) == pwlq.ERR_INVALID_ARG
    bad_k = list(args); bad_k[5] = pwlq.MAX_K + 1
    assert lib.pwlq_search(*bad_k) == pwlq.ERR_UNSUPPORTED
    small_ws = list(args); small_ws[12] = 16
    assert lib.pwlq_search(*small_ws) == pwlq.ERR_WORKSPACE
    assert lib.pwlq_quantize(fake, 1, 8, 4, fake, fake, fake, fake, null, 7, null) == pwlq.ERR_INVALID_ARG
    assert lib.pwlq_dequantize(fake, fake, 1, 8, 1, fake, fake, fake, 0, null) == pwlq.ERR_INVALID_ARG
    assert lib.pwlq_search_workspace_bytes(0, 1, 1) == 0
    assert lib.pwlq_search_workspace_bytes(4, 100, 16) >= 256
    assert lib.pwlq_search_workspace_bytes(1, 1 << 20, 64) >= (1 << 20) // 8192 * 64 * 8
