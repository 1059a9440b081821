"""Thin Python binding of ``libpwlq.so`` (argument marshalling only).

Every step of the path runs in the library's CUDA kernels; PyTorch is used for
device memory and streams.  The functions mirror the C entry points declared in
``include/pwlq.h`` and take CUDA tensors (or, for ``encode_host``, pinned host
tensors).  There is no CPU fallback: if the shared library has not been built,
or a tensor is not on a CUDA device, the call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# PWLQ_LIBRARY selects another build of the same C ABI (e.g. one compiled with other options)
_LIB_PATH = os.environ.get("PWLQ_LIBRARY") or os.path.join(_HERE, "libpwlq.so")
_lib = None

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_NONFINITE, ERR_TIMEOUT = range(7)
CODES_U8, CODES_PACKED = 0, 1
MODEL_GAUSS_APPROX, MODEL_GAUSS_ROOT, MODEL_LAPLACE = 0, 1, 2
MAX_K = 4096
MAX_K2 = 64

_P, _I64, _INT, _SZ = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
_SIGNATURES = {
    "pwlq_absmax": (_INT, [_P, _I64, _I64, _P, _P]),
    "pwlq_absmax_ragged": (_INT, [_P, _P, _I64, _I64, _P, _P]),
    "pwlq_search_workspace_bytes": (_SZ, [_I64, _I64, _INT]),
    "pwlq_search": (_INT, [_P, _I64, _I64, _INT, _P, _INT, _P, _P, _P, _P, _P, _P, _SZ, _P]),
    "pwlq_search_ragged": (_INT, [_P, _P, _I64, _I64, _I64, _INT, _P, _INT, _P, _P, _P, _P, _P, _P,
                                  _SZ, _P]),
    "pwlq_search_partial": (_INT, [_P, _I64, _I64, _INT, _P, _INT, _P, _P, _P, _P, _SZ, _P]),
    "pwlq_search_finish": (_INT, [_P, _INT, _I64, _INT, _P, _P, _P, _P, _P, _P, _P, _P, _P]),
    "pwlq_quantize": (_INT, [_P, _I64, _I64, _INT, _P, _P, _P, _P, _P, _INT, _P]),
    "pwlq_quantize_ragged": (_INT, [_P, _P, _I64, _I64, _INT, _P, _P, _P, _P, _P, _INT, _P]),
    "pwlq_dequantize": (_INT, [_P, _P, _I64, _I64, _INT, _P, _P, _P, _INT, _P]),
    "pwlq_dequantize_ragged": (_INT, [_P, _P, _P, _I64, _I64, _INT, _P, _P, _P, _INT, _P]),
    "pwlq_rowmap_bytes": (_SZ, [_I64]),
    "pwlq_rowmap_build": (_INT, [_P, _I64, _I64, _I64, _P, _SZ, _P]),
    "pwlq_absmax_mapped": (_INT, [_P, _P, _I64, _I64, _I64, _P, _P, _P]),
    "pwlq_quantize_mapped": (_INT, [_P, _P, _I64, _I64, _I64, _P, _INT, _P, _P, _P, _P, _P, _INT, _P]),
    "pwlq_dequantize_mapped": (_INT, [_P, _P, _P, _I64, _I64, _I64, _P, _INT, _P, _P, _P, _INT, _P]),
    "pwlq_minmax": (_INT, [_P, _I64, _I64, _P, _P, _P]),
    "pwlq_minmax_ragged": (_INT, [_P, _P, _I64, _I64, _P, _P, _P]),
    "pwlq_search_unsigned": (_INT, [_P, _I64, _I64, _INT, _P, _INT, _P, _P, _P, _P, _P, _P, _P, _SZ,
                                    _P]),
    "pwlq_search_unsigned_ragged": (_INT, [_P, _P, _I64, _I64, _I64, _INT, _P, _INT, _P, _P, _P, _P,
                                           _P, _P, _P, _SZ, _P]),
    "pwlq_quantize_unsigned": (_INT, [_P, _I64, _I64, _INT, _P, _P, _P, _P, _P, _P, _INT, _P]),
    "pwlq_quantize_unsigned_ragged": (_INT, [_P, _P, _I64, _I64, _INT, _P, _P, _P, _P, _P, _P, _INT,
                                             _P]),
    "pwlq_dequantize_unsigned": (_INT, [_P, _P, _I64, _I64, _INT, _P, _P, _P, _P, _INT, _P]),
    "pwlq_dequantize_unsigned_ragged": (_INT, [_P, _P, _P, _I64, _I64, _INT, _P, _P, _P, _P, _INT,
                                               _P]),
    "pwlq_search2_workspace_bytes": (_SZ, [_I64, _I64, _INT]),
    "pwlq_search2": (_INT, [_P, _I64, _I64, _INT, _P, _INT, _P, _P, _P, _P, _P, _P, _P, _P, _SZ, _P]),
    "pwlq_search2_ragged": (_INT, [_P, _P, _I64, _I64, _I64, _INT, _P, _INT, _P, _P, _P, _P, _P,
                                   _P, _P, _P, _SZ, _P]),
    "pwlq_search3": (_INT, [_P, _I64, _I64, _INT, _P, _INT, _P, _P, _P, _P, _P, _P, _SZ, _P]),
    "pwlq_search3_ragged": (_INT, [_P, _P, _I64, _I64, _I64, _INT, _P, _INT, _P, _P, _P, _P, _P,
                                   _P, _SZ, _P]),
    "pwlq_quantize3": (_INT, [_P, _I64, _I64, _INT, _P, _P, _P, _P, _P, _INT, _P]),
    "pwlq_quantize3_ragged": (_INT, [_P, _P, _I64, _I64, _INT, _P, _P, _P, _P, _P, _INT, _P]),
    "pwlq_dequantize3": (_INT, [_P, _P, _I64, _I64, _INT, _P, _P, _P, _INT, _P]),
    "pwlq_dequantize3_ragged": (_INT, [_P, _P, _P, _I64, _I64, _INT, _P, _P, _P, _INT, _P]),
    "pwlq_quantize2": (_INT, [_P, _I64, _I64, _INT, _P, _P, _P, _P, _P, _P, _INT, _P]),
    "pwlq_quantize2_ragged": (_INT, [_P, _P, _I64, _I64, _INT, _P, _P, _P, _P, _P, _P, _INT, _P]),
    "pwlq_dequantize2": (_INT, [_P, _P, _I64, _I64, _INT, _P, _P, _P, _P, _INT, _P]),
    "pwlq_dequantize2_ragged": (_INT, [_P, _P, _P, _I64, _I64, _INT, _P, _P, _P, _P, _INT, _P]),
    "pwlq_bias_workspace_bytes": (_SZ, [_I64, _I64]),
    "pwlq_bias_correction": (_INT, [_P, _I64, _I64, _INT, _P, _P, _P, _P, _P, _SZ, _P]),
    "pwlq_bias_correction_ragged": (_INT, [_P, _P, _I64, _I64, _I64, _INT, _P, _P, _P, _P, _P, _SZ,
                                           _P]),
    "pwlq_dequantize_bc": (_INT, [_P, _P, _I64, _I64, _INT, _P, _P, _P, _P, _P, _INT, _P]),
    "pwlq_dequantize_bc_ragged": (_INT, [_P, _P, _P, _I64, _I64, _INT, _P, _P, _P, _P, _P, _INT,
                                         _P]),
    "pwlq_dense_bytes": (_SZ, [_I64, _INT]),
    "pwlq_pack_dense": (_INT, [_P, _P, _I64, _INT, _P, _P]),
    "pwlq_unpack_dense": (_INT, [_P, _I64, _INT, _P, _P, _P]),
    "pwlq_encode_host_scratch_bytes": (_SZ, [_I64, _I64, _I64, _INT]),
    "pwlq_encode_host_status_offset": (_SZ, [_I64, _I64, _I64, _INT]),
    "pwlq_encode_host": (_INT, [_P, _P, _I64, _I64, _I64, _INT, _P, _INT, _P, _P, _P, _P, _P, _P,
                                _INT, _P, _SZ, _P, _P]),
    "pwlq_encode_host_unsigned": (_INT, [_P, _P, _I64, _I64, _I64, _INT, _P, _INT, _P, _P, _P, _P, _P,
                                         _P, _P, _INT, _P, _SZ, _P, _P]),
    "pwlq_search_noalloc": (_INT, [_P, _I64, _I64, _INT, _P, _INT, _P, _P, _P, _P, _P, _P, _P]),
    "pwlq_search_noalloc_max_bytes": (_SZ, []),
    "pwlq_select_workspace_bytes": (_SZ, [_I64, _I64]),
    "pwlq_select_analytic": (_INT, [_P, _I64, _I64, _P, _INT, _P, _P, _P, _SZ, _P]),
    "pwlq_select_analytic_ragged": (_INT, [_P, _P, _I64, _I64, _I64, _P, _INT, _P, _P, _P, _SZ, _P]),
    "pwlq_device_status": (_INT, []),
    "pwlq_status_string": (ctypes.c_char_p, [_INT]),
    "pwlq_version": (ctypes.c_char_p, []),
}
# exported by the library but not declared in the public header: hooks for the test suite
_TEST_HOOKS = {
    "pwlq_selftest_expire_wait": (_INT, [_INT, _P]),
}


class PwlqError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} (status {status})")


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Loads the C-ABI library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None or path is not None:
        path = path or _LIB_PATH
        if not os.path.exists(path):
            raise RuntimeError(
                f"{path} is missing: build it with `python -m paper_2002_00104_b200.build` "
                "(nvcc, sm_100a); this package has no CPU or PyTorch fallback")
        lib = ctypes.CDLL(path)
        for name, (res, args) in {**_SIGNATURES, **_TEST_HOOKS}.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def exported_symbols():
    return sorted(_SIGNATURES)


def device_status() -> int:
    """0, or 1 << ERR_TIMEOUT if a bounded device wait has expired on the current device since
    the previous call, 1 << ERR_INVALID_ARG if a call was given row maps of another layout
    (synchronises; reading clears the flags)."""
    return int(load_library().pwlq_device_status())


def selftest_expire_wait(polls: int = 48, stream=None) -> None:
    """Runs a one-warp kernel whose bounded wait is certain to run out (test hook)."""
    _check(load_library().pwlq_selftest_expire_wait(int(polls), _stream(stream)),
           "pwlq_selftest_expire_wait")


def status_string(status: int) -> str:
    return load_library().pwlq_status_string(int(status)).decode()


def version() -> str:
    return load_library().pwlq_version().decode()


def _dev(t: Optional[torch.Tensor], dtype, what: str):
    if t is None:
        return None
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise ValueError(f"{what} must be a contiguous CUDA tensor of {dtype}")
    return t.data_ptr()


def _stream(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _check(rc: int, what: str):
    if rc != OK:
        raise PwlqError(rc, what)


def _shape(x: torch.Tensor, row_offsets):
    """(C, n, total) of a dense [C, ...] tensor, or (C, None, total) for ragged rows."""
    if row_offsets is None:
        if x.dim() < 2:
            raise ValueError("dense input must be [C, n] (use x[None] for a single row)")
        C = x.shape[0]
        return C, x.numel() // C, x.numel()
    return row_offsets.numel() - 1, None, x.numel()


def code_bytes(total: int, bits: int, layout: int) -> int:
    return (total + 1) // 2 if (layout == CODES_PACKED and bits <= 4) else total


def rowmap_bytes(total: int) -> int:
    return int(load_library().pwlq_rowmap_bytes(int(total)))


def rowmap_build(C, total, row_offsets=None, n=0, device=None, out=None, stream=None):
    """Row maps of a layout (``pwlq_rowmap_build``) in a uint8 tensor, for the ``rowmap=``
    argument of ``absmax`` / ``quantize`` / ``dequantize``."""
    lib = load_library()
    need = rowmap_bytes(total)
    if out is None:
        dev = device if device is not None else row_offsets.device
        out = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    rc = lib.pwlq_rowmap_build(_dev(row_offsets, torch.int64, "row_offsets"), int(C), int(n),
                               int(total), _dev(out, torch.uint8, "rowmap"), out.numel(),
                               _stream(stream))
    _check(rc, "pwlq_rowmap_build")
    return out


def absmax(x, row_offsets=None, out=None, stream=None, rowmap=None):
    lib = load_library()
    C, n, total = _shape(x, row_offsets)
    m = out if out is not None else torch.empty(C, dtype=torch.float32, device=x.device)
    if rowmap is not None:
        rc = lib.pwlq_absmax_mapped(_dev(x, torch.float32, "x"),
                                    _dev(row_offsets, torch.int64, "row_offsets"), C,
                                    0 if row_offsets is not None else n, total,
                                    _dev(rowmap, torch.uint8, "rowmap"),
                                    _dev(m, torch.float32, "out"), _stream(stream))
    elif row_offsets is None:
        rc = lib.pwlq_absmax(_dev(x, torch.float32, "x"), C, n, _dev(m, torch.float32, "out"),
                             _stream(stream))
    else:
        rc = lib.pwlq_absmax_ragged(_dev(x, torch.float32, "x"),
                                    _dev(row_offsets, torch.int64, "row_offsets"), C, total,
                                    _dev(m, torch.float32, "out"), _stream(stream))
    _check(rc, "pwlq_absmax")
    return m


def search_workspace_bytes(C: int, max_n: int, K: int) -> int:
    return int(load_library().pwlq_search_workspace_bytes(C, max_n, K))


def search(x, bits, ratios, m=None, row_offsets=None, max_n=None, want_sse=False,
           workspace=None, out=None, stream=None):
    """Returns dict(p, err, idx, sse or None, workspace).  ``workspace[:4]`` holds the status."""
    lib = load_library()
    C, n, total = _shape(x, row_offsets)
    K = ratios.numel()
    longest = n if row_offsets is None else int(max_n)
    need = search_workspace_bytes(C, longest, K)
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=x.device)
    if out is None:
        out = {"p": torch.empty(C, dtype=torch.float32, device=x.device),
               "err": torch.empty(C, dtype=torch.float32, device=x.device),
               "idx": torch.empty(C, dtype=torch.int32, device=x.device),
               "sse": torch.empty((C, K), dtype=torch.float32, device=x.device) if want_sse else None}
    args_tail = (int(bits), _dev(ratios, torch.float32, "ratios"), K, _dev(m, torch.float32, "m"),
                 _dev(out["p"], torch.float32, "p"), _dev(out["err"], torch.float32, "err"),
                 _dev(out["idx"], torch.int32, "idx"), _dev(out.get("sse"), torch.float32, "sse"),
                 _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream))
    if row_offsets is None:
        rc = lib.pwlq_search(_dev(x, torch.float32, "x"), C, n, *args_tail)
    else:
        rc = lib.pwlq_search_ragged(_dev(x, torch.float32, "x"),
                                    _dev(row_offsets, torch.int64, "row_offsets"), C, total,
                                    longest, *args_tail)
    _check(rc, "pwlq_search")
    out = dict(out)
    out["workspace"] = workspace
    return out


def search_partial(x, bits, ratios, m, lo=None, workspace=None, out=None, stream=None):
    """Binary64 per-candidate sums ``[C, K]`` of one piece ``x`` ``[C, n]`` of rows whose common
    ranges are ``m`` (see ``pwlq_search_partial``).  Returns (sums, workspace)."""
    lib = load_library()
    C, n, _ = _shape(x, None)
    K = ratios.numel()
    if workspace is None:
        workspace = torch.empty(max(search_workspace_bytes(C, n, K), 256), dtype=torch.uint8,
                                device=x.device)
    sums = out if out is not None else torch.empty((C, K), dtype=torch.float64, device=x.device)
    _check(lib.pwlq_search_partial(_dev(x, torch.float32, "x"), C, n, int(bits),
                                   _dev(ratios, torch.float32, "ratios"), K,
                                   _dev(m, torch.float32, "m"), _dev(lo, torch.float32, "lo"),
                                   _dev(sums, torch.float64, "sums"),
                                   _dev(workspace, torch.uint8, "workspace"), workspace.numel(),
                                   _stream(stream)), "pwlq_search_partial")
    return sums, workspace


def search_finish(sums, m, ratios, lo=None, want_sse=False, stream=None):
    """Adds the stacked pieces' sums ``[parts, C, K]`` in order and takes the first minimum of
    every row.  Returns dict(p, err, idx, sse or None, status)."""
    lib = load_library()
    parts, C, K = sums.shape
    out = {"p": torch.empty(C, dtype=torch.float32, device=sums.device),
           "err": torch.empty(C, dtype=torch.float32, device=sums.device),
           "idx": torch.empty(C, dtype=torch.int32, device=sums.device),
           "sse": torch.empty((C, K), dtype=torch.float32, device=sums.device) if want_sse else None,
           "status": torch.zeros(1, dtype=torch.int32, device=sums.device)}
    _check(lib.pwlq_search_finish(_dev(sums, torch.float64, "sums"), int(parts), C, K,
                                  _dev(m, torch.float32, "m"), _dev(lo, torch.float32, "lo"),
                                  _dev(ratios, torch.float32, "ratios"),
                                  _dev(out["p"], torch.float32, "p"),
                                  _dev(out["err"], torch.float32, "err"),
                                  _dev(out["idx"], torch.int32, "idx"),
                                  _dev(out["sse"], torch.float32, "sse"),
                                  _dev(out["status"], torch.int32, "status"), _stream(stream)),
           "pwlq_search_finish")
    return out


def search_noalloc(x, bits, ratios, m=None, want_sse=False, stream=None):
    """``pwlq_search`` for callers that cannot allocate device memory: the workspace is a fixed
    array inside the library (``noalloc_max_bytes()`` per GPU), shared by all calls on a device,
    so overlapping calls must be ordered by the caller.  Dense ``[C, n]`` input only; problems
    that need more workspace than the array raise ``PwlqError(ERR_UNSUPPORTED)``.  The output
    tensors created here are a convenience of this Python wrapper; the C entry point itself only
    receives inputs and outputs.  Returns dict(p, err, idx, sse or None, status)."""
    lib = load_library()
    C, n, _ = _shape(x, None)
    K = ratios.numel()
    out = {"p": torch.empty(C, dtype=torch.float32, device=x.device),
           "err": torch.empty(C, dtype=torch.float32, device=x.device),
           "idx": torch.empty(C, dtype=torch.int32, device=x.device),
           "sse": torch.empty((C, K), dtype=torch.float32, device=x.device) if want_sse else None,
           "status": torch.zeros(1, dtype=torch.int32, device=x.device)}
    rc = lib.pwlq_search_noalloc(_dev(x, torch.float32, "x"), C, n, int(bits),
                                 _dev(ratios, torch.float32, "ratios"), K,
                                 _dev(m, torch.float32, "m"), _dev(out["p"], torch.float32, "p"),
                                 _dev(out["err"], torch.float32, "err"),
                                 _dev(out["idx"], torch.int32, "idx"),
                                 _dev(out["sse"], torch.float32, "sse"),
                                 _dev(out["status"], torch.int32, "status"), _stream(stream))
    _check(rc, "pwlq_search_noalloc")
    return out


def noalloc_max_bytes() -> int:
    return int(load_library().pwlq_search_noalloc_max_bytes())


def select_analytic(x, m, model, row_offsets=None, max_n=None, want_scale=False, stream=None):
    """Analytic breakpoint per row (the paper's own selection rule).  Returns (p, scale or None)."""
    lib = load_library()
    C, n, total = _shape(x, row_offsets)
    longest = n if row_offsets is None else int(max_n)
    need = int(lib.pwlq_select_workspace_bytes(C, longest))
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=x.device)
    p = torch.empty(C, dtype=torch.float32, device=x.device)
    scale = torch.empty(C, dtype=torch.float32, device=x.device) if want_scale else None
    tail = (_dev(m, torch.float32, "m"), int(model), _dev(p, torch.float32, "p"),
            _dev(scale, torch.float32, "scale"), _dev(ws, torch.uint8, "workspace"), ws.numel(),
            _stream(stream))
    if row_offsets is None:
        rc = lib.pwlq_select_analytic(_dev(x, torch.float32, "x"), C, n, *tail)
    else:
        rc = lib.pwlq_select_analytic_ragged(_dev(x, torch.float32, "x"),
                                             _dev(row_offsets, torch.int64, "row_offsets"), C,
                                             total, longest, *tail)
    _check(rc, "pwlq_select_analytic")
    return p, scale


def search_status(workspace) -> int:
    """Device status bits of the last search that used this workspace (synchronises)."""
    return int(workspace[:4].view(torch.int32).item())


def quantize(x, bits, m, p, layout=CODES_U8, row_offsets=None, want_fake=False, out=None,
             stream=None, rowmap=None):
    """Returns (codes uint8, region_mask uint8, fake fp32 or None)."""
    lib = load_library()
    C, n, total = _shape(x, row_offsets)
    if out is None:
        codes = torch.empty(code_bytes(total, bits, layout), dtype=torch.uint8, device=x.device)
        mask = torch.empty((total + 7) // 8, dtype=torch.uint8, device=x.device)
        fake = torch.empty(total, dtype=torch.float32, device=x.device) if want_fake else None
    else:
        codes, mask, fake = out
    tail = (int(bits), _dev(m, torch.float32, "m"), _dev(p, torch.float32, "p"),
            _dev(codes, torch.uint8, "codes"), _dev(mask, torch.uint8, "mask"),
            _dev(fake, torch.float32, "fake"), int(layout), _stream(stream))
    if rowmap is not None:
        rc = lib.pwlq_quantize_mapped(_dev(x, torch.float32, "x"),
                                      _dev(row_offsets, torch.int64, "row_offsets"), C,
                                      0 if row_offsets is not None else n, total,
                                      _dev(rowmap, torch.uint8, "rowmap"), *tail)
    elif row_offsets is None:
        rc = lib.pwlq_quantize(_dev(x, torch.float32, "x"), C, n, *tail)
    else:
        rc = lib.pwlq_quantize_ragged(_dev(x, torch.float32, "x"),
                                      _dev(row_offsets, torch.int64, "row_offsets"), C, total, *tail)
    _check(rc, "pwlq_quantize")
    return codes, mask, fake


def dequantize(codes, mask, bits, m, p, C=None, n=None, layout=CODES_U8, row_offsets=None,
               out=None, stream=None, rowmap=None):
    lib = load_library()
    if row_offsets is None:
        total = int(C) * int(n)
    else:
        C = row_offsets.numel() - 1
        total = int(out.numel()) if out is not None else int(row_offsets[-1].item())
    y = out if out is not None else torch.empty(total, dtype=torch.float32, device=codes.device)
    tail = (int(bits), _dev(m, torch.float32, "m"), _dev(p, torch.float32, "p"),
            _dev(y, torch.float32, "y"), int(layout), _stream(stream))
    if rowmap is not None:
        rc = lib.pwlq_dequantize_mapped(_dev(codes, torch.uint8, "codes"),
                                        _dev(mask, torch.uint8, "mask"),
                                        _dev(row_offsets, torch.int64, "row_offsets"), int(C),
                                        0 if row_offsets is not None else int(n), total,
                                        _dev(rowmap, torch.uint8, "rowmap"), *tail)
    elif row_offsets is None:
        rc = lib.pwlq_dequantize(_dev(codes, torch.uint8, "codes"), _dev(mask, torch.uint8, "mask"),
                                 int(C), int(n), *tail)
    else:
        rc = lib.pwlq_dequantize_ragged(_dev(codes, torch.uint8, "codes"),
                                        _dev(mask, torch.uint8, "mask"),
                                        _dev(row_offsets, torch.int64, "row_offsets"), C, total,
                                        *tail)
    _check(rc, "pwlq_dequantize")
    return y


# ---- one-sided ranges [lo, hi] (unsigned tensors): b-bit levels, no sign bit
def minmax(x, row_offsets=None, out=None, stream=None):
    """Returns (lo, hi), the per-row minimum and maximum."""
    lib = load_library()
    C, n, total = _shape(x, row_offsets)
    lo, hi = out if out is not None else (torch.empty(C, dtype=torch.float32, device=x.device),
                                          torch.empty(C, dtype=torch.float32, device=x.device))
    if row_offsets is None:
        rc = lib.pwlq_minmax(_dev(x, torch.float32, "x"), C, n, _dev(lo, torch.float32, "lo"),
                             _dev(hi, torch.float32, "hi"), _stream(stream))
    else:
        rc = lib.pwlq_minmax_ragged(_dev(x, torch.float32, "x"),
                                    _dev(row_offsets, torch.int64, "row_offsets"), C, total,
                                    _dev(lo, torch.float32, "lo"), _dev(hi, torch.float32, "hi"),
                                    _stream(stream))
    _check(rc, "pwlq_minmax")
    return lo, hi


def search_unsigned(x, bits, ratios, lo, hi, row_offsets=None, max_n=None, want_sse=False,
                    workspace=None, out=None, stream=None):
    """Returns dict(p, err, idx, sse or None, workspace).  ``workspace[:4]`` holds the status."""
    lib = load_library()
    C, n, total = _shape(x, row_offsets)
    K = ratios.numel()
    longest = n if row_offsets is None else int(max_n)
    need = search_workspace_bytes(C, longest, K)
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=x.device)
    if out is None:
        out = {"p": torch.empty(C, dtype=torch.float32, device=x.device),
               "err": torch.empty(C, dtype=torch.float32, device=x.device),
               "idx": torch.empty(C, dtype=torch.int32, device=x.device),
               "sse": torch.empty((C, K), dtype=torch.float32, device=x.device) if want_sse else None}
    args_tail = (int(bits), _dev(ratios, torch.float32, "ratios"), K, _dev(lo, torch.float32, "lo"),
                 _dev(hi, torch.float32, "hi"),
                 _dev(out["p"], torch.float32, "p"), _dev(out["err"], torch.float32, "err"),
                 _dev(out["idx"], torch.int32, "idx"), _dev(out.get("sse"), torch.float32, "sse"),
                 _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream))
    if row_offsets is None:
        rc = lib.pwlq_search_unsigned(_dev(x, torch.float32, "x"), C, n, *args_tail)
    else:
        rc = lib.pwlq_search_unsigned_ragged(_dev(x, torch.float32, "x"),
                                             _dev(row_offsets, torch.int64, "row_offsets"), C,
                                             total, longest, *args_tail)
    _check(rc, "pwlq_search_unsigned")
    out = dict(out)
    out["workspace"] = workspace
    return out


def quantize_unsigned(x, bits, lo, hi, p, layout=CODES_U8, row_offsets=None, want_fake=False,
                      out=None, stream=None):
    """Returns (codes uint8, region_mask uint8, fake fp32 or None)."""
    lib = load_library()
    C, n, total = _shape(x, row_offsets)
    if out is None:
        codes = torch.empty(code_bytes(total, bits, layout), dtype=torch.uint8, device=x.device)
        mask = torch.empty((total + 7) // 8, dtype=torch.uint8, device=x.device)
        fake = torch.empty(total, dtype=torch.float32, device=x.device) if want_fake else None
    else:
        codes, mask, fake = out
    tail = (int(bits), _dev(lo, torch.float32, "lo"), _dev(hi, torch.float32, "hi"),
            _dev(p, torch.float32, "p"), _dev(codes, torch.uint8, "codes"),
            _dev(mask, torch.uint8, "mask"), _dev(fake, torch.float32, "fake"), int(layout),
            _stream(stream))
    if row_offsets is None:
        rc = lib.pwlq_quantize_unsigned(_dev(x, torch.float32, "x"), C, n, *tail)
    else:
        rc = lib.pwlq_quantize_unsigned_ragged(_dev(x, torch.float32, "x"),
                                               _dev(row_offsets, torch.int64, "row_offsets"), C,
                                               total, *tail)
    _check(rc, "pwlq_quantize_unsigned")
    return codes, mask, fake


def dequantize_unsigned(codes, mask, bits, lo, hi, p, C=None, n=None, layout=CODES_U8,
                        row_offsets=None, out=None, stream=None):
    lib = load_library()
    if row_offsets is None:
        total = int(C) * int(n)
    else:
        C = row_offsets.numel() - 1
        total = int(out.numel()) if out is not None else int(row_offsets[-1].item())
    y = out if out is not None else torch.empty(total, dtype=torch.float32, device=codes.device)
    tail = (int(bits), _dev(lo, torch.float32, "lo"), _dev(hi, torch.float32, "hi"),
            _dev(p, torch.float32, "p"), _dev(y, torch.float32, "y"), int(layout), _stream(stream))
    if row_offsets is None:
        rc = lib.pwlq_dequantize_unsigned(_dev(codes, torch.uint8, "codes"),
                                          _dev(mask, torch.uint8, "mask"), int(C), int(n), *tail)
    else:
        rc = lib.pwlq_dequantize_unsigned_ragged(_dev(codes, torch.uint8, "codes"),
                                                 _dev(mask, torch.uint8, "mask"),
                                                 _dev(row_offsets, torch.int64, "row_offsets"), C,
                                                 total, *tail)
    _check(rc, "pwlq_dequantize_unsigned")
    return y


# ---- two breakpoints: regions [0, p1], (p1, p2], (p2, m]; two-bit region index per value
def search2_workspace_bytes(C: int, max_n: int, K: int) -> int:
    return int(load_library().pwlq_search2_workspace_bytes(int(C), int(max_n), int(K)))


def search2(x, bits, ratios, m, row_offsets=None, max_n=None, want_sse=False, workspace=None,
            stream=None):
    """Pair search; returns dict(p1, p2, err, idx1, idx2, sse ([C, K, K] or None), workspace)."""
    lib = load_library()
    C, n, total = _shape(x, row_offsets)
    K = ratios.numel()
    longest = n if row_offsets is None else int(max_n)
    if workspace is None:
        workspace = torch.empty(search2_workspace_bytes(C, longest, K), dtype=torch.uint8,
                                device=x.device)
    f32 = lambda: torch.empty(C, dtype=torch.float32, device=x.device)
    i32 = lambda: torch.empty(C, dtype=torch.int32, device=x.device)
    out = {"p1": f32(), "p2": f32(), "err": f32(), "idx1": i32(), "idx2": i32(),
           "sse": torch.empty((C, K, K), dtype=torch.float32, device=x.device) if want_sse else None}
    tail = (int(bits), _dev(ratios, torch.float32, "ratios"), K, _dev(m, torch.float32, "m"),
            _dev(out["p1"], torch.float32, "p1"), _dev(out["p2"], torch.float32, "p2"),
            _dev(out["err"], torch.float32, "err"), _dev(out["idx1"], torch.int32, "idx1"),
            _dev(out["idx2"], torch.int32, "idx2"), _dev(out["sse"], torch.float32, "sse"),
            _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream))
    if row_offsets is None:
        rc = lib.pwlq_search2(_dev(x, torch.float32, "x"), C, n, *tail)
    else:
        rc = lib.pwlq_search2_ragged(_dev(x, torch.float32, "x"),
                                     _dev(row_offsets, torch.int64, "row_offsets"), C, total,
                                     longest, *tail)
    _check(rc, "pwlq_search2")
    out["workspace"] = workspace
    return out


def quantize2(x, bits, m, p1, p2, layout=CODES_U8, row_offsets=None, want_fake=False, out=None,
              stream=None):
    """Returns (codes uint8, region2 uint8 (two bits per value), fake fp32 or None)."""
    lib = load_library()
    C, n, total = _shape(x, row_offsets)
    if out is None:
        codes = torch.empty(code_bytes(total, bits, layout), dtype=torch.uint8, device=x.device)
        region = torch.empty((total + 3) // 4, dtype=torch.uint8, device=x.device)
        fake = torch.empty(total, dtype=torch.float32, device=x.device) if want_fake else None
    else:
        codes, region, fake = out
    tail = (int(bits), _dev(m, torch.float32, "m"), _dev(p1, torch.float32, "p1"),
            _dev(p2, torch.float32, "p2"), _dev(codes, torch.uint8, "codes"),
            _dev(region, torch.uint8, "region2"), _dev(fake, torch.float32, "fake"), int(layout),
            _stream(stream))
    if row_offsets is None:
        rc = lib.pwlq_quantize2(_dev(x, torch.float32, "x"), C, n, *tail)
    else:
        rc = lib.pwlq_quantize2_ragged(_dev(x, torch.float32, "x"),
                                       _dev(row_offsets, torch.int64, "row_offsets"), C, total,
                                       *tail)
    _check(rc, "pwlq_quantize2")
    return codes, region, fake


def dequantize2(codes, region, bits, m, p1, p2, C=None, n=None, layout=CODES_U8, row_offsets=None,
                out=None, stream=None):
    lib = load_library()
    if row_offsets is None:
        total = int(C) * int(n)
    else:
        C = row_offsets.numel() - 1
        total = int(out.numel()) if out is not None else int(row_offsets[-1].item())
    y = out if out is not None else torch.empty(total, dtype=torch.float32, device=codes.device)
    tail = (int(bits), _dev(m, torch.float32, "m"), _dev(p1, torch.float32, "p1"),
            _dev(p2, torch.float32, "p2"), _dev(y, torch.float32, "y"), int(layout),
            _stream(stream))
    if row_offsets is None:
        rc = lib.pwlq_dequantize2(_dev(codes, torch.uint8, "codes"),
                                  _dev(region, torch.uint8, "region2"), int(C), int(n), *tail)
    else:
        rc = lib.pwlq_dequantize2_ragged(_dev(codes, torch.uint8, "codes"),
                                         _dev(region, torch.uint8, "region2"),
                                         _dev(row_offsets, torch.int64, "row_offsets"), C, total,
                                         *tail)
    _check(rc, "pwlq_dequantize2")
    return y


# ---- three breakpoints: the breakpoints of a row side by side, [C, 3]
def search3(x, bits, ratios, m, row_offsets=None, max_n=None, want_sse=False, workspace=None,
            stream=None):
    """Triple search; returns dict(p [C, 3], err, idx [C, 3], sse ([C, K, K, K] or None),
    workspace)."""
    lib = load_library()
    C, n, total = _shape(x, row_offsets)
    K = ratios.numel()
    longest = n if row_offsets is None else int(max_n)
    if workspace is None:
        workspace = torch.empty(search2_workspace_bytes(C, longest, K), dtype=torch.uint8,
                                device=x.device)
    out = {"p": torch.empty((C, 3), dtype=torch.float32, device=x.device),
           "err": torch.empty(C, dtype=torch.float32, device=x.device),
           "idx": torch.empty((C, 3), dtype=torch.int32, device=x.device),
           "sse": torch.empty((C, K, K, K), dtype=torch.float32, device=x.device) if want_sse else None}
    tail = (int(bits), _dev(ratios, torch.float32, "ratios"), K, _dev(m, torch.float32, "m"),
            _dev(out["p"], torch.float32, "p"), _dev(out["err"], torch.float32, "err"),
            _dev(out["idx"], torch.int32, "idx"), _dev(out["sse"], torch.float32, "sse"),
            _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream))
    if row_offsets is None:
        rc = lib.pwlq_search3(_dev(x, torch.float32, "x"), C, n, *tail)
    else:
        rc = lib.pwlq_search3_ragged(_dev(x, torch.float32, "x"),
                                     _dev(row_offsets, torch.int64, "row_offsets"), C, total,
                                     longest, *tail)
    _check(rc, "pwlq_search3")
    out["workspace"] = workspace
    return out


def quantize3(x, bits, m, p, layout=CODES_U8, row_offsets=None, want_fake=False, out=None,
              stream=None):
    """p: [C, 3].  Returns (codes uint8, region2 uint8 (two bits per value), fake fp32 or None)."""
    lib = load_library()
    C, n, total = _shape(x, row_offsets)
    if out is None:
        codes = torch.empty(code_bytes(total, bits, layout), dtype=torch.uint8, device=x.device)
        region = torch.empty((total + 3) // 4, dtype=torch.uint8, device=x.device)
        fake = torch.empty(total, dtype=torch.float32, device=x.device) if want_fake else None
    else:
        codes, region, fake = out
    tail = (int(bits), _dev(m, torch.float32, "m"), _dev(p, torch.float32, "p"),
            _dev(codes, torch.uint8, "codes"), _dev(region, torch.uint8, "region2"),
            _dev(fake, torch.float32, "fake"), int(layout), _stream(stream))
    if row_offsets is None:
        rc = lib.pwlq_quantize3(_dev(x, torch.float32, "x"), C, n, *tail)
    else:
        rc = lib.pwlq_quantize3_ragged(_dev(x, torch.float32, "x"),
                                       _dev(row_offsets, torch.int64, "row_offsets"), C, total,
                                       *tail)
    _check(rc, "pwlq_quantize3")
    return codes, region, fake


def dequantize3(codes, region, bits, m, p, C=None, n=None, layout=CODES_U8, row_offsets=None,
                out=None, stream=None):
    lib = load_library()
    if row_offsets is None:
        total = int(C) * int(n)
    else:
        C = row_offsets.numel() - 1
        total = int(out.numel()) if out is not None else int(row_offsets[-1].item())
    y = out if out is not None else torch.empty(total, dtype=torch.float32, device=codes.device)
    tail = (int(bits), _dev(m, torch.float32, "m"), _dev(p, torch.float32, "p"),
            _dev(y, torch.float32, "y"), int(layout), _stream(stream))
    if row_offsets is None:
        rc = lib.pwlq_dequantize3(_dev(codes, torch.uint8, "codes"),
                                  _dev(region, torch.uint8, "region2"), int(C), int(n), *tail)
    else:
        rc = lib.pwlq_dequantize3_ragged(_dev(codes, torch.uint8, "codes"),
                                         _dev(region, torch.uint8, "region2"),
                                         _dev(row_offsets, torch.int64, "row_offsets"), C, total,
                                         *tail)
    _check(rc, "pwlq_dequantize3")
    return y


# ---- bias correction and dense (b+1)-bit storage
def bias_correction(x, bits, m, p, row_offsets=None, max_n=None, workspace=None, stream=None):
    """Returns (xi, beta): the folded scale and offset of every row."""
    lib = load_library()
    C, n, total = _shape(x, row_offsets)
    longest = n if row_offsets is None else int(max_n)
    need = int(lib.pwlq_bias_workspace_bytes(C, longest))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=x.device)
    xi = torch.empty(C, dtype=torch.float32, device=x.device)
    beta = torch.empty(C, dtype=torch.float32, device=x.device)
    tail = (int(bits), _dev(m, torch.float32, "m"), _dev(p, torch.float32, "p"),
            _dev(xi, torch.float32, "xi"), _dev(beta, torch.float32, "beta"),
            _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream))
    if row_offsets is None:
        rc = lib.pwlq_bias_correction(_dev(x, torch.float32, "x"), C, n, *tail)
    else:
        rc = lib.pwlq_bias_correction_ragged(_dev(x, torch.float32, "x"),
                                             _dev(row_offsets, torch.int64, "row_offsets"), C,
                                             total, longest, *tail)
    _check(rc, "pwlq_bias_correction")
    return xi, beta


def dequantize_bc(codes, mask, bits, m, p, xi, beta, C=None, n=None, layout=CODES_U8,
                  row_offsets=None, out=None, stream=None):
    lib = load_library()
    if row_offsets is None:
        total = int(C) * int(n)
    else:
        C = row_offsets.numel() - 1
        total = int(out.numel()) if out is not None else int(row_offsets[-1].item())
    y = out if out is not None else torch.empty(total, dtype=torch.float32, device=codes.device)
    tail = (int(bits), _dev(m, torch.float32, "m"), _dev(p, torch.float32, "p"),
            _dev(xi, torch.float32, "xi"), _dev(beta, torch.float32, "beta"),
            _dev(y, torch.float32, "y"), int(layout), _stream(stream))
    if row_offsets is None:
        rc = lib.pwlq_dequantize_bc(_dev(codes, torch.uint8, "codes"),
                                    _dev(mask, torch.uint8, "mask"), int(C), int(n), *tail)
    else:
        rc = lib.pwlq_dequantize_bc_ragged(_dev(codes, torch.uint8, "codes"),
                                           _dev(mask, torch.uint8, "mask"),
                                           _dev(row_offsets, torch.int64, "row_offsets"), C, total,
                                           *tail)
    _check(rc, "pwlq_dequantize_bc")
    return y


def dense_bytes(total: int, bits: int) -> int:
    return int(load_library().pwlq_dense_bytes(total, bits))


def pack_dense(codes_u8, mask, bits, out=None, stream=None):
    lib = load_library()
    total = codes_u8.numel()
    if out is None:
        out = torch.empty(dense_bytes(total, bits), dtype=torch.uint8, device=codes_u8.device)
    _check(lib.pwlq_pack_dense(_dev(codes_u8, torch.uint8, "codes"), _dev(mask, torch.uint8, "mask"),
                               total, int(bits), _dev(out, torch.uint8, "out"), _stream(stream)),
           "pwlq_pack_dense")
    return out


def unpack_dense(stream_bytes, total, bits, stream=None):
    lib = load_library()
    codes = torch.empty(total, dtype=torch.uint8, device=stream_bytes.device)
    mask = torch.empty((total + 7) // 8, dtype=torch.uint8, device=stream_bytes.device)
    _check(lib.pwlq_unpack_dense(_dev(stream_bytes, torch.uint8, "stream"), int(total), int(bits),
                                 _dev(codes, torch.uint8, "codes"), _dev(mask, torch.uint8, "mask"),
                                 _stream(stream)), "pwlq_unpack_dense")
    return codes, mask


def encode_host_scratch_bytes(C: int, total: int, max_n: int, K: int) -> int:
    return int(load_library().pwlq_encode_host_scratch_bytes(C, total, max_n, K))


def encode_host_status(dev_scratch, C: int, total: int, max_n: int, K: int) -> int:
    """Status word of the search inside the last ``encode_host`` call that used ``dev_scratch``
    (synchronises)."""
    off = int(load_library().pwlq_encode_host_status_offset(C, total, max_n, K))
    return int(dev_scratch[off:off + 4].view(torch.int32).item())


def _host(t: Optional[torch.Tensor], dtype, what: str):
    if t is None:
        return None
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{what} must be a contiguous host tensor of {dtype}")
    return t.data_ptr()


def encode_host(x_host, row_offsets_host, C, max_n, bits, ratios_host, out_host, layout,
                dev_scratch, stream=None):
    """Whole path from (pinned) host tensors; ``out_host`` = dict(m, p, err, idx, codes, mask) of
    host tensors that receive the results once the stream is synchronised."""
    lib = load_library()
    total = x_host.numel()
    rc = lib.pwlq_encode_host(
        _host(x_host, torch.float32, "x_host"), _host(row_offsets_host, torch.int64, "row_offsets"),
        int(C), total, int(max_n), int(bits), _host(ratios_host, torch.float32, "ratios"),
        ratios_host.numel(), _host(out_host["m"], torch.float32, "m"),
        _host(out_host["p"], torch.float32, "p"), _host(out_host.get("err"), torch.float32, "err"),
        _host(out_host["idx"], torch.int32, "idx"), _host(out_host["codes"], torch.uint8, "codes"),
        _host(out_host["mask"], torch.uint8, "mask"), int(layout),
        _dev(dev_scratch, torch.uint8, "dev_scratch"), dev_scratch.numel(), None, _stream(stream))
    _check(rc, "pwlq_encode_host")


def encode_host_unsigned(x_host, row_offsets_host, C, max_n, bits, ratios_host, out_host, layout,
                         dev_scratch, stream=None):
    """One-sided form of ``encode_host``; ``out_host`` = dict(lo, hi, p, err, idx, codes, mask)."""
    lib = load_library()
    total = x_host.numel()
    rc = lib.pwlq_encode_host_unsigned(
        _host(x_host, torch.float32, "x_host"), _host(row_offsets_host, torch.int64, "row_offsets"),
        int(C), total, int(max_n), int(bits), _host(ratios_host, torch.float32, "ratios"),
        ratios_host.numel(), _host(out_host["lo"], torch.float32, "lo"),
        _host(out_host["hi"], torch.float32, "hi"), _host(out_host["p"], torch.float32, "p"),
        _host(out_host.get("err"), torch.float32, "err"), _host(out_host["idx"], torch.int32, "idx"),
        _host(out_host["codes"], torch.uint8, "codes"), _host(out_host["mask"], torch.uint8, "mask"),
        int(layout), _dev(dev_scratch, torch.uint8, "dev_scratch"), dev_scratch.numel(), None,
        _stream(stream))
    _check(rc, "pwlq_encode_host_unsigned")
