"""ctypes front end of ``pwlq_oracle.c`` (test infrastructure, not product code).

The C file is the oracle; this module only compiles it with gcc
(``-O2 -ffp-contract=off``, no fast-math, so every binary32 operation rounds
once) and marshals numpy arrays.  Rows are either a dense ``[C, n]`` view or a
ragged set given by ``row_offsets`` (``C + 1`` ascending flat offsets).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pwlq_oracle.c")
_SO = os.path.join(_HERE, "libpwlq_oracle.so")


class OracleError(RuntimeError):
    pass


def _compile(src: str, so: str) -> None:
    cmd = ["gcc", "-std=c99", "-O2", "-ffp-contract=off", "-fno-fast-math",
           "-fPIC", "-shared", "-o", so, src, "-lm"]
    subprocess.run(cmd, check=True)


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        _compile(_SRC, _SO)
    return _SO


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _rows(x, row_offsets):
    """Returns (flat fp32 array, offsets array or None, C, n)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if row_offsets is None:
        if x.ndim == 1:
            x = x.reshape(1, -1)
        x2 = x.reshape(x.shape[0], -1)
        return x2.reshape(-1), None, x2.shape[0], x2.shape[1]
    ro = np.ascontiguousarray(row_offsets, dtype=np.int64)
    flat = x.reshape(-1)
    assert ro[0] == 0 and ro[-1] == flat.size and np.all(np.diff(ro) >= 0)
    return flat, ro, ro.size - 1, 0


def _check(rc, what):
    if rc != 0:
        raise OracleError(f"{what}: status {rc}")


def code_bytes(total, bits, layout):
    return (total + 1) // 2 if (layout == 1 and bits <= 4) else total


class OracleLib:
    """One compiled copy of the oracle.  ``OracleLib()`` is the oracle itself; the tests also load
    deliberately broken copies through ``so_path`` to show that the pins notice them."""

    OracleError = OracleError

    def __init__(self, so_path: str | None = None):
        lib = ctypes.CDLL(so_path or build())
        P = ctypes.c_void_p
        I64 = ctypes.c_int64
        lib.pwlq_oracle_absmax.argtypes = [P, P, I64, I64, P]
        lib.pwlq_oracle_search.argtypes = [P, P, I64, I64, ctypes.c_int, P, ctypes.c_int, P,
                                           P, P, P, P, P]
        lib.pwlq_oracle_quantize.argtypes = [P, P, I64, I64, ctypes.c_int, P, P, P, P, P,
                                             ctypes.c_int]
        lib.pwlq_oracle_dequantize.argtypes = [P, P, P, I64, I64, ctypes.c_int, P, P, P,
                                               ctypes.c_int]
        lib.pwlq_oracle_elem.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_float,
                                         ctypes.c_int, P, P, P, P]
        lib.pwlq_oracle_elem.restype = None
        lib.pwlq_oracle_params.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_int, P]
        lib.pwlq_oracle_params.restype = None
        lib.pwlq_oracle_analytic_p.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_int]
        lib.pwlq_oracle_analytic_p.restype = ctypes.c_double
        lib.pwlq_oracle_select_analytic.argtypes = [P, P, I64, I64, P, ctypes.c_int, P, P]
        lib.pwlq_oracle_minmax.argtypes = [P, P, I64, I64, P, P]
        lib.pwlq_oracle_search_u.argtypes = [P, P, I64, I64, ctypes.c_int, P, ctypes.c_int, P, P,
                                             P, P, P, P, P]
        lib.pwlq_oracle_quantize_u.argtypes = [P, P, I64, I64, ctypes.c_int, P, P, P, P, P, P,
                                               ctypes.c_int]
        lib.pwlq_oracle_dequantize_u.argtypes = [P, P, P, I64, I64, ctypes.c_int, P, P, P, P,
                                                 ctypes.c_int]
        lib.pwlq_oracle_elem_u.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_float,
                                           ctypes.c_float, ctypes.c_int, P, P, P]
        lib.pwlq_oracle_elem_u.restype = None
        lib.pwlq_oracle_search2.argtypes = [P, P, I64, I64, ctypes.c_int, P, ctypes.c_int, P, P, P,
                                            P, P, P, P, P]
        lib.pwlq_oracle_quantize2.argtypes = [P, P, I64, I64, ctypes.c_int, P, P, P, P, P, P,
                                              ctypes.c_int]
        lib.pwlq_oracle_search3.argtypes = [P, P, I64, I64, ctypes.c_int, P, ctypes.c_int, P, P, P,
                                            P, P]
        lib.pwlq_oracle_quantize3.argtypes = [P, P, I64, I64, ctypes.c_int, P, P, P, P, P,
                                              ctypes.c_int]
        lib.pwlq_oracle_dequantize3.argtypes = [P, P, P, I64, I64, ctypes.c_int, P, P, P,
                                                ctypes.c_int]
        lib.pwlq_oracle_dequantize2.argtypes = [P, P, P, I64, I64, ctypes.c_int, P, P, P, P,
                                                ctypes.c_int]
        lib.pwlq_oracle_bias_correction.argtypes = [P, P, I64, I64, ctypes.c_int, P, P, P, P]
        lib.pwlq_oracle_dequantize_bc.argtypes = [P, P, P, I64, I64, ctypes.c_int, P, P, P, P, P,
                                                  ctypes.c_int]
        lib.pwlq_oracle_pack_dense.argtypes = [P, P, I64, ctypes.c_int, P]
        lib.pwlq_oracle_unpack_dense.argtypes = [P, I64, ctypes.c_int, P, P]
        self._lib = lib

    def absmax(self, x, row_offsets=None):
        flat, ro, C, n = _rows(x, row_offsets)
        m = np.empty(C, dtype=np.float32)
        _check(self._lib.pwlq_oracle_absmax(_ptr(flat), _ptr(ro), C, n, _ptr(m)), "absmax")
        return m

    def search(self, x, bits, ratios, m=None, row_offsets=None, want_sse=True):
        """Returns dict(p, err, idx, sse (float32 [C,K]), sse64 (float64 [C,K]))."""
        flat, ro, C, n = _rows(x, row_offsets)
        ratios = np.ascontiguousarray(ratios, dtype=np.float32)
        K = int(ratios.size)
        if m is not None:
            m = np.ascontiguousarray(m, dtype=np.float32)
            assert m.size == C
        p = np.empty(C, dtype=np.float32)
        err = np.empty(C, dtype=np.float32)
        idx = np.empty(C, dtype=np.int32)
        sse = np.empty((C, K), dtype=np.float32) if want_sse else None
        sse64 = np.empty((C, K), dtype=np.float64) if want_sse else None
        _check(self._lib.pwlq_oracle_search(_ptr(flat), _ptr(ro), C, n, int(bits), _ptr(ratios),
                                            K, _ptr(m), _ptr(p), _ptr(err), _ptr(idx),
                                            _ptr(sse), _ptr(sse64)), "search")
        return {"p": p, "err": err, "idx": idx, "sse": sse, "sse64": sse64}

    def quantize(self, x, bits, m, p, layout=0, row_offsets=None, want_fake=True):
        """Returns (codes uint8, region_mask uint8, fake fp32 or None)."""
        flat, ro, C, n = _rows(x, row_offsets)
        total = flat.size
        m = np.ascontiguousarray(m, dtype=np.float32)
        p = np.ascontiguousarray(p, dtype=np.float32)
        assert m.size == C and p.size == C
        codes = np.empty(code_bytes(total, bits, layout), dtype=np.uint8)
        mask = np.empty((total + 7) // 8, dtype=np.uint8)
        fake = np.empty(total, dtype=np.float32) if want_fake else None
        _check(self._lib.pwlq_oracle_quantize(_ptr(flat), _ptr(ro), C, n, int(bits), _ptr(m),
                                              _ptr(p), _ptr(codes), _ptr(mask), _ptr(fake),
                                              int(layout)), "quantize")
        return codes, mask, fake

    def dequantize(self, codes, mask, bits, m, p, C=None, n=None, layout=0, row_offsets=None):
        codes = np.ascontiguousarray(codes, dtype=np.uint8)
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
        m = np.ascontiguousarray(m, dtype=np.float32)
        p = np.ascontiguousarray(p, dtype=np.float32)
        if row_offsets is not None:
            ro = np.ascontiguousarray(row_offsets, dtype=np.int64)
            C, n, total = ro.size - 1, 0, int(ro[-1])
        else:
            ro, total = None, int(C) * int(n)
        assert m.size == C and p.size == C
        y = np.empty(total, dtype=np.float32)
        _check(self._lib.pwlq_oracle_dequantize(_ptr(codes), _ptr(mask), _ptr(ro), C, n,
                                                int(bits), _ptr(m), _ptr(p), _ptr(y),
                                                int(layout)), "dequantize")
        return y

    def analytic_p(self, m, scale, model):
        """Breakpoint of the assumed density (0: Gaussian ln-approximation, 1: Gaussian Eq. 9
        root, 2: Laplacian Eq. 9 root), clamped to (0, m/2]."""
        return float(self._lib.pwlq_oracle_analytic_p(float(m), float(scale), int(model)))

    def select_analytic(self, x, m, model, row_offsets=None):
        """Returns (p float32 [C], scale float64 [C]) for every row."""
        flat, ro, C, n = _rows(x, row_offsets)
        m = np.ascontiguousarray(m, dtype=np.float32)
        assert m.size == C
        p = np.empty(C, dtype=np.float32)
        scale = np.empty(C, dtype=np.float64)
        _check(self._lib.pwlq_oracle_select_analytic(_ptr(flat), _ptr(ro), C, n, _ptr(m),
                                                     int(model), _ptr(p), _ptr(scale)),
               "select_analytic")
        return p, scale

    def elem(self, x, m, p, bits):
        """One value through Eq. 3: returns (code, region, q, y)."""
        code, region, q = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
        y = ctypes.c_float()
        self._lib.pwlq_oracle_elem(float(x), float(m), float(p), int(bits), ctypes.byref(code),
                                   ctypes.byref(region), ctypes.byref(q), ctypes.byref(y))
        return code.value, region.value, q.value, y.value

    # ---- one-sided ranges [lo, hi] (unsigned tensors): b-bit levels, no sign bit
    def minmax(self, x, row_offsets=None):
        flat, ro, C, n = _rows(x, row_offsets)
        lo = np.empty(C, dtype=np.float32)
        hi = np.empty(C, dtype=np.float32)
        _check(self._lib.pwlq_oracle_minmax(_ptr(flat), _ptr(ro), C, n, _ptr(lo), _ptr(hi)),
               "minmax")
        return lo, hi

    def search_u(self, x, bits, ratios, lo, hi, row_offsets=None, want_sse=True):
        """Returns dict(p, err, idx, sse (float32 [C,K]), sse64 (float64 [C,K]))."""
        flat, ro, C, n = _rows(x, row_offsets)
        ratios = np.ascontiguousarray(ratios, dtype=np.float32)
        K = int(ratios.size)
        lo = np.ascontiguousarray(lo, dtype=np.float32)
        hi = np.ascontiguousarray(hi, dtype=np.float32)
        assert lo.size == C and hi.size == C
        p = np.empty(C, dtype=np.float32)
        err = np.empty(C, dtype=np.float32)
        idx = np.empty(C, dtype=np.int32)
        sse = np.empty((C, K), dtype=np.float32) if want_sse else None
        sse64 = np.empty((C, K), dtype=np.float64) if want_sse else None
        _check(self._lib.pwlq_oracle_search_u(_ptr(flat), _ptr(ro), C, n, int(bits), _ptr(ratios),
                                              K, _ptr(lo), _ptr(hi), _ptr(p), _ptr(err),
                                              _ptr(idx), _ptr(sse), _ptr(sse64)), "search_u")
        return {"p": p, "err": err, "idx": idx, "sse": sse, "sse64": sse64}

    def quantize_u(self, x, bits, lo, hi, p, layout=0, row_offsets=None, want_fake=True):
        """Returns (codes uint8, region_mask uint8, fake fp32 or None)."""
        flat, ro, C, n = _rows(x, row_offsets)
        total = flat.size
        lo = np.ascontiguousarray(lo, dtype=np.float32)
        hi = np.ascontiguousarray(hi, dtype=np.float32)
        p = np.ascontiguousarray(p, dtype=np.float32)
        assert lo.size == C and hi.size == C and p.size == C
        codes = np.empty(code_bytes(total, bits, layout), dtype=np.uint8)
        mask = np.empty((total + 7) // 8, dtype=np.uint8)
        fake = np.empty(total, dtype=np.float32) if want_fake else None
        _check(self._lib.pwlq_oracle_quantize_u(_ptr(flat), _ptr(ro), C, n, int(bits), _ptr(lo),
                                                _ptr(hi), _ptr(p), _ptr(codes), _ptr(mask),
                                                _ptr(fake), int(layout)), "quantize_u")
        return codes, mask, fake

    def dequantize_u(self, codes, mask, bits, lo, hi, p, C=None, n=None, layout=0,
                     row_offsets=None):
        codes = np.ascontiguousarray(codes, dtype=np.uint8)
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
        lo = np.ascontiguousarray(lo, dtype=np.float32)
        hi = np.ascontiguousarray(hi, dtype=np.float32)
        p = np.ascontiguousarray(p, dtype=np.float32)
        if row_offsets is not None:
            ro = np.ascontiguousarray(row_offsets, dtype=np.int64)
            C, n, total = ro.size - 1, 0, int(ro[-1])
        else:
            ro, total = None, int(C) * int(n)
        assert lo.size == C and hi.size == C and p.size == C
        y = np.empty(total, dtype=np.float32)
        _check(self._lib.pwlq_oracle_dequantize_u(_ptr(codes), _ptr(mask), _ptr(ro), C, n,
                                                  int(bits), _ptr(lo), _ptr(hi), _ptr(p),
                                                  _ptr(y), int(layout)), "dequantize_u")
        return y

    def elem_u(self, x, lo, hi, p, bits):
        """One value through the one-sided quantizer: returns (code, region, y)."""
        code, region = ctypes.c_int(), ctypes.c_int()
        y = ctypes.c_float()
        self._lib.pwlq_oracle_elem_u(float(x), float(lo), float(hi), float(p), int(bits),
                                     ctypes.byref(code), ctypes.byref(region), ctypes.byref(y))
        return code.value, region.value, y.value

    # ---- two breakpoints: regions [0, p1], (p1, p2], (p2, m]; region index in two bits per value
    def search2(self, x, bits, ratios, m, row_offsets=None, want_sse=True):
        """Returns dict(p1, p2, err, idx1, idx2, sse64 [C,K,K] (entries i < j valid))."""
        flat, ro, C, n = _rows(x, row_offsets)
        ratios = np.ascontiguousarray(ratios, dtype=np.float32)
        K = int(ratios.size)
        m = np.ascontiguousarray(m, dtype=np.float32)
        assert m.size == C
        p1 = np.empty(C, dtype=np.float32)
        p2 = np.empty(C, dtype=np.float32)
        err = np.empty(C, dtype=np.float32)
        i1 = np.empty(C, dtype=np.int32)
        i2 = np.empty(C, dtype=np.int32)
        sse64 = np.empty((C, K, K), dtype=np.float64) if want_sse else None
        _check(self._lib.pwlq_oracle_search2(_ptr(flat), _ptr(ro), C, n, int(bits), _ptr(ratios),
                                             K, _ptr(m), _ptr(p1), _ptr(p2), _ptr(err), _ptr(i1),
                                             _ptr(i2), None, _ptr(sse64)), "search2")
        return {"p1": p1, "p2": p2, "err": err, "idx1": i1, "idx2": i2, "sse64": sse64}

    def quantize2(self, x, bits, m, p1, p2, layout=0, row_offsets=None, want_fake=True):
        """Returns (codes uint8, region2 uint8 (two bits per value), fake fp32 or None)."""
        flat, ro, C, n = _rows(x, row_offsets)
        total = flat.size
        m, p1, p2 = (np.ascontiguousarray(v, dtype=np.float32) for v in (m, p1, p2))
        assert m.size == C and p1.size == C and p2.size == C
        codes = np.empty(code_bytes(total, bits, layout), dtype=np.uint8)
        region = np.empty((total + 3) // 4, dtype=np.uint8)
        fake = np.empty(total, dtype=np.float32) if want_fake else None
        _check(self._lib.pwlq_oracle_quantize2(_ptr(flat), _ptr(ro), C, n, int(bits), _ptr(m),
                                               _ptr(p1), _ptr(p2), _ptr(codes), _ptr(region),
                                               _ptr(fake), int(layout)), "quantize2")
        return codes, region, fake

    def dequantize2(self, codes, region, bits, m, p1, p2, C=None, n=None, layout=0,
                    row_offsets=None):
        codes = np.ascontiguousarray(codes, dtype=np.uint8)
        region = np.ascontiguousarray(region, dtype=np.uint8)
        m, p1, p2 = (np.ascontiguousarray(v, dtype=np.float32) for v in (m, p1, p2))
        if row_offsets is not None:
            ro = np.ascontiguousarray(row_offsets, dtype=np.int64)
            C, n, total = ro.size - 1, 0, int(ro[-1])
        else:
            ro, total = None, int(C) * int(n)
        assert m.size == C and p1.size == C and p2.size == C
        y = np.empty(total, dtype=np.float32)
        _check(self._lib.pwlq_oracle_dequantize2(_ptr(codes), _ptr(region), _ptr(ro), C, n,
                                                 int(bits), _ptr(m), _ptr(p1), _ptr(p2), _ptr(y),
                                                 int(layout)), "dequantize2")
        return y

    # ---- three breakpoints: four regions, region index 0..3 in the two bits per value
    def search3(self, x, bits, ratios, m, row_offsets=None, want_sse=True):
        """Returns dict(p [C,3], err, idx [C,3], sse64 [C,K,K,K] (entries i < j < k valid))."""
        flat, ro, C, n = _rows(x, row_offsets)
        ratios = np.ascontiguousarray(ratios, dtype=np.float32)
        K = int(ratios.size)
        m = np.ascontiguousarray(m, dtype=np.float32)
        assert m.size == C
        p = np.empty((C, 3), dtype=np.float32)
        err = np.empty(C, dtype=np.float32)
        idx = np.empty((C, 3), dtype=np.int32)
        sse64 = np.empty((C, K, K, K), dtype=np.float64) if want_sse else None
        _check(self._lib.pwlq_oracle_search3(_ptr(flat), _ptr(ro), C, n, int(bits), _ptr(ratios),
                                             K, _ptr(m), _ptr(p), _ptr(err), _ptr(idx),
                                             _ptr(sse64)), "search3")
        return {"p": p, "err": err, "idx": idx, "sse64": sse64}

    def quantize3(self, x, bits, m, p, layout=0, row_offsets=None, want_fake=True):
        """p: [C, 3].  Returns (codes uint8, region2 uint8 (two bits per value), fake or None)."""
        flat, ro, C, n = _rows(x, row_offsets)
        total = flat.size
        m = np.ascontiguousarray(m, dtype=np.float32)
        p = np.ascontiguousarray(p, dtype=np.float32).reshape(-1, 3)
        assert m.size == C and p.shape[0] == C
        codes = np.empty(code_bytes(total, bits, layout), dtype=np.uint8)
        region = np.empty((total + 3) // 4, dtype=np.uint8)
        fake = np.empty(total, dtype=np.float32) if want_fake else None
        _check(self._lib.pwlq_oracle_quantize3(_ptr(flat), _ptr(ro), C, n, int(bits), _ptr(m),
                                               _ptr(p), _ptr(codes), _ptr(region), _ptr(fake),
                                               int(layout)), "quantize3")
        return codes, region, fake

    def dequantize3(self, codes, region, bits, m, p, C=None, n=None, layout=0, row_offsets=None):
        codes = np.ascontiguousarray(codes, dtype=np.uint8)
        region = np.ascontiguousarray(region, dtype=np.uint8)
        m = np.ascontiguousarray(m, dtype=np.float32)
        p = np.ascontiguousarray(p, dtype=np.float32).reshape(-1, 3)
        if row_offsets is not None:
            ro = np.ascontiguousarray(row_offsets, dtype=np.int64)
            C, n, total = ro.size - 1, 0, int(ro[-1])
        else:
            ro, total = None, int(C) * int(n)
        assert m.size == C and p.shape[0] == C
        y = np.empty(total, dtype=np.float32)
        _check(self._lib.pwlq_oracle_dequantize3(_ptr(codes), _ptr(region), _ptr(ro), C, n,
                                                 int(bits), _ptr(m), _ptr(p), _ptr(y),
                                                 int(layout)), "dequantize3")
        return y

    # ---- bias correction (folded scale xi and offset beta per row) and dense (b+1)-bit storage
    def bias_correction(self, x, bits, m, p, row_offsets=None):
        """Returns (xi float32 [C], beta float32 [C])."""
        flat, ro, C, n = _rows(x, row_offsets)
        m = np.ascontiguousarray(m, dtype=np.float32)
        p = np.ascontiguousarray(p, dtype=np.float32)
        assert m.size == C and p.size == C
        xi = np.empty(C, dtype=np.float32)
        beta = np.empty(C, dtype=np.float32)
        _check(self._lib.pwlq_oracle_bias_correction(_ptr(flat), _ptr(ro), C, n, int(bits), _ptr(m),
                                                     _ptr(p), _ptr(xi), _ptr(beta)),
               "bias_correction")
        return xi, beta

    def dequantize_bc(self, codes, mask, bits, m, p, xi, beta, C=None, n=None, layout=0,
                      row_offsets=None):
        codes = np.ascontiguousarray(codes, dtype=np.uint8)
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
        m, p, xi, beta = (np.ascontiguousarray(v, dtype=np.float32) for v in (m, p, xi, beta))
        if row_offsets is not None:
            ro = np.ascontiguousarray(row_offsets, dtype=np.int64)
            C, n, total = ro.size - 1, 0, int(ro[-1])
        else:
            ro, total = None, int(C) * int(n)
        assert m.size == C and p.size == C and xi.size == C and beta.size == C
        y = np.empty(total, dtype=np.float32)
        _check(self._lib.pwlq_oracle_dequantize_bc(_ptr(codes), _ptr(mask), _ptr(ro), C, n,
                                                   int(bits), _ptr(m), _ptr(p), _ptr(xi),
                                                   _ptr(beta), _ptr(y), int(layout)),
               "dequantize_bc")
        return y

    def pack_dense(self, codes_u8, mask, bits):
        codes_u8 = np.ascontiguousarray(codes_u8, dtype=np.uint8)
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
        total = codes_u8.size
        out = np.empty((total * (bits + 1) + 7) // 8, dtype=np.uint8)
        _check(self._lib.pwlq_oracle_pack_dense(_ptr(codes_u8), _ptr(mask), total, int(bits),
                                                _ptr(out)), "pack_dense")
        return out

    def unpack_dense(self, stream, total, bits):
        stream = np.ascontiguousarray(stream, dtype=np.uint8)
        codes = np.empty(total, dtype=np.uint8)
        mask = np.empty((total + 7) // 8, dtype=np.uint8)
        _check(self._lib.pwlq_oracle_unpack_dense(_ptr(stream), int(total), int(bits), _ptr(codes),
                                                  _ptr(mask)), "unpack_dense")
        return codes, mask

    def params(self, m, p, bits):
        """(L, s1, inv1, s2, inv2) as binary32 values."""
        out = np.empty(5, dtype=np.float32)
        self._lib.pwlq_oracle_params(float(m), float(p), int(bits), _ptr(out))
        return out


_default = None


def _get() -> OracleLib:
    global _default
    if _default is None:
        _default = OracleLib()
    return _default


def __getattr__(name):
    """Module-level access to the default oracle's methods: ``pwlq_oracle.search(...)`` is
    ``OracleLib().search(...)`` on one shared instance."""
    if not name.startswith("_") and callable(getattr(OracleLib, name, None)):
        return getattr(_get(), name)
    raise AttributeError(name)
