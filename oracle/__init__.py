"""CPU oracle for the PWLQ hot path -- test infrastructure only.

Only the tests, the smoke check and the benchmark's CPU-baseline leg import
this package.  It shares no code with the CUDA path.
"""
from .pwlq_oracle import (  # noqa: F401
    OracleError, OracleLib, absmax, analytic_p, bias_correction, build, code_bytes, dequantize,
    dequantize2, dequantize_bc, pack_dense, unpack_dense,
    dequantize_u, elem,
    elem_u, minmax, params, quantize, quantize2, quantize_u, search, search2, search_u,
    select_analytic,
)
