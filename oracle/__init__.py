"""CPU oracle for the PWLQ hot path -- test infrastructure only.

Only the tests, the smoke check and the benchmark's CPU-baseline leg import
this package.  It shares no code with the CUDA path.
"""
from . import pwlq_oracle as _impl
from .pwlq_oracle import OracleError, OracleLib, build, code_bytes  # noqa: F401


def __getattr__(name):
    """``oracle.search(...)`` and the like: methods of one shared ``OracleLib``."""
    return getattr(_impl, name)
