"""QLESS hot path on B200 (sm_100a): quantized gradient datastore construction and search.

The arithmetic lives in the CUDA library built from ``csrc/`` (C ABI declared in
``include/qless.h``); :mod:`.binding` marshals torch device tensors into those calls.
Importing this package loads nothing; the first call loads the shared library and raises
if it has not been built.
"""
from . import workloads  # noqa: F401  (input generators only; no CUDA needed)

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
