"""B200-native emulated-rank collectives (one-shot / two-shot allreduce, reduce-scatter,
allgather) behind a C ABI, with a thin ctypes binding of the same names.

Importing the package loads nothing; the first call into ``binding`` loads
``libnuna.so`` (built in-tree by ``build.build()``) and raises if it is missing.
There is no CPU fallback.
"""
from . import workloads  # noqa: F401  (pure input generation; no native code)

__all__ = ["workloads", "binding", "build"]
