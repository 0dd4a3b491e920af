"""CPU oracle for the emulated collectives -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It does not import the CUDA package and shares nothing with it.

``nuna_oracle.c`` is the plain definition (bf16 storage, binary32 fold in rank
order, one final round to nearest even); this module compiles it with gcc and
exposes it over numpy ``uint16`` arrays.  ``exact_model`` is a second, exact
rational-arithmetic model used to pin the C code on small inputs, and
``nap_planner`` restates the paper's placement algorithm (Algorithm 1).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nuna_oracle.c")
_LIB = os.path.join(_HERE, "libnuna_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc, -O2, strict IEEE: no fast-math) and return the library path."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-fno-fast-math", "-ffp-contract=off", "-fopenmp",
           "-fPIC", "-shared", "-Wall", "-Wextra", "-o", tmp, _SRC]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        pp = ctypes.POINTER(ctypes.c_void_p)
        for name in ("nuna_oracle_allreduce_bf16", "nuna_oracle_reduce_scatter_bf16",
                     "nuna_oracle_allgather_bf16", "nuna_oracle_alltoall_bf16"):
            fn = getattr(lib, name)
            fn.argtypes = [pp, pp, ctypes.c_int, ctypes.c_size_t, ctypes.c_int]
            fn.restype = None
        for name in ("nuna_oracle_allreduce_f16", "nuna_oracle_allreduce_f32",
                     "nuna_oracle_reduce_scatter_f16", "nuna_oracle_reduce_scatter_f32"):
            fn = getattr(lib, name)
            fn.argtypes = [pp, pp, ctypes.c_int, ctypes.c_size_t, ctypes.c_int]
            fn.restype = None
        lib.nuna_oracle_rne_f16.argtypes = [ctypes.c_float]
        lib.nuna_oracle_rne_f16.restype = ctypes.c_uint16
        lib.nuna_oracle_widen_f16.argtypes = [ctypes.c_uint16]
        lib.nuna_oracle_widen_f16.restype = ctypes.c_float
        lib.nuna_oracle_fold_bf16.argtypes = [ctypes.c_void_p, ctypes.c_int]
        lib.nuna_oracle_fold_bf16.restype = ctypes.c_uint16
        lib.nuna_oracle_rne_bf16.argtypes = [ctypes.c_float]
        lib.nuna_oracle_rne_bf16.restype = ctypes.c_uint16
        lib.nuna_oracle_widen_bf16.argtypes = [ctypes.c_uint16]
        lib.nuna_oracle_widen_bf16.restype = ctypes.c_float
        _lib = lib
    return _lib


# Element types.  Buffers are raw bit patterns: uint16 for bf16 / f16, uint32 for f32.
STORAGE = {"bf16": np.uint16, "f16": np.uint16, "f32": np.uint32}


def _ptrs(arrs: Sequence[np.ndarray]):
    tab = (ctypes.c_void_p * len(arrs))()
    for i, a in enumerate(arrs):
        assert a.dtype in (np.uint16, np.uint32) and a.flags.c_contiguous
        tab[i] = a.ctypes.data
    return tab


def _check_src(src: Sequence[np.ndarray], length: int, storage=np.uint16):
    if len(src) < 1:
        raise ValueError("need at least one rank")
    for a in src:
        if a.dtype != storage or a.ndim != 1 or len(a) != length:
            raise ValueError(f"every rank buffer must be a 1-D {np.dtype(storage).name} array of the same length")


def allreduce(src: Sequence[np.ndarray], nthreads: int = 1, dtype: str = "bf16",
              out: Sequence[np.ndarray] = None) -> List[np.ndarray]:
    """One result array per destination rank (all equal by definition).

    ``out``: optional destination arrays to write into (one per rank, same shape and storage type as the
    sources).  Without it fresh arrays are allocated on every call, and a timing of repeated calls then
    measures the allocator's page faults as much as the fold."""
    n, count = len(src), len(src[0])
    _check_src(src, count, STORAGE[dtype])
    src = [np.ascontiguousarray(a) for a in src]
    if out is None:
        dst = [np.empty(count, dtype=STORAGE[dtype]) for _ in range(n)]
    else:
        if len(out) != n:
            raise ValueError("need one destination per rank")
        _check_src(out, count, STORAGE[dtype])
        if not all(a.flags.c_contiguous and a.flags.writeable for a in out):
            raise ValueError("destinations must be contiguous and writeable")
        dst = list(out)
    getattr(_load(), f"nuna_oracle_allreduce_{dtype}")(_ptrs(src), _ptrs(dst), n, count, int(nthreads))
    return dst


def reduce_scatter(src: Sequence[np.ndarray], nthreads: int = 1, dtype: str = "bf16") -> List[np.ndarray]:
    """``src[k]`` holds ``N*S`` elements; returns N arrays of S elements."""
    n, total = len(src), len(src[0])
    _check_src(src, total, STORAGE[dtype])
    if total % n:
        raise ValueError("source length must be a multiple of the rank count")
    shard = total // n
    src = [np.ascontiguousarray(a) for a in src]
    dst = [np.empty(shard, dtype=STORAGE[dtype]) for _ in range(n)]
    getattr(_load(), f"nuna_oracle_reduce_scatter_{dtype}")(_ptrs(src), _ptrs(dst), n, shard, int(nthreads))
    return dst


def allgather(src: Sequence[np.ndarray], nthreads: int = 1) -> List[np.ndarray]:
    """``src[r]`` holds S elements; returns N arrays of ``N*S`` elements."""
    n, shard = len(src), len(src[0])
    _check_src(src, shard)
    src = [np.ascontiguousarray(a) for a in src]
    dst = [np.empty(n * shard, dtype=np.uint16) for _ in range(n)]
    _load().nuna_oracle_allgather_bf16(_ptrs(src), _ptrs(dst), n, shard, int(nthreads))
    return dst


def alltoall(src: Sequence[np.ndarray], nthreads: int = 1) -> List[np.ndarray]:
    """``src[r]`` holds N blocks of S elements (block d goes to rank d); returns N arrays of ``N*S``."""
    n, total = len(src), len(src[0])
    _check_src(src, total)
    if total % n:
        raise ValueError("source length must be a multiple of the rank count")
    src = [np.ascontiguousarray(a) for a in src]
    dst = [np.empty(total, dtype=np.uint16) for _ in range(n)]
    _load().nuna_oracle_alltoall_bf16(_ptrs(src), _ptrs(dst), n, total // n, int(nthreads))
    return dst


def fold(vals) -> int:
    """Rank-ordered sum of one column of bf16 patterns."""
    a = np.ascontiguousarray(np.asarray(vals, dtype=np.uint16))
    return int(_load().nuna_oracle_fold_bf16(a.ctypes.data, len(a)))


def rne_f16(x: float) -> int:
    return int(_load().nuna_oracle_rne_f16(x))


def widen_f16(h: int) -> float:
    return float(_load().nuna_oracle_widen_f16(h))


def rne_bf16(x: float) -> int:
    return int(_load().nuna_oracle_rne_bf16(x))


def widen_bf16(h: int) -> float:
    return float(_load().nuna_oracle_widen_bf16(h))
