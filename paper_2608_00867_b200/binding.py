"""ctypes binding of ``include/nuna.h``: same names, argument marshalling only.

Rank buffers are passed as sequences of torch CUDA tensors (or raw device
addresses); every step of every collective runs in the library's CUDA kernels.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

NUNA_OK = 0
NUNA_ERR_INVALID_ARG = 1
NUNA_ERR_UNSUPPORTED_DTYPE = 2
NUNA_ERR_ALIGNMENT = 3
NUNA_ERR_ALIAS = 4
NUNA_ERR_CUDA = 5
NUNA_ERR_TIMEOUT = 6
NUNA_ERR_CAPTURING = 7
NUNA_ERR_TOO_MANY_RANKS = 8
NUNA_ERR_TOO_LARGE = 9

NUNA_BF16, NUNA_F16, NUNA_F32 = 0, 1, 2
NUNA_MAX_RANKS = 16
NUNA_PLACE_ROUNDROBIN, NUNA_PLACE_AWARE, NUNA_PLACE_AUTO = 0, 1, 2
NUNA_TWOSHOT_PUT = 16
NUNA_HINT_RESIDENT = 32
NUNA_LAUNCH_PDL = 64

_LIB_PATH = os.environ.get("NUNA_LIB") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libnuna.so")
_lib = None


class NunaError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: {status_string(status)} (status {status})")
        self.status = status


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2608_00867_b200.build` "
                               "(the collectives have no CPU fallback)")
        L = ctypes.CDLL(_LIB_PATH)
        vpp = ctypes.POINTER(ctypes.c_void_p)
        coll = [vpp, vpp, ctypes.c_int, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint, ctypes.c_void_p]
        for name in ("nuna_allreduce_oneshot", "nuna_allreduce_twoshot", "nuna_reduce_scatter", "nuna_allgather"):
            getattr(L, name).argtypes = coll
            getattr(L, name).restype = ctypes.c_int
        L.nuna_allreduce_host.argtypes = [vpp, vpp, ctypes.c_int, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint, ctypes.c_int]
        L.nuna_allreduce_host.restype = ctypes.c_int
        L.nuna_init.argtypes = [ctypes.c_size_t]
        L.nuna_init.restype = ctypes.c_int
        L.nuna_device_status.argtypes = [ctypes.POINTER(ctypes.c_int)]
        L.nuna_device_status.restype = ctypes.c_int
        L.nuna_launch_floor.argtypes = [ctypes.c_uint, ctypes.c_uint, ctypes.c_void_p]
        L.nuna_launch_floor.restype = ctypes.c_int
        L.nuna_chain_create.argtypes = [vpp, vpp, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_size_t, ctypes.c_int,
                                        ctypes.c_uint, ctypes.c_int, ctypes.POINTER(ctypes.c_void_p)]
        L.nuna_chain_create.restype = ctypes.c_int
        L.nuna_chain_launch.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        L.nuna_chain_launch.restype = ctypes.c_int
        L.nuna_chain_destroy.argtypes = [ctypes.c_void_p]
        L.nuna_chain_destroy.restype = ctypes.c_int
        L.nuna_launch_count.argtypes = []
        L.nuna_launch_count.restype = ctypes.c_ulonglong
        L.nuna_status_string.argtypes = [ctypes.c_int]
        L.nuna_status_string.restype = ctypes.c_char_p
        L.nuna_shutdown.argtypes = []
        L.nuna_shutdown.restype = ctypes.c_int
        L.nuna_debug_barrier_selftest.argtypes = [ctypes.c_uint, ctypes.c_uint, ctypes.c_uint, ctypes.POINTER(ctypes.c_uint)]
        L.nuna_debug_barrier_selftest.restype = ctypes.c_int
        _lib = L
    return _lib


def _addr(x) -> int:
    return int(x.data_ptr()) if hasattr(x, "data_ptr") else int(x)


def ptr_table(bufs: Sequence):
    tab = (ctypes.c_void_p * max(len(bufs), 1))()
    for i, b in enumerate(bufs):
        tab[i] = _addr(b)
    return tab


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    if hasattr(stream, "cuda_stream"):
        return stream.cuda_stream or None
    return int(stream) or None


def _finish(status: int, what: str, check: bool) -> int:
    if check and status != NUNA_OK:
        raise NunaError(status, what)
    return status


def _collective(name, src, dst, count, dtype, flags, stream, check, nranks=None):
    n = len(src) if nranks is None else nranks
    st = getattr(lib(), name)(ptr_table(src), ptr_table(dst), n, count, dtype, flags, _stream(stream))
    return _finish(st, name, check)


def nuna_init(scratch_bytes: int = 0, check: bool = True) -> int:
    return _finish(lib().nuna_init(scratch_bytes), "nuna_init", check)


def nuna_allreduce_oneshot(src, dst, count, dtype=NUNA_BF16, flags=0, stream=None, check=True, nranks=None) -> int:
    return _collective("nuna_allreduce_oneshot", src, dst, count, dtype, flags, stream, check, nranks)


def nuna_allreduce_twoshot(src, dst, count, dtype=NUNA_BF16, flags=0, stream=None, check=True, nranks=None) -> int:
    return _collective("nuna_allreduce_twoshot", src, dst, count, dtype, flags, stream, check, nranks)


def nuna_reduce_scatter(src, dst, shard_count, dtype=NUNA_BF16, flags=0, stream=None, check=True, nranks=None) -> int:
    return _collective("nuna_reduce_scatter", src, dst, shard_count, dtype, flags, stream, check, nranks)


def nuna_allgather(src, dst, shard_count, dtype=NUNA_BF16, flags=0, stream=None, check=True, nranks=None) -> int:
    return _collective("nuna_allgather", src, dst, shard_count, dtype, flags, stream, check, nranks)


def nuna_allreduce_host(src, dst, count, dtype=NUNA_BF16, flags=0, two_shot=False, check=True) -> int:
    """``src`` / ``dst``: host buffers (numpy arrays, CPU tensors or addresses)."""
    def haddr(x):
        if hasattr(x, "ctypes"):
            return x.ctypes.data
        return _addr(x)
    s = (ctypes.c_void_p * len(src))(*[haddr(x) for x in src])
    d = (ctypes.c_void_p * len(dst))(*[haddr(x) for x in dst])
    st = lib().nuna_allreduce_host(s, d, len(src), count, dtype, flags, 1 if two_shot else 0)
    return _finish(st, "nuna_allreduce_host", check)


def nuna_chain_create(src_sets, dst_sets, nnodes, count, dtype=NUNA_BF16, flags=0, two_shot=False, check=True):
    """``src_sets`` / ``dst_sets``: sequences (one per buffer set) of per-rank buffers.  Returns a handle."""
    nsets, nranks = len(src_sets), len(src_sets[0])
    flat_s = [b for s in src_sets for b in s]
    flat_d = [b for s in dst_sets for b in s]
    handle = ctypes.c_void_p()
    st = lib().nuna_chain_create(ptr_table(flat_s), ptr_table(flat_d), nsets, nnodes, nranks, count, dtype, flags,
                                 1 if two_shot else 0, ctypes.byref(handle))
    _finish(st, "nuna_chain_create", check)
    return handle if st == NUNA_OK else st


def nuna_chain_launch(chain, stream=None, check=True) -> int:
    return _finish(lib().nuna_chain_launch(chain, _stream(stream)), "nuna_chain_launch", check)


def nuna_chain_destroy(chain) -> int:
    return lib().nuna_chain_destroy(chain)


def nuna_device_status() -> int:
    out = ctypes.c_int(0)
    st = lib().nuna_device_status(ctypes.byref(out))
    if st != NUNA_OK:
        raise NunaError(st, "nuna_device_status")
    return out.value


def nuna_launch_floor(blocks: int, flags: int = 0, stream=None, check: bool = True) -> int:
    return _finish(lib().nuna_launch_floor(blocks, flags, _stream(stream)), "nuna_launch_floor", check)


def nuna_launch_count() -> int:
    return int(lib().nuna_launch_count())


def status_string(status: int) -> str:
    return lib().nuna_status_string(status).decode()


nuna_status_string = status_string


def nuna_shutdown() -> int:
    return lib().nuna_shutdown()


def debug_barrier_selftest(grid: int, expected: int, timeout_ms: int):
    passed = ctypes.c_uint(0)
    st = lib().nuna_debug_barrier_selftest(grid, expected, timeout_ms, ctypes.byref(passed))
    return st, passed.value
