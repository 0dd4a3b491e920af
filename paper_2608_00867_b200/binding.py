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
DTYPE_BY_NAME = {"bf16": NUNA_BF16, "f16": NUNA_F16, "f32": NUNA_F32}
ELEM_SIZE = {NUNA_BF16: 2, NUNA_F16: 2, NUNA_F32: 4}
NUNA_MAX_RANKS = 16
NUNA_PLACE_ROUNDROBIN, NUNA_PLACE_AWARE, NUNA_PLACE_AUTO = 0, 1, 2
NUNA_TWOSHOT_PUT = 16
NUNA_HINT_RESIDENT = 32
NUNA_LAUNCH_PDL = 64
NUNA_PLACE_SM_LISTS = 128
NUNA_PLACE_CLUSTER = 256
NUNA_PLACE_STAGED = 512
NUNA_TWOSHOT_SYNC = 1024
NUNA_CHAIN_PERSISTENT = 2048
NUNA_CHAIN_GRAPH = 4096
NUNA_TWOSHOT_SYS_SCOPE = 8192
NUNA_PLACE_REGS = 16384

NUNA_MAX_SMS, NUNA_MAX_PROBE_BUFS, NUNA_PROBE_REGIONS, NUNA_MAX_PROBE_LINES = 256, 32, 8, 2048
NUNA_TOPO_UNIFORM, NUNA_TOPO_NONUNIFORM = 0, 1
NUNA_HIST_BINS, NUNA_HIST_FIRST, NUNA_HIST_STEP = 48, 200, 4
NUNA_SCAN_LINES, NUNA_SCAN_RUN_BINS, NUNA_SCAN_LEVELS, NUNA_SCAN_BLOCKS = 512, 16, 3, 8
NUNA_OPT_BLOCKS, NUNA_OPT_UNROLL, NUNA_OPT_COLOC, NUNA_OPT_AUTO_MIN_BYTES, NUNA_OPT_TIMEOUT_MS = 0, 1, 2, 3, 4
NUNA_OPT_DOMAINS, NUNA_OPT_STAGE_VECS, NUNA_OPT_TWOSHOT_VECS, NUNA_OPT_AG_BULK_VECS = 5, 6, 7, 8
NUNA_OPT_REGS_VECS, NUNA_OPT_PREFETCH = 9, 10


class NunaTopology(ctypes.Structure):
    """Mirror of ``nuna_topology_t`` (include/nuna.h)."""
    _fields_ = [
        ("num_sms", ctypes.c_int), ("sms_reported", ctypes.c_int),
        ("num_bufs", ctypes.c_int), ("num_regions", ctypes.c_int), ("num_lines", ctypes.c_int),
        ("num_domains", ctypes.c_int), ("verdict", ctypes.c_int),
        ("chain_nodes", ctypes.c_int), ("chain_steps", ctypes.c_int), ("chain_walk_ok", ctypes.c_int),
        ("self_pointer_mismatches", ctypes.c_int),
        ("nonuniformity", ctypes.c_float), ("noise", ctypes.c_float),
        ("near_lat", ctypes.c_float), ("far_lat", ctypes.c_float), ("domain_gap", ctypes.c_float),
        ("sm_reported", ctypes.c_int * NUNA_MAX_SMS),
        ("sm_domain", ctypes.c_int * NUNA_MAX_SMS),
        ("sm_lat_hit", ctypes.c_float * NUNA_MAX_SMS),
        ("sm_lat_miss", ctypes.c_float * NUNA_MAX_SMS),
        ("lat_hit", (ctypes.c_float * NUNA_MAX_PROBE_BUFS) * NUNA_MAX_SMS),
        ("region_home0", (ctypes.c_float * NUNA_PROBE_REGIONS) * NUNA_MAX_PROBE_BUFS),
        ("line_buf", ctypes.c_ubyte * NUNA_MAX_PROBE_LINES),
        ("line_region", ctypes.c_ubyte * NUNA_MAX_PROBE_LINES),
        ("line_home", ctypes.c_ubyte * NUNA_MAX_PROBE_LINES),
        ("hist_near", ctypes.c_uint * NUNA_HIST_BINS),
        ("hist_far", ctypes.c_uint * NUNA_HIST_BINS),
        ("scan_lines", ctypes.c_int), ("scan_longest_run", ctypes.c_int),
        ("scan_home", ctypes.c_ubyte * NUNA_SCAN_LINES),
        ("scan_run_hist", ctypes.c_uint * NUNA_SCAN_RUN_BINS),
        ("scan_level_share", (ctypes.c_float * NUNA_SCAN_BLOCKS) * NUNA_SCAN_LEVELS),
        ("scan_level_spread", ctypes.c_float * NUNA_SCAN_LEVELS),
        ("sm_read_gbs", ctypes.c_float * NUNA_MAX_SMS),
    ]


class NunaPlanInput(ctypes.Structure):
    """Mirror of ``nuna_plan_input_t`` (include/nuna.h)."""
    _ip, _lp = ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_longlong)
    _fields_ = [
        ("num_tbs", ctypes.c_int), ("tb_gpu", _ip), ("tb_chunk_begin", _ip), ("tb_chunks", _ip),
        ("num_chunks", ctypes.c_int), ("chunk_bytes", _lp),
        ("num_cus", ctypes.c_int), ("cu_domain", _ip), ("cu_rank", _ip),
        ("num_stacks", ctypes.c_int), ("cu_stack", _ip),
        ("r_max_cu", ctypes.c_longlong), ("r_max_stack", ctypes.c_longlong), ("nar_max", ctypes.c_int),
    ]


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
        for name in ("nuna_allreduce", "nuna_allreduce_oneshot", "nuna_allreduce_twoshot", "nuna_reduce_scatter", "nuna_allgather",
                     "nuna_alltoall"):
            getattr(L, name).argtypes = coll
            getattr(L, name).restype = ctypes.c_int
        L.nuna_allreduce_twoshot_static.argtypes = [vpp, vpp, ctypes.c_int, ctypes.c_size_t, ctypes.c_int, ctypes.c_void_p]
        L.nuna_allreduce_twoshot_static.restype = ctypes.c_int
        L.nuna_allreduce_host.argtypes = [vpp, vpp, ctypes.c_int, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint, ctypes.c_int]
        L.nuna_allreduce_host.restype = ctypes.c_int
        L.nuna_set_option.argtypes = [ctypes.c_int, ctypes.c_longlong]
        L.nuna_set_option.restype = ctypes.c_int
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
        L.nuna_probe_topology.argtypes = [vpp, ctypes.POINTER(ctypes.c_size_t), ctypes.c_int,
                                          ctypes.POINTER(NunaTopology), ctypes.c_void_p]
        L.nuna_probe_topology.restype = ctypes.c_int
        L.nuna_debug_analyse_topology.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float),
                                                  ctypes.c_int, ctypes.c_int, ctypes.POINTER(NunaTopology)]
        L.nuna_debug_analyse_topology.restype = ctypes.c_int
        L.nuna_debug_chain.argtypes = [ctypes.POINTER(ctypes.c_uint), ctypes.c_int, ctypes.c_ulonglong, ctypes.c_uint,
                                       ctypes.c_int, ctypes.POINTER(ctypes.c_uint)]
        L.nuna_debug_chain.restype = ctypes.c_int
        up = ctypes.POINTER(ctypes.c_uint)
        L.nuna_debug_plan_oneshot.argtypes = [ctypes.POINTER(NunaTopology), ctypes.c_int, ctypes.c_int, ctypes.c_size_t,
                                              ctypes.c_size_t, ctypes.c_int, ctypes.c_int, up, up]
        L.nuna_debug_plan_oneshot.restype = ctypes.c_int
        ip = ctypes.POINTER(ctypes.c_int)
        L.nuna_plan_placement.argtypes = [ctypes.POINTER(NunaPlanInput), ip, ip, ip, ip]
        L.nuna_plan_placement.restype = ctypes.c_int
        L.nuna_launch_count.argtypes = []
        L.nuna_launch_count.restype = ctypes.c_ulonglong
        L.nuna_status_string.argtypes = [ctypes.c_int]
        L.nuna_status_string.restype = ctypes.c_char_p
        L.nuna_shutdown.argtypes = []
        L.nuna_shutdown.restype = ctypes.c_int
        L.nuna_debug_barrier_selftest.argtypes = [ctypes.c_uint, ctypes.c_uint, ctypes.c_uint, ctypes.POINTER(ctypes.c_uint)]
        L.nuna_debug_barrier_selftest.restype = ctypes.c_int
        L.nuna_debug_access_latency.argtypes = [vpp, vpp, ctypes.c_size_t, ctypes.c_int, ctypes.POINTER(ctypes.c_uint)]
        L.nuna_debug_access_latency.restype = ctypes.c_int
        L.nuna_debug_oneshot_regs_traced.argtypes = [vpp, vpp, ctypes.c_size_t, ctypes.c_uint, ctypes.c_uint, ctypes.c_void_p,
                                                     ctypes.POINTER(ctypes.c_uint), ctypes.c_void_p]
        L.nuna_debug_oneshot_regs_traced.restype = ctypes.c_int
        L.nuna_debug_launch_floor.argtypes = [ctypes.c_uint, ctypes.c_uint, ctypes.c_int, ctypes.c_void_p]
        L.nuna_debug_launch_floor.restype = ctypes.c_int
        L.nuna_debug_twoshot.argtypes = [vpp, vpp, ctypes.c_int, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint, ctypes.c_uint]
        L.nuna_debug_twoshot.restype = ctypes.c_int
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


def nuna_set_option(option: int, value: int, check: bool = True) -> int:
    return _finish(lib().nuna_set_option(option, value), "nuna_set_option", check)


def nuna_allreduce_oneshot(src, dst, count, dtype=NUNA_BF16, flags=0, stream=None, check=True, nranks=None) -> int:
    return _collective("nuna_allreduce_oneshot", src, dst, count, dtype, flags, stream, check, nranks)


def nuna_allreduce(src, dst, count, dtype=NUNA_BF16, flags=0, stream=None, check=True, nranks=None) -> int:
    return _collective("nuna_allreduce", src, dst, count, dtype, flags, stream, check, nranks)


def nuna_allreduce_twoshot(src, dst, count, dtype=NUNA_BF16, flags=0, stream=None, check=True, nranks=None) -> int:
    return _collective("nuna_allreduce_twoshot", src, dst, count, dtype, flags, stream, check, nranks)


def nuna_reduce_scatter(src, dst, shard_count, dtype=NUNA_BF16, flags=0, stream=None, check=True, nranks=None) -> int:
    return _collective("nuna_reduce_scatter", src, dst, shard_count, dtype, flags, stream, check, nranks)


def nuna_allgather(src, dst, shard_count, dtype=NUNA_BF16, flags=0, stream=None, check=True, nranks=None) -> int:
    return _collective("nuna_allgather", src, dst, shard_count, dtype, flags, stream, check, nranks)


def nuna_alltoall(src, dst, block_count, dtype=NUNA_BF16, flags=0, stream=None, check=True, nranks=None) -> int:
    return _collective("nuna_alltoall", src, dst, block_count, dtype, flags, stream, check, nranks)


NUNA_STATIC_MAX_COUNT = 2 * 1024 * 1024


def nuna_allreduce_twoshot_static(src, dst, count, dtype=NUNA_BF16, stream=None, check=True) -> int:
    """The two-shot allreduce that never allocates: its scratch is a fixed array inside the library
    (at most NUNA_STATIC_MAX_COUNT elements per rank).  For callers that cannot call cudaMalloc."""
    st = lib().nuna_allreduce_twoshot_static(ptr_table(src), ptr_table(dst), len(src), count, dtype, _stream(stream))
    return _finish(st, "nuna_allreduce_twoshot_static", check)


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


def nuna_probe_topology(bufs, nbytes=None, stream=None, check=True):
    """Probes the given device buffers; returns a ``NunaTopology`` (or the status when check=False fails)."""
    if nbytes is None:
        nbytes = [b.numel() * b.element_size() for b in bufs]
    sizes = (ctypes.c_size_t * len(bufs))(*[int(x) for x in nbytes])
    topo = NunaTopology()
    st = lib().nuna_probe_topology(ptr_table(bufs), sizes, len(bufs), ctypes.byref(topo), _stream(stream))
    _finish(st, "nuna_probe_topology", check)
    return topo if st == NUNA_OK else st


def debug_analyse_topology(lat, lat_rep):
    """Host-side clustering / verdict on a caller-supplied (num_sms x num_lines) float32 latency matrix."""
    import numpy as np
    a = np.ascontiguousarray(lat, dtype=np.float32)
    b = np.ascontiguousarray(lat_rep, dtype=np.float32)
    topo = NunaTopology()
    fp = ctypes.POINTER(ctypes.c_float)
    st = lib().nuna_debug_analyse_topology(a.ctypes.data_as(fp), b.ctypes.data_as(fp), a.shape[0], a.shape[1],
                                           ctypes.byref(topo))
    if st != NUNA_OK:
        raise NunaError(st, "nuna_debug_analyse_topology")
    return topo


def debug_plan_oneshot(topo, num_sms: int, nranks: int, ntiles: int, tile_bytes: int, generic: bool, domains: int = 0):
    """Per-SM work lists planned for a one-shot: returns a list (one entry per SM) of tile lists."""
    import numpy as np
    off = np.zeros(num_sms + 1, dtype=np.uint32)
    tiles = np.zeros(max(ntiles, 1), dtype=np.uint32)
    up = ctypes.POINTER(ctypes.c_uint)
    st = lib().nuna_debug_plan_oneshot(ctypes.byref(topo) if topo is not None else None, num_sms, nranks, ntiles,
                                       tile_bytes, 1 if generic else 0, domains, off.ctypes.data_as(up),
                                       tiles.ctypes.data_as(up))
    if st != NUNA_OK:
        raise NunaError(st, "nuna_debug_plan_oneshot")
    return [tiles[off[s]:off[s + 1]].tolist() for s in range(num_sms)]


def debug_chain(nnodes: int, seed: int, start: int, steps: int):
    """The probe's single-cycle permutation and the node a host walk of `steps` steps ends on."""
    import numpy as np
    nxt = np.zeros(nnodes, dtype=np.uint32)
    end = ctypes.c_uint(0)
    st = lib().nuna_debug_chain(nxt.ctypes.data_as(ctypes.POINTER(ctypes.c_uint)), nnodes, seed, start, steps,
                                ctypes.byref(end))
    if st != NUNA_OK:
        raise NunaError(st, "nuna_debug_chain")
    return nxt, end.value


def nuna_plan_placement(tb_gpu, tb_chunks, chunk_bytes, cu_domain, cu_rank, cu_stack, num_stacks,
                        r_max_cu, r_max_stack, nar_max, check=True):
    """Algorithm 1 on the host.  ``tb_chunks``: one list of chunk ids per thread block.
    Returns (m_compute, m_memory, tb_domain, tb_group) as lists."""
    import numpy as np
    T, C, U = len(tb_gpu), len(chunk_bytes), len(cu_domain)
    begin = np.zeros(T + 1, dtype=np.int32)
    for t, cs in enumerate(tb_chunks):
        begin[t + 1] = begin[t] + len(cs)
    flat = np.array([c for cs in tb_chunks for c in cs] or [0], dtype=np.int32)
    arrs = {
        "tb_gpu": np.array(list(tb_gpu) or [0], dtype=np.int32), "begin": begin, "flat": flat,
        "bytes": np.array(list(chunk_bytes) or [0], dtype=np.int64),
        "dom": np.array(cu_domain, dtype=np.int32), "rank": np.array(cu_rank, dtype=np.int32),
        "stack": np.array(cu_stack, dtype=np.int32),
    }
    ip, lp = ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_longlong)
    inp = NunaPlanInput(T, arrs["tb_gpu"].ctypes.data_as(ip), arrs["begin"].ctypes.data_as(ip),
                        arrs["flat"].ctypes.data_as(ip), C, arrs["bytes"].ctypes.data_as(lp), U,
                        arrs["dom"].ctypes.data_as(ip), arrs["rank"].ctypes.data_as(ip), num_stacks,
                        arrs["stack"].ctypes.data_as(ip), r_max_cu, r_max_stack, nar_max)
    mc = np.full(max(T, 1), -1, dtype=np.int32)
    mm = np.full(max(C, 1), -1, dtype=np.int32)
    td = np.full(max(T, 1), -1, dtype=np.int32)
    tg = np.full(max(T, 1), -1, dtype=np.int32)
    st = lib().nuna_plan_placement(ctypes.byref(inp), mc.ctypes.data_as(ip), mm.ctypes.data_as(ip),
                                   td.ctypes.data_as(ip), tg.ctypes.data_as(ip))
    _finish(st, "nuna_plan_placement", check)
    if st != NUNA_OK:
        return st
    return mc[:T].tolist(), mm[:C].tolist(), td[:T].tolist(), tg[:T].tolist()


def nuna_device_status() -> int:
    out = ctypes.c_int(0)
    st = lib().nuna_device_status(ctypes.byref(out))
    if st != NUNA_OK:
        raise NunaError(st, "nuna_device_status")
    return out.value


def nuna_launch_floor(blocks: int, flags: int = 0, stream=None, check: bool = True) -> int:
    return _finish(lib().nuna_launch_floor(blocks, flags, _stream(stream)), "nuna_launch_floor", check)


def debug_launch_floor(blocks: int, flags: int = 0, trigger_first: bool = False, stream=None) -> int:
    return _finish(lib().nuna_debug_launch_floor(blocks, flags, 1 if trigger_first else 0, _stream(stream)),
                   "nuna_debug_launch_floor", True)


def nuna_launch_count() -> int:
    return int(lib().nuna_launch_count())


def status_string(status: int) -> str:
    return lib().nuna_status_string(status).decode()


nuna_status_string = status_string


def nuna_shutdown() -> int:
    return lib().nuna_shutdown()


DEBUG_LAT_BINS, DEBUG_LAT_STEP = 64, 32


def debug_access_latency(src, dst, count, placement: int, launches: int = 1):
    """Histogram (numpy uint32[DEBUG_LAT_BINS], bins of DEBUG_LAT_STEP cycles) of first-load latencies of the
    8-rank bf16 one-shot under a placement: 0 round-robin, 1 co-located groups, 2 per-SM work lists."""
    import numpy as np
    hist = np.zeros(DEBUG_LAT_BINS, dtype=np.uint32)
    for _ in range(launches):
        st = lib().nuna_debug_access_latency(ptr_table(src), ptr_table(dst), count, placement,
                                             hist.ctypes.data_as(ctypes.POINTER(ctypes.c_uint)))
        if st != NUNA_OK:
            raise NunaError(st, "nuna_debug_access_latency")
    return hist


DEBUG_TRACE_BLOCKS = 1024


def debug_oneshot_regs_traced(src, dst, count, flags: int, slot: int, trace, stream=None) -> int:
    """One traced launch of the register-sharing one-shot (8 ranks, bf16): thread 0 of block b writes its start,
    wait-return and end times (global-timer ns) and its SM to ``trace`` (a device int64 tensor viewed as
    [slots][DEBUG_TRACE_BLOCKS][4]) at ``slot``.  Capturable.  Returns the grid size."""
    grid = ctypes.c_uint(0)
    st = lib().nuna_debug_oneshot_regs_traced(ptr_table(src), ptr_table(dst), count, flags, slot,
                                              ctypes.c_void_p(_addr(trace)), ctypes.byref(grid), _stream(stream))
    if st != NUNA_OK:
        raise NunaError(st, "nuna_debug_oneshot_regs_traced")
    return grid.value


def debug_twoshot(src, dst, count, dtype=NUNA_BF16, timeout_ms: int = 1000, unset_flags: bool = False) -> int:
    """Test hook: the flag-synchronised two-shot with an explicit timeout; with unset_flags its consumers
    wait for flags nobody publishes, so every (bounded) wait runs out."""
    return lib().nuna_debug_twoshot(ptr_table(src), ptr_table(dst), len(src), count, dtype, timeout_ms,
                                    1 if unset_flags else 0)


def debug_barrier_selftest(grid: int, expected: int, timeout_ms: int):
    passed = ctypes.c_uint(0)
    st = lib().nuna_debug_barrier_selftest(grid, expected, timeout_ms, ctypes.byref(passed))
    return st, passed.value
