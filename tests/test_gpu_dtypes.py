"""Parity of the binary16 and binary32 element types against the oracle (bf16 is covered in
test_gpu_parity.py).  Bit-exact, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_00867_b200 import binding as nb
from paper_2608_00867_b200 import workloads

pytestmark = pytest.mark.gpu

WORD = {"f16": (np.uint16, np.int16, torch.int16), "f32": (np.uint32, np.int32, torch.int32)}
COUNTS = [1, 3, 4, 5, 7, 8, 9, 17, 2047, 2049, 4096, 100003, 262144]


def upload(arrs, dtype):
    _, sview, _ = WORD[dtype]
    return [torch.from_numpy(a.view(sview).copy()).cuda() for a in arrs]


def fresh(n, count, dtype):
    return [torch.full((count,), 0x5A5A, dtype=WORD[dtype][2], device="cuda") for _ in range(n)]


def download(ts, dtype):
    torch.cuda.synchronize()
    return [t.cpu().numpy().view(WORD[dtype][0]) for t in ts]


def is_nan(a, dtype):
    if dtype == "f16":
        return ((a & 0x7C00) == 0x7C00) & ((a & 0x03FF) != 0)
    return ((a & 0x7F800000) == 0x7F800000) & ((a & 0x007FFFFF) != 0)


def assert_same_bits(got, want, dtype, what):
    nan = is_nan(want, dtype)
    assert np.array_equal(is_nan(got, dtype), nan), what + ": NaN positions differ"
    bad = np.nonzero((got != want) & ~nan)[0]
    assert bad.size == 0, f"{what}: {bad.size} mismatches, first {bad[:4]} got {got[bad[:4]]} want {want[bad[:4]]}"


ALGOS = {
    "oneshot": lambda s, d, c, dt: nb.nuna_allreduce_oneshot(s, d, c, dtype=dt),
    "oneshot_aware": lambda s, d, c, dt: nb.nuna_allreduce_oneshot(s, d, c, dtype=dt, flags=nb.NUNA_PLACE_AWARE),
    "oneshot_cluster": lambda s, d, c, dt: nb.nuna_allreduce_oneshot(s, d, c, dtype=dt,
                                                                    flags=nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_CLUSTER),
    "oneshot_staged": lambda s, d, c, dt: nb.nuna_allreduce_oneshot(s, d, c, dtype=dt,
                                                                   flags=nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_STAGED),
    "oneshot_regs": lambda s, d, c, dt: nb.nuna_allreduce_oneshot(s, d, c, dtype=dt,
                                                                 flags=nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_REGS | nb.NUNA_LAUNCH_PDL),
    "oneshot_sm_lists": lambda s, d, c, dt: nb.nuna_allreduce_oneshot(s, d, c, dtype=dt,
                                                                     flags=nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_SM_LISTS),
    "twoshot": lambda s, d, c, dt: nb.nuna_allreduce_twoshot(s, d, c, dtype=dt),
    "twoshot_pdl_sys": lambda s, d, c, dt: nb.nuna_allreduce_twoshot(s, d, c, dtype=dt,
                                                                    flags=nb.NUNA_LAUNCH_PDL | nb.NUNA_TWOSHOT_SYS_SCOPE),
    "twoshot_put": lambda s, d, c, dt: nb.nuna_allreduce_twoshot(s, d, c, dtype=dt, flags=nb.NUNA_TWOSHOT_PUT),
    "twoshot_static": lambda s, d, c, dt: nb.nuna_allreduce_twoshot_static(s, d, c, dtype=dt),
}


@pytest.mark.parametrize("dtype", ["f16", "f32"])
@pytest.mark.parametrize("n", [1, 2, 3, 8, 16])
@pytest.mark.parametrize("algo", sorted(ALGOS))
def test_allreduce_special_values(dtype, n, algo):
    dt = nb.DTYPE_BY_NAME[dtype]
    for count in COUNTS:
        src = workloads.special_values(n, count, seed=31 * n + count % 613, dtype=dtype)
        want = oracle.allreduce(src, nthreads=4, dtype=dtype)[0]
        dst = fresh(n, count, dtype)
        ALGOS[algo](upload(src, dtype), dst, count, dt)
        for d, got in enumerate(download(dst, dtype)):
            assert_same_bits(got, want, dtype, f"{algo} {dtype} n={n} count={count} dst={d}")
    assert nb.nuna_device_status() == nb.NUNA_OK


@pytest.mark.parametrize("dtype", ["f16", "f32"])
@pytest.mark.parametrize("n,shard", [(8, 4096), (8, 1000), (16, 33), (3, 4), (5, 2049), (2, 1), (8, 65536)])
def test_reduce_scatter_allgather_alltoall(dtype, n, shard):
    dt = nb.DTYPE_BY_NAME[dtype]
    src = workloads.special_values(n, n * shard, seed=n + shard, dtype=dtype)
    want_rs = oracle.reduce_scatter(src, nthreads=4, dtype=dtype)
    dsrc = upload(src, dtype)
    rs = fresh(n, shard, dtype)
    nb.nuna_reduce_scatter(dsrc, rs, shard, dtype=dt)
    got_rs = download(rs, dtype)
    for r in range(n):
        assert_same_bits(got_rs[r], want_rs[r], dtype, f"rs {dtype} n={n} shard={shard} r={r}")
    # bit copies: compare as 16-bit units with the oracle's copy routines
    as16 = lambda arrs: [np.ascontiguousarray(a).view(np.uint16) for a in arrs]
    ag = fresh(n, n * shard, dtype)
    nb.nuna_allgather(rs, ag, shard, dtype=dt)
    want_ag = oracle.allgather(as16(got_rs))
    for d, got in enumerate(download(ag, dtype)):
        assert np.array_equal(got.view(np.uint16), want_ag[d])
    a2a = fresh(n, n * shard, dtype)
    nb.nuna_alltoall(dsrc, a2a, shard, dtype=dt)
    k = 2 if dtype == "f32" else 1
    want_a2a = oracle.alltoall(as16(src))                     # blocks of shard*k 16-bit units: same transpose
    for d, got in enumerate(download(a2a, dtype)):
        assert np.array_equal(got.view(np.uint16), want_a2a[d]), (dtype, n, shard, d, k)


@pytest.mark.parametrize("dtype", ["f16", "f32"])
def test_benchmark_shaped_values_chain_and_host_entry(dtype):
    dt = nb.DTYPE_BY_NAME[dtype]
    n, count = 8, 32 * 8192
    src = workloads.rank_buffers_typed(n, count, "normal", seed=3, dtype=dtype)
    want = oracle.allreduce(src, nthreads=8, dtype=dtype)[0]
    dsrc = upload(src, dtype)
    for two_shot in (False, True):
        dst = fresh(n, count, dtype)
        chain = nb.nuna_chain_create([dsrc], [dst], 5, count, dtype=dt, two_shot=two_shot,
                                     flags=0 if two_shot else nb.NUNA_LAUNCH_PDL | nb.NUNA_PLACE_AUTO | nb.NUNA_HINT_RESIDENT)
        nb.nuna_chain_launch(chain)
        for got in download(dst, dtype):
            assert np.array_equal(got, want)
        nb.nuna_chain_destroy(chain)
        hdst = [np.zeros(count, dtype=WORD[dtype][0]) for _ in range(n)]
        nb.nuna_allreduce_host(src, hdst, count, dtype=dt, two_shot=two_shot)
        assert all(np.array_equal(h, want) for h in hdst)


def test_static_entry_limit_is_in_bytes():
    n = 2
    ok = nb.NUNA_STATIC_MAX_COUNT // 2                         # binary32 elements that fill the 4 MiB array
    src = [torch.zeros(ok + 4, dtype=torch.int32, device="cuda") for _ in range(n)]
    dst = [torch.zeros(ok + 4, dtype=torch.int32, device="cuda") for _ in range(n)]
    assert nb.nuna_allreduce_twoshot_static(src, dst, ok + 4, dtype=nb.NUNA_F32, check=False) == nb.NUNA_ERR_TOO_LARGE
    assert nb.nuna_allreduce_twoshot_static(src, dst, ok, dtype=nb.NUNA_F32, check=False) == nb.NUNA_OK
    torch.cuda.synchronize()
