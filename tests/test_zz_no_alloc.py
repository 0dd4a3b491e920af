"""The allocation-free two-shot allreduce.

Some users of this library cannot allocate device memory where they call it: a serving
process whose framework owns every byte of the GPU through its own pool, or a request loop
that must not pay for (or survive the failure of) a cudaMalloc.  For them the library has one
entry point whose scratch is a fixed array compiled into it.  This file checks that entry
point, through the C ABI, against the ordinary two-shot allreduce and against the CPU oracle:
same bits, twice in a row (the array keeps the first call's shard, which must not leak into the
second result), and a clear refusal beyond the array's size.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_00867_b200 import binding as nb
from paper_2608_00867_b200 import workloads

pytestmark = pytest.mark.gpu


def upload(arrs):
    return [torch.from_numpy(a.view(np.int16).copy()).cuda() for a in arrs]


def run_both(src, count):
    n = len(src)
    dsrc = upload(src)
    ref = [torch.zeros(count, dtype=torch.int16, device="cuda") for _ in range(n)]
    got = [torch.full((count,), 0x5A5A, dtype=torch.int16, device="cuda") for _ in range(n)]
    nb.nuna_allreduce_twoshot(dsrc, ref, count)                 # the existing entry point
    nb.nuna_allreduce_twoshot_static(dsrc, got, count)          # the one that allocates nothing
    torch.cuda.synchronize()
    return ref, got


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    # first call: the benchmark's decode activation; second: a shorter, ragged message with awkward
    # values, so anything left in the shared array by the first call would show up as wrong bits
    w = workloads.config_decode_activation()
    first = workloads.make(w)
    second = workloads.special_values(5, 100003, seed=2)
    for src, count in ((first, w.count), (second, 100003)):
        ref, got = run_both(src, count)
        want = oracle.allreduce(src, nthreads=4)[0]
        nan = ((want & 0x7F80) == 0x7F80) & ((want & 0x007F) != 0)
        for r, g in zip(ref, got):
            assert torch.equal(r, g)                            # bit for bit, every destination
            h = g.cpu().numpy().view(np.uint16)
            assert np.array_equal(h[~nan], want[~nan])          # and the same bits as the CPU oracle
            assert (((h[nan] & 0x7F80) == 0x7F80) & ((h[nan] & 0x007F) != 0)).all()
    # and once more with the first message: the array now holds the second call's shard
    ref, got = run_both(first, w.count)
    assert all(torch.equal(r, g) for r, g in zip(ref, got))


def test_device_memory_in_use_does_not_change():
    """The entry point exists for callers that must not allocate: after the first call on the device, further
    calls of any size leave the amount of free device memory exactly where it was."""
    n = 4
    bufs = {c: ([torch.zeros(c, dtype=torch.int16, device="cuda") for _ in range(n)],
                [torch.zeros(c, dtype=torch.int16, device="cuda") for _ in range(n)]) for c in (8, 4099, 1 << 20)}
    nb.nuna_allreduce_twoshot_static(*bufs[8], 8)                # first call on the device: set-up, no allocation either
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for _ in range(3):
        for c, (src, dst) in bufs.items():
            nb.nuna_allreduce_twoshot_static(src, dst, c)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before


def test_sizes_beyond_the_fixed_array_are_refused():
    n = 2
    count = nb.NUNA_STATIC_MAX_COUNT + 8
    src = [torch.zeros(count, dtype=torch.int16, device="cuda") for _ in range(n)]
    dst = [torch.full((count,), 7, dtype=torch.int16, device="cuda") for _ in range(n)]
    before = nb.nuna_launch_count()
    assert nb.nuna_allreduce_twoshot_static(src, dst, count, check=False) == nb.NUNA_ERR_TOO_LARGE
    assert nb.nuna_launch_count() == before                     # nothing was launched
    torch.cuda.synchronize()
    assert all(int(d.min()) == 7 and int(d.max()) == 7 for d in dst)
    # the largest allowed size works
    count = nb.NUNA_STATIC_MAX_COUNT
    src = workloads.rank_buffers(n, count, "normal", seed=8)
    ref, got = run_both(src, count)
    assert all(torch.equal(r, g) for r, g in zip(ref, got))
    assert np.array_equal(got[0].cpu().numpy().view(np.uint16), oracle.allreduce(src, nthreads=4)[0])
    assert nb.nuna_device_status() == nb.NUNA_OK                # also reads the fixed arrays' own status word


@pytest.mark.parametrize("dtype", ["f16", "f32"])
def test_other_element_types_and_the_limit_in_bytes(dtype):
    """The limit is the array's size in bytes: 2 Mi 16-bit elements, 1 Mi binary32 elements."""
    n = 3
    code = nb.DTYPE_BY_NAME[dtype]
    tdt = torch.int32 if dtype == "f32" else torch.int16
    limit = nb.NUNA_STATIC_MAX_COUNT * 2 // nb.ELEM_SIZE[code]
    src = workloads.rank_buffers_typed(n, limit, "normal", 17, dtype)
    want = oracle.allreduce(src, nthreads=4, dtype=dtype)[0]
    dsrc = [torch.from_numpy(a.view(np.int32 if dtype == "f32" else np.int16).copy()).cuda() for a in src]
    for _ in range(2):                                          # two calls in a row on the shared array
        dst = [torch.zeros(limit, dtype=tdt, device="cuda") for _ in range(n)]
        nb.nuna_allreduce_twoshot_static(dsrc, dst, limit, dtype=code)
        torch.cuda.synchronize()
        for d in dst:
            assert np.array_equal(d.cpu().numpy().view(want.dtype), want)
    over = limit + 16 // nb.ELEM_SIZE[code]
    big = [torch.zeros(over, dtype=tdt, device="cuda") for _ in range(2 * n)]
    assert nb.nuna_allreduce_twoshot_static(big[:n], big[n:], over, dtype=code, check=False) == nb.NUNA_ERR_TOO_LARGE
