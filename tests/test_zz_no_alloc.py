"""The allocation-free two-shot allreduce.

Some users of this library cannot allocate device memory where they call it: a serving
process whose framework owns every byte of the GPU through its own pool, or a request loop
that must not pay for (or survive the failure of) a cudaMalloc.  For them the library has one
entry point whose scratch is a fixed array compiled into it.  This file checks that entry
point, through the C ABI, against the ordinary two-shot allreduce: same bits, twice in a row
(the array keeps the first call's shard, which must not leak into the second result), and a
clear refusal beyond the array's size.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

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
        for r, g in zip(ref, got):
            assert torch.equal(r, g)                            # bit for bit, every destination
    # and once more with the first message: the array now holds the second call's shard
    ref, got = run_both(first, w.count)
    assert all(torch.equal(r, g) for r, g in zip(ref, got))


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
