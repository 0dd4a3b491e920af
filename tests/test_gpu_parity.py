"""Parity of the CUDA library against the CPU oracle, through the C ABI.  Bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_00867_b200 import binding as nb
from paper_2608_00867_b200 import workloads

pytestmark = pytest.mark.gpu

GUARD = 64          # sentinel elements on each side of every destination
SENTINEL = 0x5A5A
POISON = 0xDEAD


def upload(arrs):
    return [torch.from_numpy(a.view(np.int16).copy()).cuda() for a in arrs]


class Dst:
    """Destination buffers with guard zones; the payload starts 16-byte aligned."""

    def __init__(self, n, count):
        self.count = count
        self.full = []
        self.view = []
        for _ in range(n):
            t = torch.full((count + 2 * GUARD,), SENTINEL, dtype=torch.int16, device="cuda")
            t[GUARD:GUARD + count] = np.int16(np.uint16(POISON).view(np.int16))
            self.full.append(t)
            self.view.append(t[GUARD:GUARD + count])

    def numpy(self):
        torch.cuda.synchronize()
        out = []
        for t in self.full:
            h = t.cpu().numpy().view(np.uint16)
            assert (h[:GUARD] == SENTINEL).all() and (h[GUARD + self.count:] == SENTINEL).all(), "guard zone overwritten"
            out.append(h[GUARD:GUARD + self.count].copy())
        return out


def is_nan(a):
    return ((a & 0x7F80) == 0x7F80) & ((a & 0x007F) != 0)


def assert_same_bits(got, want, what=""):
    """Equal bit patterns; where the oracle has a NaN the GPU must have a NaN (payload unpinned)."""
    assert got.shape == want.shape, what
    nan = is_nan(want)
    assert np.array_equal(is_nan(got), nan), what + ": NaN positions differ"
    bad = np.nonzero((got != want) & ~nan)[0]
    assert bad.size == 0, f"{what}: {bad.size} mismatches, first at {bad[:5]}: got {got[bad[:5]]} want {want[bad[:5]]}"


COUNTS = [1, 7, 8, 9, 15, 16, 17, 2047, 2048, 2049, 4096, 6151, 100003, 262144]


@pytest.mark.parametrize("n", [1, 2, 3, 5, 8, 16])
@pytest.mark.parametrize("algo", ["oneshot", "oneshot_aware", "oneshot_staged", "oneshot_regs", "oneshot_sm_lists", "twoshot",
                                  "twoshot_pdl", "twoshot_sys", "twoshot_put"])
def test_allreduce_special_values_all_counts(n, algo):
    for count in COUNTS:
        src = workloads.special_values(n, count, seed=1000 * n + count % 997)
        want = oracle.allreduce(src, nthreads=4)
        dsrc, dst = upload(src), Dst(n, count)
        if algo == "oneshot":
            nb.nuna_allreduce_oneshot(dsrc, dst.view, count)
        elif algo == "oneshot_aware":
            nb.nuna_allreduce_oneshot(dsrc, dst.view, count, flags=nb.NUNA_PLACE_AWARE)
        elif algo == "oneshot_staged":
            nb.nuna_allreduce_oneshot(dsrc, dst.view, count, flags=nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_STAGED)
        elif algo == "oneshot_regs":
            nb.nuna_allreduce_oneshot(dsrc, dst.view, count, flags=nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_REGS)
        elif algo == "oneshot_sm_lists":
            nb.nuna_allreduce_oneshot(dsrc, dst.view, count, flags=nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_SM_LISTS)
        else:
            f = {"twoshot": 0, "twoshot_pdl": nb.NUNA_LAUNCH_PDL, "twoshot_put": nb.NUNA_TWOSHOT_PUT,
                 "twoshot_sys": nb.NUNA_TWOSHOT_SYS_SCOPE | nb.NUNA_LAUNCH_PDL}[algo]
            nb.nuna_allreduce_twoshot(dsrc, dst.view, count, flags=f)
        got = dst.numpy()
        for d in range(n):
            assert_same_bits(got[d], want[d], f"{algo} n={n} count={count} dst={d}")
    assert nb.nuna_device_status() == nb.NUNA_OK


def test_experimental_cluster_placement_one_case():
    """NUNA_PLACE_CLUSTER is an experiment that the automatic choice never takes: one parity case."""
    n = 8
    for count in (9, 2049, 100003):
        src = workloads.special_values(n, count, seed=3 + count)
        want = oracle.allreduce(src, nthreads=4)
        dst = Dst(n, count)
        nb.nuna_allreduce_oneshot(upload(src), dst.view, count, flags=nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_CLUSTER)
        for d, got in enumerate(dst.numpy()):
            assert_same_bits(got, want[d], f"cluster count={count} dst={d}")


@pytest.mark.parametrize("vecs", [32, 64, 128, 256])
def test_staged_oneshot_tile_sizes(vecs):
    """The shared-memory staged kernel at every tile size the option allows, sizes around the tile edges."""
    n = 8
    try:
        nb.nuna_set_option(nb.NUNA_OPT_STAGE_VECS, vecs)
        for count in (8 * vecs - 8, 8 * vecs, 8 * vecs + 8, 8 * vecs * 3 + 5, 32 * 8192):
            src = workloads.special_values(n, count, seed=vecs + count % 101)
            want = oracle.allreduce(src, nthreads=4)[0]
            for flags in (nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_STAGED,
                          nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_STAGED | nb.NUNA_LAUNCH_PDL | nb.NUNA_HINT_RESIDENT):
                dst = Dst(n, count)
                nb.nuna_allreduce_oneshot(upload(src), dst.view, count, flags=flags)
                for got in dst.numpy():
                    assert_same_bits(got, want, f"staged vecs={vecs} count={count}")
    finally:
        nb.nuna_set_option(nb.NUNA_OPT_STAGE_VECS, 0)
    assert nb.nuna_device_status() == nb.NUNA_OK


@pytest.mark.parametrize("vecs", [0, 8, 56, 104, 256])
@pytest.mark.parametrize("n", [3, 8, 16])
def test_register_oneshot_tile_sizes_and_prefetch(vecs, n):
    """The register-sharing kernel at tile sizes from one line to a full block (0 = chosen by size), counts around
    the tile edges and with a ragged tail, launched plainly, behind a dependent launch with the L2 prefetch ahead of
    the wait, with the prefetch switched off, and with the resident hint (which also suppresses it): the prefetch
    and the tile size change no bit."""
    tv = vecs if vecs else 56
    base = nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_REGS
    try:
        nb.nuna_set_option(nb.NUNA_OPT_REGS_VECS, vecs)
        for count in (8 * tv - 8, 8 * tv, 8 * tv + 8, 8 * tv * 5 + 3, 24 * 8192 + 1):
            src = workloads.special_values(n, count, seed=7 * n + vecs + count % 101)
            want = oracle.allreduce(src, nthreads=4)[0]
            dsrc = upload(src)
            for flags, no_prefetch in ((base, 0), (base | nb.NUNA_LAUNCH_PDL, 0), (base | nb.NUNA_LAUNCH_PDL, 1),
                                       (base | nb.NUNA_LAUNCH_PDL | nb.NUNA_HINT_RESIDENT, 0)):
                nb.nuna_set_option(nb.NUNA_OPT_PREFETCH, no_prefetch)
                dst = Dst(n, count)
                # two calls back to back: the second one's prefetch runs while the first is still writing
                nb.nuna_allreduce_oneshot(dsrc, dst.view, count, flags=flags)
                nb.nuna_allreduce_oneshot(dsrc, dst.view, count, flags=flags)
                for got in dst.numpy():
                    assert_same_bits(got, want, f"regs vecs={vecs} n={n} count={count} flags={flags} nopf={no_prefetch}")
            if vecs == 0:                                            # a capped grid: blocks loop over several tiles
                for blocks in (1, 5, 37):
                    nb.nuna_set_option(nb.NUNA_OPT_BLOCKS, blocks)
                    dst = Dst(n, count)
                    nb.nuna_allreduce_oneshot(dsrc, dst.view, count, flags=base | nb.NUNA_LAUNCH_PDL)
                    for got in dst.numpy():
                        assert_same_bits(got, want, f"regs blocks={blocks} n={n} count={count}")
                nb.nuna_set_option(nb.NUNA_OPT_BLOCKS, 0)
    finally:
        nb.nuna_set_option(nb.NUNA_OPT_REGS_VECS, 0)
        nb.nuna_set_option(nb.NUNA_OPT_PREFETCH, 0)
        nb.nuna_set_option(nb.NUNA_OPT_BLOCKS, 0)
    assert nb.nuna_device_status() == nb.NUNA_OK


@pytest.mark.parametrize("algo", ["oneshot_regs", "twoshot_put", "twoshot_flags"])
def test_prefetch_ahead_of_the_wait_sees_the_predecessors_writes(algo):
    """A chain x -> allreduce -> allreduce -> ... in which every call's sources are the previous call's destinations,
    launched back to back with dependent launches: each kernel's prefetch is issued while its predecessor is still
    writing the very lines it asks for.  The values grow by a factor of N per node, so a stale line shows."""
    n, count, nodes = 8, 64 * 1024, 5
    src = [np.full(count, 0x3F80, dtype=np.uint16) for _ in range(n)]          # bf16 1.0
    a, b = Dst(n, count), Dst(n, count)
    call, flags = {"oneshot_regs": (nb.nuna_allreduce_oneshot, nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_REGS),
                   "twoshot_put": (nb.nuna_allreduce_twoshot, nb.NUNA_TWOSHOT_PUT),
                   "twoshot_flags": (nb.nuna_allreduce_twoshot, 0)}[algo]
    flags |= nb.NUNA_LAUNCH_PDL
    for _ in range(20):
        cur = upload(src)
        for k in range(nodes):
            out = a if k % 2 == 0 else b
            call(cur, out.view, count, flags=flags)
            cur = out.view
        got = out.numpy()
        want = np.float32(n) ** nodes                                           # 8^5 = 32768, exact in bf16
        for g in got:
            vals = (g.astype(np.uint32) << 16).view(np.float32)
            assert (vals == want).all()
    assert nb.nuna_device_status() == nb.NUNA_OK


def test_config_small_two_ranks():
    w = workloads.config_small_oneshot()
    src = workloads.make(w)
    want = oracle.allreduce(src)
    dst = Dst(w.nranks, w.count)
    nb.nuna_allreduce_oneshot(upload(src), dst.view, w.count)
    got = dst.numpy()
    for d in range(w.nranks):
        assert np.array_equal(got[d], want[d])


@pytest.mark.parametrize("flags", [nb.NUNA_PLACE_ROUNDROBIN, nb.NUNA_PLACE_AWARE, nb.NUNA_PLACE_AUTO,
                                   nb.NUNA_PLACE_AUTO | nb.NUNA_HINT_RESIDENT, nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_STAGED,
                                   nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_REGS | nb.NUNA_LAUNCH_PDL])
def test_config_decode_activation_all_placements(flags):
    w = workloads.config_decode_activation()
    src = workloads.make(w)
    want = oracle.allreduce(src, nthreads=4)
    dsrc = upload(src)
    for call in (nb.nuna_allreduce_oneshot, nb.nuna_allreduce_twoshot):
        dst = Dst(w.nranks, w.count)
        call(dsrc, dst.view, w.count, flags=flags)
        got = dst.numpy()
        for d in range(w.nranks):
            assert np.array_equal(got[d], want[d])


@pytest.mark.parametrize("n,shard", [(8, 4096), (8, 1000), (16, 33), (3, 8), (5, 2049), (8, 65536), (2, 1)])
@pytest.mark.parametrize("pdl", [0, nb.NUNA_LAUNCH_PDL])
def test_reduce_scatter_and_allgather(n, shard, pdl):
    src = workloads.special_values(n, n * shard, seed=n * 31 + shard)
    want_rs = oracle.reduce_scatter(src, nthreads=4)
    dsrc = upload(src)
    rs = Dst(n, shard)
    nb.nuna_reduce_scatter(dsrc, rs.view, shard, flags=pdl)
    got_rs = rs.numpy()
    for r in range(n):
        assert_same_bits(got_rs[r], want_rs[r], f"rs n={n} shard={shard} r={r}")
    # allgather of the GPU's own shards: raw bit copy, NaN payloads included
    want_ag = oracle.allgather(got_rs)
    ag = Dst(n, n * shard)
    nb.nuna_allgather(rs.view, ag.view, shard, flags=pdl)
    got_ag = ag.numpy()
    for d in range(n):
        assert np.array_equal(got_ag[d], want_ag[d])
    # allreduce == allgather(reduce_scatter) byte for byte (NaN payload aside)
    ar = Dst(n, n * shard)
    nb.nuna_allreduce_oneshot(dsrc, ar.view, n * shard)
    got_ar = ar.numpy()
    for d in range(n):
        assert_same_bits(got_ag[d], got_ar[d], "ar vs ag(rs)")


@pytest.mark.parametrize("bulk_vecs", [0, 1, 8, 2048])
def test_allgather_and_alltoall_copy_forms(bulk_vecs):
    """Bulk-copy form (default and extreme tile sizes) and register form of the two pure copies: raw bits,
    ragged shard lengths, 16-byte-only alignment of the shards inside the destinations."""
    rng = np.random.Generator(np.random.PCG64(17 + bulk_vecs))
    try:
        nb.nuna_set_option(nb.NUNA_OPT_AG_BULK_VECS, bulk_vecs)
        for n, shard in ((16, 32768), (8, 8), (5, 2056), (3, 100000), (16, 24), (2, 300008)):
            src = [rng.integers(0, 1 << 16, size=shard, dtype=np.uint32).astype(np.uint16) for _ in range(n)]
            dst = Dst(n, n * shard)
            nb.nuna_allgather(upload(src), dst.view, shard, flags=nb.NUNA_LAUNCH_PDL)
            want = oracle.allgather(src)
            for d, got in enumerate(dst.numpy()):
                assert np.array_equal(got, want[d]), ("allgather", n, shard, d)
            asrc = [rng.integers(0, 1 << 16, size=n * shard, dtype=np.uint32).astype(np.uint16) for _ in range(n)]
            adst = Dst(n, n * shard)
            nb.nuna_alltoall(upload(asrc), adst.view, shard)
            awant = oracle.alltoall(asrc, nthreads=4)
            for d, got in enumerate(adst.numpy()):
                assert np.array_equal(got, awant[d]), ("alltoall", n, shard, d)
    finally:
        nb.nuna_set_option(nb.NUNA_OPT_AG_BULK_VECS, 0)
    assert nb.nuna_device_status() == nb.NUNA_OK


def test_allgather_large_output_takes_the_bulk_copy_form_by_default():
    """Beyond 128 MiB of output the default allgather is the bulk-copy form with its size-chosen tile: 8 ranks x 5 MiB
    + 16 bytes (a ragged last tile), raw bits, every destination compared in full on the device."""
    n, shard = 8, 5 * 512 * 1024 + 8
    g = torch.Generator(device="cuda")
    g.manual_seed(99)
    src = [torch.randint(-32768, 32767, (shard,), generator=g, device="cuda", dtype=torch.int16) for _ in range(n)]
    dst = [torch.full((n * shard,), -1, dtype=torch.int16, device="cuda") for _ in range(n)]
    nb.nuna_allgather(src, dst, shard, flags=nb.NUNA_LAUNCH_PDL)
    torch.cuda.synchronize()
    want = oracle.allgather([x.cpu().numpy().view(np.uint16) for x in src])[0]
    assert np.array_equal(dst[0].cpu().numpy().view(np.uint16), want)
    for d in dst[1:]:
        assert torch.equal(d, dst[0])                                # all destinations identical
    assert nb.nuna_device_status() == nb.NUNA_OK


def test_config_allgather16_raw_bits():
    w = workloads.config_allgather16()
    rng = np.random.Generator(np.random.PCG64(w.seed))
    for src in (workloads.make(w),
                [rng.integers(0, 1 << 16, size=w.count, dtype=np.uint32).astype(np.uint16) for _ in range(w.nranks)]):
        want = oracle.allgather(src)
        dst = Dst(w.nranks, w.nranks * w.count)
        nb.nuna_allgather(upload(src), dst.view, w.count)
        got = dst.numpy()
        for d in range(w.nranks):
            assert np.array_equal(got[d], want[d])


@pytest.mark.parametrize("n,block", [(8, 4096), (8, 1000), (16, 33), (3, 8), (5, 2049), (8, 65536), (2, 1), (1, 77), (16, 8192)])
def test_alltoall_raw_bits(n, block):
    rng = np.random.Generator(np.random.PCG64(n * 1000 + block))
    src = [rng.integers(0, 1 << 16, size=n * block, dtype=np.uint32).astype(np.uint16) for _ in range(n)]
    want = oracle.alltoall(src, nthreads=4)
    dst = Dst(n, n * block)
    nb.nuna_alltoall(upload(src), dst.view, block, flags=nb.NUNA_LAUNCH_PDL if block % 2 else 0)
    got = dst.numpy()
    for d in range(n):
        assert np.array_equal(got[d], want[d]), (n, block, d)
    # twice = identity
    back = Dst(n, n * block)
    nb.nuna_alltoall(dst.view, back.view, block, flags=nb.NUNA_LAUNCH_PDL)
    for r, g in enumerate(back.numpy()):
        assert np.array_equal(g, src[r])


def test_sweep_sizes_one_and_two_shot_agree_with_oracle():
    for w in workloads.config_size_sweep(13, 22):
        src = workloads.make(w)
        want = oracle.allreduce(src, nthreads=8)[0]
        dsrc = upload(src)
        for call, flags in ((nb.nuna_allreduce_oneshot, 0), (nb.nuna_allreduce_oneshot, nb.NUNA_PLACE_AWARE),
                            (nb.nuna_allreduce_oneshot, nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_STAGED | nb.NUNA_LAUNCH_PDL),
                            (nb.nuna_allreduce_oneshot, nb.NUNA_PLACE_AUTO | nb.NUNA_LAUNCH_PDL),
                            (nb.nuna_allreduce_twoshot, 0), (nb.nuna_allreduce_twoshot, nb.NUNA_LAUNCH_PDL),
                            (nb.nuna_allreduce_twoshot, nb.NUNA_TWOSHOT_PUT)):
            dst = Dst(w.nranks, w.count)
            call(dsrc, dst.view, w.count, flags=flags)
            got = dst.numpy()
            for d in range(w.nranks):
                assert np.array_equal(got[d], want), (w.name, call.__name__, flags, d)


def test_full_size_64MiB_every_column_and_invariants():
    """The largest benchmarked message (8 ranks x 64 MiB), in the launch configuration the benchmark times.
    The oracle folds all 32 Mi columns (all host threads); every variant must reproduce every bit."""
    import os
    w = workloads.config_size_sweep(26, 26)[0]
    n, count = w.nranks, w.count
    gen = torch.Generator(device="cuda")
    gen.manual_seed(w.seed)
    dsrc = [torch.randn(count, generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16).view(torch.int16)
            for _ in range(n)]
    # one "awkward" column block: wide exponent spread so the fold order is observable
    sp = workloads.special_values(n, 4096, seed=5)
    for r in range(n):
        dsrc[r][count - 4096:] = torch.from_numpy(sp[r].view(np.int16)).cuda()
    host = [t.cpu().numpy().view(np.uint16) for t in dsrc]
    want = oracle.allreduce(host, nthreads=os.cpu_count() or 4)[0]
    del host
    dwant = torch.from_numpy(want.view(np.int16)).cuda()
    nan = torch.from_numpy(is_nan(want)).cuda()
    P = nb.NUNA_LAUNCH_PDL
    for call, flags in ((nb.nuna_allreduce_oneshot, 0), (nb.nuna_allreduce_oneshot, nb.NUNA_PLACE_AWARE),
                        (nb.nuna_allreduce_oneshot, nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_STAGED | P),
                        (nb.nuna_allreduce_oneshot, nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_REGS | P),
                        (nb.nuna_allreduce_oneshot, nb.NUNA_PLACE_AUTO | P),
                        (nb.nuna_allreduce_twoshot, 0), (nb.nuna_allreduce_twoshot, P),
                        (nb.nuna_allreduce_twoshot, nb.NUNA_TWOSHOT_PUT | P), (nb.nuna_allreduce, 0)):
        dst = [torch.full((count,), -1, dtype=torch.int16, device="cuda") for _ in range(n)]
        call(dsrc, dst, count, flags=flags)
        torch.cuda.synchronize()
        same = (dst[0] == dwant) | nan
        assert bool(same.all()), f"{call.__name__} flags={flags}: {int((~same).sum())} columns differ from the oracle"
        got_nan = dst[0][nan].cpu().numpy().view(np.uint16)
        assert is_nan(got_nan).all()
        for d in range(1, n):
            assert torch.equal(dst[0], dst[d])                        # all destinations identical
        del dst
    assert nb.nuna_device_status() == nb.NUNA_OK


def test_graph_replay_gives_same_bits():
    w = workloads.config_decode_activation()
    src = workloads.make(w)
    want = oracle.allreduce(src, nthreads=4)[0]
    dsrc = upload(src)
    dst = [torch.zeros(w.count, dtype=torch.int16, device="cuda") for _ in range(w.nranks)]
    nb.nuna_init(2 * w.count)
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            nb.nuna_allreduce_oneshot(dsrc, dst, w.count, stream=s)
            nb.nuna_allreduce_twoshot(dsrc, dst, w.count, stream=s)
    for _ in range(3):
        for t in dst:
            t.zero_()
        g.replay()
        torch.cuda.synchronize()
        for t in dst:
            assert np.array_equal(t.cpu().numpy().view(np.uint16), want)


def test_traced_launch_matches_oracle_and_orders_its_timestamps():
    """The measurement aid that timestamps every block of the register-sharing one-shot: the destinations still
    receive the oracle's bits, every block reports start <= wait-return <= end on an SM that exists, and a launch
    behind a predecessor never returns from its wait before that predecessor's last block has issued its stores."""
    w = workloads.config_decode_activation()
    src = workloads.make(w)
    want = oracle.allreduce(src, nthreads=4)[0]
    dsrc = upload(src)
    nodes, TB = 6, nb.DEBUG_TRACE_BLOCKS
    for flags in (0, nb.NUNA_LAUNCH_PDL, nb.NUNA_LAUNCH_PDL | nb.NUNA_HINT_RESIDENT):
        dst = [torch.zeros(w.count, dtype=torch.int16, device="cuda") for _ in range(w.nranks)]
        trace = torch.zeros(nodes * TB * 4, dtype=torch.int64, device="cuda")
        grid = 0
        for i in range(nodes):
            grid = nb.debug_oneshot_regs_traced(dsrc, dst, w.count, flags, i, trace)
        torch.cuda.synchronize()
        for t in dst:
            assert np.array_equal(t.cpu().numpy().view(np.uint16), want)
        assert 0 < grid <= TB
        t = trace.cpu().numpy().reshape(nodes, TB, 4)[:, :grid]
        assert (t[:, :, 0] > 0).all() and (t[:, :, 0] <= t[:, :, 1]).all() and (t[:, :, 1] <= t[:, :, 2]).all()
        assert (t[:, :, 3] >= 0).all() and (t[:, :, 3] < torch.cuda.get_device_properties(0).multi_processor_count).all()
        for i in range(1, nodes):                                   # 32 ns = the timer's resolution
            assert t[i, :, 1].min() + 32 >= t[i - 1, :, 2].max(), f"flags={flags}: node {i} passed its wait early"
        assert (t[:, grid:, :] == 0).all() if grid < TB else True
    assert nb.nuna_device_status() == nb.NUNA_OK


def test_headline_launch_configuration_matches_oracle():
    """The configuration the benchmark times: 8 x 512 KiB, placement AUTO with dependent launches, as nodes of one
    CUDA graph rotating over buffer sets (distinct data in each), replayed.  Every destination of every set is
    compared with the oracle after each replay, so a prefetch or a dependent launch that ran ahead of its data would show."""
    w = workloads.config_decode_activation()
    nsets, passes = 6, 3
    srcs = [workloads.rank_buffers(w.nranks, w.count, "normal", seed=500 + k) for k in range(nsets)]
    want = [oracle.allreduce(x, nthreads=4)[0] for x in srcs]
    dsrc = [upload(x) for x in srcs]
    ddst = [[torch.zeros(w.count, dtype=torch.int16, device="cuda") for _ in range(w.nranks)] for _ in range(nsets)]
    flags = nb.NUNA_PLACE_AUTO | nb.NUNA_LAUNCH_PDL
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        nb.nuna_allreduce_oneshot(dsrc[0], ddst[0], w.count, flags=flags, stream=s)
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=s):
            for _ in range(passes):
                for k in range(nsets):
                    nb.nuna_allreduce_oneshot(dsrc[k], ddst[k], w.count, flags=flags, stream=s)
    for _ in range(3):
        for dset in ddst:
            for t in dset:
                t.zero_()
        torch.cuda.synchronize()
        with torch.cuda.stream(s):
            g.replay()
        torch.cuda.synchronize()
        for k in range(nsets):
            for t in ddst[k]:
                assert np.array_equal(t.cpu().numpy().view(np.uint16), want[k]), f"set {k}"
    assert nb.nuna_device_status() == nb.NUNA_OK


@pytest.mark.parametrize("flags", [0, nb.NUNA_LAUNCH_PDL, nb.NUNA_LAUNCH_PDL | nb.NUNA_PLACE_AUTO | nb.NUNA_HINT_RESIDENT,
                                   nb.NUNA_CHAIN_GRAPH, nb.NUNA_CHAIN_PERSISTENT])
@pytest.mark.parametrize("two_shot", [False, True])
def test_chain_every_node_matches_oracle(flags, two_shot):
    if two_shot and (flags & nb.NUNA_CHAIN_PERSISTENT):
        pytest.skip("the single-kernel chain runs one-shot nodes only")
    tokens = 8
    w = workloads.config_decode_chain(tokens)
    nsets, nnodes = 2, 6
    srcs = [workloads.rank_buffers(w.nranks, w.count, "normal", seed=w.seed + s) for s in range(nsets)]
    want = [oracle.allreduce(s, nthreads=4)[0] for s in srcs]
    dsrc = [upload(s) for s in srcs]
    ddst = [[torch.zeros(w.count, dtype=torch.int16, device="cuda") for _ in range(w.nranks)] for _ in range(nsets)]
    chain = nb.nuna_chain_create(dsrc, ddst, nnodes, w.count, flags=flags, two_shot=two_shot)
    try:
        for _ in range(3):
            for dset in ddst:
                for t in dset:
                    t.zero_()
            nb.nuna_chain_launch(chain)
            torch.cuda.synchronize()
            for s in range(nsets):
                for t in ddst[s]:
                    assert np.array_equal(t.cpu().numpy().view(np.uint16), want[s])
    finally:
        nb.nuna_chain_destroy(chain)
    assert nb.nuna_device_status() == nb.NUNA_OK


@pytest.mark.parametrize("mode", [0, nb.NUNA_CHAIN_GRAPH, nb.NUNA_CHAIN_PERSISTENT])
@pytest.mark.parametrize("tokens", [1, 8, 64, 256])
def test_decode_chain_160_nodes_as_benchmarked(tokens, mode):
    """The benchmark's chain: 160 nodes over two alternating buffer sets, AUTO placement under the
    resident hint, dependent launch; as a graph, as one kernel, and as the library picks.  Both sets'
    destinations are checked (each set is written 80 times)."""
    w = workloads.config_decode_chain(tokens)
    flags = nb.NUNA_PLACE_AUTO | nb.NUNA_HINT_RESIDENT | nb.NUNA_LAUNCH_PDL | mode
    srcs = [workloads.rank_buffers(w.nranks, w.count, "normal", seed=w.seed + s) for s in range(2)]
    want = [oracle.allreduce(s, nthreads=8)[0] for s in srcs]
    dsrc = [upload(s) for s in srcs]
    ddst = [[torch.zeros(w.count, dtype=torch.int16, device="cuda") for _ in range(w.nranks)] for _ in range(2)]
    chain = nb.nuna_chain_create(dsrc, ddst, workloads.CHAIN_NODES, w.count, flags=flags)
    try:
        for _ in range(2):
            nb.nuna_chain_launch(chain)
        torch.cuda.synchronize()
        for s in range(2):
            for t in ddst[s]:
                assert np.array_equal(t.cpu().numpy().view(np.uint16), want[s])
    finally:
        nb.nuna_chain_destroy(chain)


def test_persistent_chain_ragged_counts_ranks_and_dtypes():
    """The single-kernel chain on awkward shapes: tails, non-power-of-two rank counts, three buffer sets."""
    for n, count in ((8, 8192), (8, 5), (3, 100003), (16, 4099), (5, 2048), (1, 777), (2, 65536 + 3)):
        nsets, nnodes = 3, 7
        srcs = [workloads.special_values(n, count, seed=n * 7 + count % 13 + s) for s in range(nsets)]
        want = [oracle.allreduce(s, nthreads=4)[0] for s in srcs]
        dsrc = [upload(s) for s in srcs]
        dsts = [Dst(n, count) for _ in range(nsets)]
        chain = nb.nuna_chain_create(dsrc, [d.view for d in dsts], nnodes, count, flags=nb.NUNA_CHAIN_PERSISTENT)
        try:
            nb.nuna_chain_launch(chain)
            nb.nuna_chain_launch(chain)
            for s in range(nsets):
                for got in dsts[s].numpy():
                    assert_same_bits(got, want[s], f"persistent chain n={n} count={count} set={s}")
        finally:
            nb.nuna_chain_destroy(chain)
    # refused where it cannot run: two-shot nodes, too many sets
    a = [[torch.zeros(64, dtype=torch.int16, device="cuda") for _ in range(2)] for _ in range(18)]
    assert nb.nuna_chain_create(a[:9], a[9:], 4, 64, flags=nb.NUNA_CHAIN_PERSISTENT, check=False) == nb.NUNA_ERR_INVALID_ARG
    assert nb.nuna_chain_create(a[:2], a[2:4], 4, 64, flags=nb.NUNA_CHAIN_PERSISTENT, two_shot=True,
                                check=False) == nb.NUNA_ERR_INVALID_ARG
    assert nb.nuna_chain_create(a[:2], a[2:4], 4, 64, flags=nb.NUNA_CHAIN_PERSISTENT | nb.NUNA_CHAIN_GRAPH,
                                check=False) == nb.NUNA_ERR_INVALID_ARG


def test_scratch_growth_after_capture_keeps_captured_graphs_valid():
    """A chain of flag-synchronised two-shots captures the scratch address.  A later, larger two-shot call
    grows the scratch; the old allocation must stay alive so that replaying the chain is still correct."""
    n, small, big = 8, 8 * 8192, 9 * (1 << 20)
    nb.nuna_init(2 * small)
    src = workloads.special_values(n, small, seed=321)
    want = oracle.allreduce(src, nthreads=4)[0]
    dsrc = upload(src)
    dst = Dst(n, small)
    chain = nb.nuna_chain_create([dsrc], [dst.view], 4, small, two_shot=True)
    try:
        nb.nuna_chain_launch(chain)
        for got in dst.numpy():
            assert_same_bits(got, want, "before growth")
        # the largest scratch any earlier test may have asked for is 128 MiB: go beyond it
        huge = 80 * (1 << 20)
        hsrc = [torch.zeros(huge, dtype=torch.int16, device="cuda") for _ in range(2)]
        hdst = [torch.empty(huge, dtype=torch.int16, device="cuda") for _ in range(2)]
        nb.nuna_allreduce_twoshot(hsrc, hdst, huge)                 # grows the scratch (160 MiB)
        torch.cuda.synchronize()
        del hsrc, hdst
        bsrc = workloads.special_values(n, big, seed=5)
        bdst = [torch.empty(big, dtype=torch.int16, device="cuda") for _ in range(n)]
        nb.nuna_allreduce_twoshot(upload(bsrc), bdst, big)          # uses the new scratch
        torch.cuda.synchronize()
        assert_same_bits(bdst[n - 1].cpu().numpy().view(np.uint16), oracle.allreduce(bsrc, nthreads=8)[0], "after growth")
        for _ in range(2):
            for t in dst.view:
                t.zero_()
            nb.nuna_chain_launch(chain)                             # still names the old scratch
            for got in dst.numpy():
                assert_same_bits(got, want, "replay after growth")
    finally:
        nb.nuna_chain_destroy(chain)
    assert nb.nuna_device_status() == nb.NUNA_OK


@pytest.mark.parametrize("flags", [0, nb.NUNA_LAUNCH_PDL, nb.NUNA_LAUNCH_PDL | nb.NUNA_PLACE_AWARE, nb.NUNA_CHAIN_PERSISTENT,
                                   nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_STAGED | nb.NUNA_LAUNCH_PDL])
def test_chain_nodes_are_ordered_even_with_dependent_launch(flags):
    """Node k+1 reads what node k wrote: ones -> 8 -> 64 -> 512 -> 4096 only if every node waited."""
    n, count, levels = 8, 1 << 20, 4
    one = np.int16(0x3F80)
    bufs = [[torch.full((count,), one, dtype=torch.int16, device="cuda") for _ in range(n)]]
    for _ in range(levels):
        bufs.append([torch.zeros(count, dtype=torch.int16, device="cuda") for _ in range(n)])
    chain = nb.nuna_chain_create(bufs[:-1], bufs[1:], levels, count, flags=flags)
    try:
        for _ in range(5):
            for lvl in bufs[1:]:
                for t in lvl:
                    t.zero_()
            nb.nuna_chain_launch(chain)
            torch.cuda.synchronize()
            for lvl, expect in zip(bufs[1:], (8.0, 64.0, 512.0, 4096.0)):
                for t in lvl:
                    v = t.view(torch.bfloat16)
                    assert float(v.min()) == expect and float(v.max()) == expect
    finally:
        nb.nuna_chain_destroy(chain)


def test_sm_lists_replay_and_after_probe():
    """The work-list kernel rewinds its own cursors: graph replays and repeated calls stay correct, with
    the one-domain plan (no probe yet in this process is not guaranteed, so both orders are exercised)."""
    flags = nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_SM_LISTS
    for n, count in ((8, 32 * 8192), (8, 4096), (3, 100003), (16, 1 << 20)):
        src = workloads.special_values(n, count, seed=n + count % 89)
        want = oracle.allreduce(src, nthreads=4)[0]
        dsrc = upload(src)
        dst = [torch.zeros(count, dtype=torch.int16, device="cuda") for _ in range(n)]
        nb.nuna_allreduce_oneshot(dsrc, dst, count, flags=flags)              # builds the plan (allocates)
        g = torch.cuda.CUDAGraph()
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            with torch.cuda.graph(g, stream=s):
                nb.nuna_allreduce_oneshot(dsrc, dst, count, flags=flags, stream=s)
                nb.nuna_allreduce_oneshot(dsrc, dst, count, flags=flags | nb.NUNA_LAUNCH_PDL, stream=s)
        for _ in range(4):
            for t in dst:
                t.fill_(-1)
            g.replay()
            torch.cuda.synchronize()
            for t in dst:
                assert_same_bits(t.cpu().numpy().view(np.uint16), want, f"sm lists n={n} count={count}")
    # after a probe the plan uses two domains: new shapes get new plans, results stay the same
    probe_bufs = [torch.zeros(1 << 16, dtype=torch.int16, device="cuda") for _ in range(4)]
    nb.nuna_probe_topology(probe_bufs)
    for n, count in ((8, 32 * 8192), (8, 64 * 8192), (8, 2048 + 8), (5, 33333)):       # first shape: planned before too
        src = workloads.special_values(n, count, seed=count)
        want = oracle.allreduce(src, nthreads=4)[0]
        dst = Dst(n, count)
        for _ in range(3):
            nb.nuna_allreduce_oneshot(upload(src), dst.view, count, flags=flags)
        for got in dst.numpy():
            assert_same_bits(got, want, "sm lists after probe")


def test_tuning_options_change_the_launch_not_the_bits():
    w = workloads.config_decode_activation()
    src = workloads.special_values(w.nranks, w.count + 5, seed=44)
    want = oracle.allreduce(src, nthreads=4)[0]
    dsrc = upload(src)
    try:
        for opt, values in ((nb.NUNA_OPT_BLOCKS, (1, 7, 148, 100000)), (nb.NUNA_OPT_UNROLL, (1, 2, 4)),
                            (nb.NUNA_OPT_COLOC, (2, 4, 8))):
            for v in values:
                nb.nuna_set_option(opt, v)
                for call, flags in ((nb.nuna_allreduce_oneshot, 0), (nb.nuna_allreduce_oneshot, nb.NUNA_PLACE_AWARE),
                                    (nb.nuna_allreduce_oneshot, nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_REGS),
                                    (nb.nuna_allreduce_twoshot, 0), (nb.nuna_allreduce_twoshot, nb.NUNA_TWOSHOT_PUT)):
                    dst = Dst(w.nranks, w.count + 5)
                    call(dsrc, dst.view, w.count + 5, flags=flags)
                    assert_same_bits(dst.numpy()[w.nranks - 1], want, f"option {opt}={v} {call.__name__} {flags}")
            nb.nuna_set_option(opt, 0)
        assert nb.nuna_set_option(99, 1, check=False) == nb.NUNA_ERR_INVALID_ARG
        assert nb.nuna_set_option(nb.NUNA_OPT_BLOCKS, -1, check=False) == nb.NUNA_ERR_INVALID_ARG
    finally:
        for opt in (nb.NUNA_OPT_BLOCKS, nb.NUNA_OPT_UNROLL, nb.NUNA_OPT_COLOC):
            nb.nuna_set_option(opt, 0)
    assert nb.nuna_device_status() == nb.NUNA_OK


def test_minimum_alignment_sixteen_bytes_only():
    """Buffers that are 16-byte aligned but not 32-, 64- or 128-byte aligned, each rank at a different offset."""
    n, count = 8, 20011
    src = workloads.special_values(n, count, seed=61)
    want = oracle.allreduce(src, nthreads=4)[0]
    pad = 8 * 16
    big_s = [torch.zeros(count + pad, dtype=torch.int16, device="cuda") for _ in range(n)]
    big_d = [torch.zeros(count + pad, dtype=torch.int16, device="cuda") for _ in range(n)]
    dsrc, ddst = [], []
    for r in range(n):
        off = 8 * (2 * r + 1)                                   # odd multiples of 16 bytes
        big_s[r][off:off + count] = torch.from_numpy(src[r].view(np.int16)).cuda()
        dsrc.append(big_s[r][off:off + count])
        ddst.append(big_d[r][8 * (2 * (n - r) - 1): 8 * (2 * (n - r) - 1) + count])
        assert dsrc[-1].data_ptr() % 32 == 16 and ddst[-1].data_ptr() % 32 == 16
    for call, flags in ((nb.nuna_allreduce_oneshot, 0), (nb.nuna_allreduce_oneshot, nb.NUNA_PLACE_AWARE),
                        (nb.nuna_allreduce_twoshot, 0), (nb.nuna_allreduce_twoshot, nb.NUNA_TWOSHOT_PUT)):
        for t in big_d:
            t.zero_()
        call(dsrc, ddst, count, flags=flags)
        torch.cuda.synchronize()
        for t in ddst:
            assert_same_bits(t.cpu().numpy().view(np.uint16), want, f"{call.__name__} {flags}")


def test_two_host_threads_on_their_own_streams():
    """Calls that share no library state (one-shot, two-shot put, allgather) may be issued from
    different host threads on different streams at the same time."""
    import threading
    n, count, rounds = 8, 64 * 1024 + 3, 40
    errors = []

    def worker(tid):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            src = workloads.special_values(n, count, seed=900 + tid)
            want = oracle.allreduce(src, nthreads=2)[0]
            with torch.cuda.stream(stream):
                dsrc = upload(src)
                dst = [torch.zeros(count, dtype=torch.int16, device="cuda") for _ in range(n)]
                stream.synchronize()
                for i in range(rounds):
                    flags = (0, nb.NUNA_PLACE_AWARE, nb.NUNA_LAUNCH_PDL)[i % 3]
                    if i % 2:
                        nb.nuna_allreduce_oneshot(dsrc, dst, count, flags=flags, stream=stream)
                    else:
                        nb.nuna_allreduce_twoshot(dsrc, dst, count, flags=nb.NUNA_TWOSHOT_PUT, stream=stream)
                stream.synchronize()
                for t in dst:
                    assert_same_bits(t.cpu().numpy().view(np.uint16), want, f"thread {tid}")
        except Exception as e:                                     # noqa: BLE001 - reported by the main thread
            errors.append((tid, repr(e)))

    threads = [threading.Thread(target=worker, args=(t,)) for t in range(4)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors


def test_size_selected_allreduce_matches_oracle_on_both_sides_of_the_threshold():
    for count in (1000, 64 * 1024, 64 * 1024 + 8, 300000, 512 * 1024 + 8):
        for flags in (0, nb.NUNA_TWOSHOT_SYNC, nb.NUNA_TWOSHOT_SYNC | nb.NUNA_LAUNCH_PDL,
                      nb.NUNA_LAUNCH_PDL | nb.NUNA_PLACE_AUTO):
            src = workloads.special_values(8, count, seed=count)
            want = oracle.allreduce(src, nthreads=4)[0]
            dst = Dst(8, count)
            nb.nuna_allreduce(upload(src), dst.view, count, flags=flags)
            for got in dst.numpy():
                assert_same_bits(got, want, f"auto count={count} flags={flags}")


def test_host_buffer_entry_point():
    for n, count, two in ((8, 32 * 8192, False), (8, 32 * 8192, True), (3, 1001, False), (3, 1001, True)):
        src = workloads.rank_buffers(n, count, "normal", seed=77)
        want = oracle.allreduce(src)[0]
        dst = [np.zeros(count, dtype=np.uint16) for _ in range(n)]
        nb.nuna_allreduce_host(src, dst, count, two_shot=two)
        for d in range(n):
            assert np.array_equal(dst[d], want)


def test_host_entry_point_in_place_on_pinned_buffers():
    for n, count in ((8, 32 * 8192), (3, 1001), (16, 4096)):
        src = workloads.special_values(n, count, seed=5 + n)
        want = oracle.allreduce(src, nthreads=4)[0]
        psrc = [torch.from_numpy(a.view(np.int16).copy()).pin_memory() for a in src]
        pdst = [torch.zeros(count, dtype=torch.int16).pin_memory() for _ in range(n)]
        before = nb.nuna_launch_count()
        nb.nuna_allreduce_host(psrc, pdst, count, flags=nb.NUNA_TWOSHOT_PUT, two_shot=True)
        assert nb.nuna_launch_count() == before + 1
        for t in pdst:
            assert_same_bits(t.numpy().view(np.uint16), want, "pinned in place")
        # pageable destinations fall back to staging copies, same bits
        hdst = [np.zeros(count, dtype=np.uint16) for _ in range(n)]
        nb.nuna_allreduce_host(psrc, hdst, count, flags=nb.NUNA_TWOSHOT_PUT, two_shot=True)
        for h in hdst:
            assert_same_bits(h, want, "pageable fallback")


def test_argument_errors_launch_nothing():
    a = [torch.zeros(64, dtype=torch.int16, device="cuda") for _ in range(2)]
    b = [torch.zeros(64, dtype=torch.int16, device="cuda") for _ in range(2)]
    before = nb.nuna_launch_count()
    assert nb.nuna_allreduce_oneshot(a, b, 0) == nb.NUNA_OK
    assert nb.nuna_allreduce_oneshot(a, a, 64, check=False) == nb.NUNA_ERR_ALIAS
    assert nb.nuna_allreduce_oneshot(a, [b[0], b[0]], 64, check=False) == nb.NUNA_ERR_ALIAS
    assert nb.nuna_allreduce_oneshot(a, [b[0], a[1][16:]], 32, check=False) == nb.NUNA_ERR_ALIAS
    assert nb.nuna_allreduce_oneshot(a, [b[0], b[1][1:]], 8, check=False) == nb.NUNA_ERR_ALIGNMENT
    assert nb.nuna_allreduce_oneshot(a, b, 64, dtype=5, check=False) == nb.NUNA_ERR_UNSUPPORTED_DTYPE
    assert nb.nuna_allreduce_oneshot(a, b, 64, flags=3, check=False) == nb.NUNA_ERR_INVALID_ARG
    assert nb.nuna_allreduce_oneshot(a, b, 64, flags=nb.NUNA_TWOSHOT_PUT, check=False) == nb.NUNA_ERR_INVALID_ARG
    assert nb.nuna_allreduce_oneshot(a * 9, b * 9, 64, check=False) == nb.NUNA_ERR_TOO_MANY_RANKS
    assert nb.nuna_allreduce_oneshot([a[0], 0], b, 64, check=False) == nb.NUNA_ERR_INVALID_ARG
    assert nb.nuna_launch_count() == before
    with pytest.raises(nb.NunaError):
        nb.nuna_allreduce_oneshot(a, a, 64)


def test_twoshot_ready_flag_wait_times_out_cleanly():
    """Consumers that wait for ready flags nobody publishes: every wait runs out after 50 ms, the kernel
    returns, the status word latches NUNA_ERR_TIMEOUT, and the next ordinary call works."""
    import time
    w = workloads.config_decode_activation()
    src = workloads.make(w)
    want = oracle.allreduce(src, nthreads=4)[0]
    dsrc = upload(src)
    dst = Dst(w.nranks, w.count)
    nb.nuna_allreduce_twoshot(dsrc, dst.view, w.count)             # context, scratch and flags exist
    assert nb.nuna_device_status() == nb.NUNA_OK
    t0 = time.time()
    assert nb.debug_twoshot(dsrc, dst.view, w.count, timeout_ms=50, unset_flags=True) == nb.NUNA_OK
    torch.cuda.synchronize()
    assert time.time() - t0 < 5.0                                  # bounded: nothing hangs
    assert nb.nuna_device_status() == nb.NUNA_ERR_TIMEOUT
    assert nb.nuna_device_status() == nb.NUNA_OK                   # cleared, control words rewound
    for flags in (0, nb.NUNA_LAUNCH_PDL):
        dst = Dst(w.nranks, w.count)
        nb.nuna_allreduce_twoshot(dsrc, dst.view, w.count, flags=flags)
        for got in dst.numpy():
            assert_same_bits(got, want, "two-shot after a timed-out launch")
    assert nb.nuna_device_status() == nb.NUNA_OK


def test_access_latency_sampling_counts_every_item_and_keeps_the_result():
    """The timed variants of the one-shot loops: one latency sample per warp and work item, every sample in a
    plausible range, and the destinations still hold the oracle's bits."""
    n, count = 8, 32 * 8192
    src = workloads.special_values(n, count, seed=606)
    want = oracle.allreduce(src, nthreads=4)[0]
    dsrc = upload(src)
    nvec = count // 8
    for placement, warp_items in ((0, n * nvec // 32), (1, n * nvec // 32), (2, n * nvec // 32)):
        dst = Dst(n, count)
        hist = nb.debug_access_latency(dsrc, dst.view, count, placement, launches=2)
        assert hist.sum() == 2 * warp_items, (placement, int(hist.sum()))
        assert hist[0] == 0                                        # nothing returns in under 32 cycles
        for got in dst.numpy():
            assert_same_bits(got, want, f"timed placement {placement}")
    assert nb.nuna_device_status() == nb.NUNA_OK


def test_domain_count_changes_no_bit():
    """The work-list planner dealt over 1, 2, 4 and 8 SM domains (with and without a probed topology)."""
    flags = nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_SM_LISTS
    n, count = 8, 32 * 8192 + 3
    src = workloads.special_values(n, count, seed=808)
    want = oracle.allreduce(src, nthreads=4)[0]
    dsrc = upload(src)
    try:
        for probe_first in (False, True):
            if probe_first:
                nb.nuna_probe_topology([torch.zeros(1 << 16, dtype=torch.int16, device="cuda") for _ in range(4)])
            for D in (1, 2, 4, 8, 0):
                nb.nuna_set_option(nb.NUNA_OPT_DOMAINS, D)
                dst = Dst(n, count)
                for _ in range(2):
                    nb.nuna_allreduce_oneshot(dsrc, dst.view, count, flags=flags)
                for got in dst.numpy():
                    assert_same_bits(got, want, f"domains={D} probed={probe_first}")
    finally:
        nb.nuna_set_option(nb.NUNA_OPT_DOMAINS, 0)
    assert nb.nuna_device_status() == nb.NUNA_OK


def test_probe_while_another_thread_launches_work_lists():
    """nuna_probe_topology retires the planned work lists while another host thread keeps launching the
    work-list kernel: launches use a copy of the plan taken under the lock, so nothing dangles."""
    import threading
    n, count = 8, 16 * 8192
    flags = nb.NUNA_PLACE_AWARE | nb.NUNA_PLACE_SM_LISTS
    src = workloads.special_values(n, count, seed=4242)
    want = oracle.allreduce(src, nthreads=4)[0]
    errors, stop = [], threading.Event()

    def launcher():
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                dsrc = upload(src)
                dst = [torch.zeros(count, dtype=torch.int16, device="cuda") for _ in range(n)]
                stream.synchronize()
                rounds = 0
                while not stop.is_set() or rounds < 20:
                    nb.nuna_allreduce_oneshot(dsrc, dst, count, flags=flags, stream=stream)
                    stream.synchronize()
                    rounds += 1
                    if rounds % 10 == 0:
                        assert_same_bits(dst[rounds % n].cpu().numpy().view(np.uint16), want, "during probes")
                assert_same_bits(dst[0].cpu().numpy().view(np.uint16), want, "after probes")
        except Exception as e:                                     # noqa: BLE001 - reported by the main thread
            errors.append(repr(e))

    t = threading.Thread(target=launcher)
    t.start()
    try:
        bufs = [torch.zeros(1 << 16, dtype=torch.int16, device="cuda") for _ in range(4)]
        side = torch.cuda.Stream()
        for i in range(4):
            nb.nuna_set_option(nb.NUNA_OPT_DOMAINS, (0, 4, 2, 0)[i])
            nb.nuna_probe_topology(bufs, stream=side)
    finally:
        stop.set()
        t.join()
        nb.nuna_set_option(nb.NUNA_OPT_DOMAINS, 0)
    assert not errors, errors


def test_flag_barrier_completes_and_times_out_cleanly():
    st, passed = nb.debug_barrier_selftest(64, 64, 1000)
    assert st == nb.NUNA_OK and passed == 64
    assert nb.nuna_device_status() == nb.NUNA_OK
    # a barrier nothing can complete: every wait runs out, the status word latches, nothing hangs
    st, passed = nb.debug_barrier_selftest(32, 33, 50)
    assert st == nb.NUNA_OK and passed == 0
    assert nb.nuna_device_status() == nb.NUNA_ERR_TIMEOUT
    assert nb.nuna_device_status() == nb.NUNA_OK            # cleared and barrier words re-initialised
    # the context is still usable
    w = workloads.config_decode_activation()
    src = workloads.make(w)
    dst = Dst(w.nranks, w.count)
    nb.nuna_allreduce_twoshot(upload(src), dst.view, w.count)
    assert np.array_equal(dst.numpy()[3], oracle.allreduce(src, nthreads=4)[0])
