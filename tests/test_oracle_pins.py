"""Pins for the CPU oracle: everything here is fixed by IEEE 754 and by the
collectives' definition, not by the oracle itself.  No GPU needed."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from oracle import exact_model
from paper_2608_00867_b200 import workloads


def u16(*vals):
    return np.array(vals, dtype=np.uint16)


def ar_column(column):
    """Run one column through the array entry point (not only through fold)."""
    src = [u16(v) for v in column]
    out = oracle.allreduce(src)
    assert all(int(o[0]) == int(out[0][0]) for o in out)
    return int(out[0][0])


# ---- hand-derived single-column pins ----------------------------------------------------
# Each expected value is derived in the comment from the IEEE rules alone.
PINS = [
    # 2^24 + 1 is a binary32 tie and rounds to even (2^24) twice; minus 2^24 leaves +0.
    # A pairwise tree would give 1.0 (0x3F80), exact arithmetic 2.0 (0x4000).
    ("left fold, not a tree", [0x4B80, 0x3F80, 0x3F80, 0xCB80], 0x0000),
    # 1 + 2^24 -> 2^24; - 2^24 -> 0; + 1 -> 1.  Folding 3..0 instead would give 2.0.
    ("rank order 0..N-1", [0x3F80, 0x4B80, 0xCB80, 0x3F80], 0x3F80),
    # 1 + 2^-8 + 2^-8 = 1 + 2^-7 exactly in binary32 = next bf16 after 1.0.
    # Accumulating in bf16 would round 1 + 2^-8 back to 1.0 both times.
    ("binary32 accumulator", [0x3F80, 0x3B80, 0x3B80], 0x3F81),
    # 1 + 2^-8 is exactly half way between bf16 1.0 and 1.0078125: ties go to even (down).
    ("tie to even, down", [0x3F80, 0x3B80], 0x3F80),
    # 1.0078125 + 2^-8 is half way between 0x3F81 and 0x3F82: even is up.  Truncation gives 0x3F81.
    ("tie to even, up", [0x3F81, 0x3B80], 0x3F82),
    # (-0) + (-0) = -0; an accumulator started at +0 would give +0.
    ("accumulator starts from rank 0", [0x8000, 0x8000], 0x8000),
    # x + (-x) = +0 in round-to-nearest.
    ("exact cancellation is +0", [0xBF80, 0x3F80], 0x0000),
    # twice the largest finite bf16 overflows binary32 to +Inf.
    ("overflow", [0x7F7F, 0x7F7F], 0x7F80),
    ("overflow negative", [0xFF7F, 0xFF7F], 0xFF80),
    # smallest subnormal twice: gradual underflow, no flush to zero.
    ("subnormals kept", [0x0001, 0x0001], 0x0002),
    # largest bf16 plus half an ulp of bf16 in binary32 rounds up to Inf at the final rounding only:
    # 0x7F7F = (2-2^-7)*2^127; adding 2^119 (0x7B00) gives (2-2^-7+2^-8)*2^127, a bf16 tie -> even = Inf.
    ("final rounding can overflow", [0x7F7F, 0x7B00], 0x7F80),
    # integers: exact
    ("eight ones", [0x3F80] * 8, 0x4100),
    ("sixteen ones", [0x3F80] * 16, 0x4180),
    # 1+2+...+8 = 36 = 1.125 * 2^5 -> 0x4210
    ("1..8", [0x3F80, 0x4000, 0x4040, 0x4080, 0x40A0, 0x40C0, 0x40E0, 0x4100], 0x4210),
    ("single rank is the identity", [0x1234], 0x1234),
]


@pytest.mark.parametrize("name,column,expect", PINS, ids=[p[0] for p in PINS])
def test_hand_pins(name, column, expect):
    assert oracle.fold(column) == expect
    assert ar_column(column) == expect
    assert exact_model.fold(column) == expect


def test_nan_pins():
    assert exact_model.is_nan_bf16(oracle.fold([0x7F80, 0xFF80]))      # Inf + -Inf
    assert exact_model.is_nan_bf16(oracle.fold([0x7FC1, 0x3F80, 0x3F80]))
    assert oracle.fold([0x7F80, 0x3F80]) == 0x7F80                     # Inf + 1 = Inf
    assert oracle.fold([0x7FC0]) == 0x7FFF or exact_model.is_nan_bf16(oracle.fold([0x7FC0]))


# ---- the two conversions against torch's own (library special cases) --------------------

def test_widen_is_shift():
    for h in (0x0000, 0x8000, 0x3F80, 0x0001, 0x7F7F, 0xC2F7):
        assert oracle.widen_bf16(h) == float(
            torch.tensor([h], dtype=torch.uint16).view(torch.bfloat16).float()[0])


def test_rne_matches_torch_conversion():
    rng = np.random.Generator(np.random.PCG64(7))
    bits = rng.integers(0, 1 << 32, size=20000, dtype=np.uint64).astype(np.uint32)
    # force plenty of exact ties and near-ties in the dropped half
    bits[:4000] = (bits[:4000] & 0xFFFF0000) | 0x8000
    bits[4000:6000] = (bits[4000:6000] & 0xFFFF0000) | 0x7FFF
    bits[6000:8000] = (bits[6000:8000] & 0xFFFF0000) | 0x8001
    x = bits.view(np.float32)
    ref = torch.from_numpy(x.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    for xi, ri in zip(x, ref):
        got = oracle.rne_bf16(float(xi))
        if np.isnan(xi):
            assert exact_model.is_nan_bf16(got)
        else:
            assert got == int(ri), hex(int(np.float32(xi).view(np.uint32)))


# ---- N = 2 reduces to one library add -----------------------------------------------------

def _interesting_patterns():
    pats = set()
    for e in (0, 1, 2, 0x3B, 0x70, 0x77, 0x7E, 0x7F, 0x80, 0x86, 0x97, 0xFD, 0xFE, 0xFF):
        for m in (0, 1, 2, 0x3F, 0x40, 0x41, 0x7E, 0x7F):
            for s in (0, 1):
                pats.add((s << 15) | (e << 7) | m)
    return sorted(pats)


def test_two_ranks_equal_torch_add_all_pairs():
    pats = np.array(_interesting_patterns(), dtype=np.uint16)
    a, b = np.meshgrid(pats, pats, indexing="ij")
    a, b = a.ravel().copy(), b.ravel().copy()
    got = oracle.allreduce([a, b])[0]
    ta = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).float()
    tb = torch.from_numpy(b.view(np.int16)).view(torch.bfloat16).float()
    ref = (ta + tb).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    nan = torch.isnan(ta + tb).numpy()
    assert np.array_equal(got[~nan], ref[~nan])
    assert all(exact_model.is_nan_bf16(int(g)) for g in got[nan])
    # N = 2 is commutative: swapping the two rank buffers changes nothing
    assert np.array_equal(got, oracle.allreduce([b, a])[0])


# ---- brute force against the exact-rational model ---------------------------------------

def test_exact_model_brute_force_pairs_and_triples():
    pats = _interesting_patterns()[::3]
    for col in itertools.product(pats, repeat=2):
        e = exact_model.fold(col)
        g = oracle.fold(col)
        assert g == e or (exact_model.is_nan_bf16(e) and exact_model.is_nan_bf16(g)), col
    rng = np.random.Generator(np.random.PCG64(11))
    for _ in range(3000):
        col = [pats[i] for i in rng.integers(0, len(pats), size=3)]
        e, g = exact_model.fold(col), oracle.fold(col)
        assert g == e or (exact_model.is_nan_bf16(e) and exact_model.is_nan_bf16(g)), col


@pytest.mark.parametrize("n", [2, 3, 5, 8, 16])
def test_exact_model_random_columns(n):
    count = 600
    src = workloads.special_values(n, count, seed=100 + n)
    got = oracle.allreduce(src)[0]
    for i in range(count):
        col = [int(s[i]) for s in src]
        e = exact_model.fold(col)
        assert int(got[i]) == e or (exact_model.is_nan_bf16(e) and exact_model.is_nan_bf16(int(got[i]))), col


def test_exact_model_on_benchmark_like_values():
    src = workloads.rank_buffers(8, 400, "normal", seed=5)
    got = oracle.allreduce(src)[0]
    for i in range(400):
        assert int(got[i]) == exact_model.fold([int(s[i]) for s in src])


# ---- closed forms and metamorphic relations ------------------------------------------------

@pytest.mark.parametrize("n", [1, 2, 3, 8, 16])
def test_small_integers_sum_exactly(n):
    rng = np.random.Generator(np.random.PCG64(n))
    vals = rng.integers(-8, 9, size=(n, 1000))
    src = [torch.from_numpy(v.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
           for v in vals]
    got = oracle.allreduce(src)[0]
    back = torch.from_numpy(got.view(np.int16)).view(torch.bfloat16).float().numpy()
    assert np.array_equal(back, vals.sum(axis=0).astype(np.float32))   # |sum| <= 128: exact in bf16


def test_power_of_two_scaling_commutes():
    src = workloads.rank_buffers(8, 4096, "normal", seed=9)
    base = oracle.allreduce(src)[0]
    for k in (-20, -3, 5, 40):
        scaled = [((s.astype(np.int32) + (k << 7)).astype(np.uint16)) for s in src]   # exponent += k
        ok = np.ones(len(base), bool)
        for s in src:
            e = ((s >> 7) & 0xFF).astype(np.int32)
            ok &= (e > 30) & (e + k > 30) & (e + k < 220)     # stay clear of subnormals / overflow
        be = ((base >> 7) & 0xFF).astype(np.int32)
        ok &= (be > 30) & (be + k > 30) & (be + k < 220)
        got = oracle.allreduce(scaled)[0]
        want = (base.astype(np.int32) + (k << 7)).astype(np.uint16)
        assert ok.sum() > 3000
        assert np.array_equal(got[ok], want[ok])


def test_swapping_first_two_ranks_changes_nothing():
    src = workloads.special_values(6, 5000, seed=21)
    a = oracle.allreduce(src)[0]
    b = oracle.allreduce([src[1], src[0]] + src[2:])[0]
    nan = np.array([exact_model.is_nan_bf16(int(x)) for x in a])
    assert np.array_equal(a[~nan], b[~nan])


def test_order_matters_beyond_the_first_two():
    # Sanity check of the pins' power.  bf16 inputs of similar magnitude sum exactly in
    # binary32 (8-bit significands, 24-bit accumulator), so benign data cannot see the
    # order; columns with a wide exponent spread can, and there reversing the ranks
    # must change some results.
    src = workloads.special_values(8, 20000, seed=3)
    a, b = oracle.allreduce(src)[0], oracle.allreduce(src[::-1])[0]
    nan = np.array([exact_model.is_nan_bf16(int(x)) for x in a])
    assert not np.array_equal(a[~nan], b[~nan])


# ---- invariants of the collectives ------------------------------------------------------------

@pytest.mark.parametrize("n,count", [(2, 4096), (8, 8 * 1000), (16, 16 * 33), (3, 3 * 7)])
def test_allreduce_is_reduce_scatter_then_allgather(n, count):
    src = workloads.rank_buffers(n, count, "normal", seed=n)
    ar = oracle.allreduce(src)
    for d in range(1, n):
        assert np.array_equal(ar[0], ar[d])                  # all destinations identical
    rs = oracle.reduce_scatter(src)
    assert all(len(x) == count // n for x in rs)
    ag = oracle.allgather(rs)
    for d in range(n):
        assert np.array_equal(ag[d], ar[d])


def test_reduce_scatter_shard_r_is_slice_r_of_the_sum():
    n, shard = 4, 129
    src = workloads.special_values(n, n * shard, seed=77)
    rs = oracle.reduce_scatter(src)
    for r in range(n):
        for j in (0, 1, shard - 1):
            assert int(rs[r][j]) == oracle.fold([int(s[r * shard + j]) for s in src])


def test_allgather_is_rank_order_concatenation_of_raw_bits():
    n, shard = 16, 257
    rng = np.random.Generator(np.random.PCG64(4))
    src = [rng.integers(0, 1 << 16, size=shard, dtype=np.uint32).astype(np.uint16) for _ in range(n)]
    out = oracle.allgather(src)
    cat = np.concatenate(src)                                # NaN payloads, -0: plain bit copy
    assert len(out) == n
    for d in range(n):
        assert np.array_equal(out[d], cat)


def test_threads_do_not_change_bits():
    src = workloads.rank_buffers(8, 100003, "normal", seed=12)
    assert np.array_equal(oracle.allreduce(src, 1)[0], oracle.allreduce(src, 8)[0])
    src = [s[:100000] for s in src]
    a, b = oracle.reduce_scatter(src, 1), oracle.reduce_scatter(src, 8)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))


def test_empty_and_single():
    assert [len(x) for x in oracle.allreduce([u16(), u16()])] == [0, 0]
    one = u16(0x3F80, 0xFFFF, 0x8000)
    assert np.array_equal(oracle.allreduce([one])[0][[0, 2]], one[[0, 2]])
    assert np.array_equal(oracle.allgather([one])[0], one)


# ---- alltoall: a block transpose of raw bits -----------------------------------------------------------

def test_alltoall_is_the_block_transpose():
    n, block = 5, 37
    rng = np.random.Generator(np.random.PCG64(6))
    src = [rng.integers(0, 1 << 16, size=n * block, dtype=np.uint32).astype(np.uint16) for _ in range(n)]
    out = oracle.alltoall(src)
    cube = np.stack([s.reshape(n, block) for s in src])          # [sender r][receiver d][i]
    want = cube.transpose(1, 0, 2)                               # [receiver d][sender r][i]  (numpy's own transpose)
    for d in range(n):
        assert np.array_equal(out[d], want[d].reshape(-1))
    # applying it twice returns every buffer to where it started
    back = oracle.alltoall(out)
    for r in range(n):
        assert np.array_equal(back[r], src[r])


def test_alltoall_of_replicated_blocks_is_allgather():
    n, block = 4, 64
    shards = workloads.rank_buffers(n, block, "uniform", seed=2)
    src = [np.tile(s, n) for s in shards]                        # rank r sends the same block to everyone
    a2a, ag = oracle.alltoall(src), oracle.allgather(shards)
    for d in range(n):
        assert np.array_equal(a2a[d], ag[d])
    assert np.array_equal(oracle.alltoall([shards[0]])[0], shards[0])   # one rank: identity
    assert np.array_equal(oracle.alltoall(src, 1)[2], oracle.alltoall(src, 8)[2])


def test_allreduce_into_caller_owned_destinations():
    """out=: same bits as the allocating form, written in place; bad destinations are refused."""
    src = workloads.special_values(5, 1003, seed=77)
    want = oracle.allreduce(src, nthreads=2)
    out = [np.full(1003, 0xBEEF, dtype=np.uint16) for _ in range(5)]
    got = oracle.allreduce(src, nthreads=2, out=out)
    assert all(g is o for g, o in zip(got, out))
    assert all(np.array_equal(o, w) for o, w in zip(out, want))
    with pytest.raises(ValueError):
        oracle.allreduce(src, out=out[:4])
    with pytest.raises(ValueError):
        oracle.allreduce(src, out=[np.zeros(1003, dtype=np.uint32) for _ in range(5)])
