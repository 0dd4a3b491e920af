"""Pins for the oracle's binary16 and binary32 variants (same fold, other storage types)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import exact_model
from paper_2608_00867_b200 import workloads


def fold16(column):
    return int(oracle.allreduce([np.array([v], dtype=np.uint16) for v in column], dtype="f16")[0][0])


def fold32(column):
    return int(oracle.allreduce([np.array([v], dtype=np.uint32) for v in column], dtype="f32")[0][0])


F16_PINS = [
    # 1 + 2^-11 is half way between 1.0 and the next half: ties to even (down)
    ("tie down", [0x3C00, 0x1000], 0x3C00),
    # (1 + 2^-10) + 2^-11: half way between 0x3C01 and 0x3C02, even is up
    ("tie up", [0x3C01, 0x1000], 0x3C02),
    # binary32 accumulator: 1 + 2^-11 + 2^-11 = 1 + 2^-10 exactly; a half accumulator would stay at 1.0
    ("binary32 accumulator", [0x3C00, 0x1000, 0x1000], 0x3C01),
    # 65504 + 2^-10 rounds back to 65504 in binary32 (ulp 2^-8 there), minus 65504 leaves +0;
    # folding the two large values first would leave 2^-10 (0x1400)
    ("left fold", [0x7BFF, 0x1400, 0xFBFF], 0x0000),
    ("rank order", [0x1400, 0x7BFF, 0xFBFF], 0x0000),
    ("other order differs", [0x7BFF, 0xFBFF, 0x1400], 0x1400),
    ("signed zero", [0x8000, 0x8000], 0x8000),
    # 65504 + 65504 = 131008 >= 65520: infinity
    ("overflow", [0x7BFF, 0x7BFF], 0x7C00),
    # 65504 + 16 = 65520: exactly the tie between 65504 and 2^16, even is 2^16 = infinity
    ("overflow at the final rounding", [0x7BFF, 0x4C00], 0x7C00),
    # 65504 + 8 = 65512 < 65520: stays finite
    ("just below overflow", [0x7BFF, 0x4800], 0x7BFF),
    ("subnormals kept", [0x0001, 0x0001], 0x0002),
    # largest subnormal + smallest subnormal = smallest normal
    ("subnormal to normal", [0x03FF, 0x0001], 0x0400),
    ("eight ones", [0x3C00] * 8, 0x4800),
    ("identity", [0x1234], 0x1234),
]


@pytest.mark.parametrize("name,column,expect", F16_PINS, ids=[p[0] for p in F16_PINS])
def test_f16_hand_pins(name, column, expect):
    assert fold16(column) == expect
    assert exact_model.fold_fmt(column, "f16") == expect


F32_PINS = [
    ("left fold", [0x4B800000, 0x3F800000, 0x3F800000, 0xCB800000], 0x00000000),     # 2^24 + 1 + 1 - 2^24 = 0
    ("rank order", [0x3F800000, 0x4B800000, 0xCB800000, 0x3F800000], 0x3F800000),
    ("tie to even", [0x3F800000, 0x33800000], 0x3F800000),                            # 1 + 2^-24
    ("tie to even up", [0x3F800001, 0x33800000], 0x3F800002),
    ("signed zero", [0x80000000, 0x80000000], 0x80000000),
    ("overflow", [0x7F7FFFFF, 0x7F7FFFFF], 0x7F800000),
    ("subnormals kept", [0x00000001, 0x00000001], 0x00000002),
    ("identity", [0x12345678], 0x12345678),
]


@pytest.mark.parametrize("name,column,expect", F32_PINS, ids=[p[0] for p in F32_PINS])
def test_f32_hand_pins(name, column, expect):
    assert fold32(column) == expect
    assert exact_model.fold_fmt(column, "f32") == expect


def test_f16_conversions_match_torch():
    # every half pattern widens like torch's own conversion
    allh = np.arange(1 << 16, dtype=np.uint32).astype(np.uint16)
    ref = torch.from_numpy(allh.view(np.int16)).view(torch.float16).float().numpy()
    for h in list(range(0, 1 << 16, 97)) + [0x0001, 0x03FF, 0x0400, 0x7BFF, 0x7C00, 0xFC00, 0x8001]:
        got = np.float32(oracle.widen_f16(h))
        assert (np.isnan(got) and np.isnan(ref[h])) or got.view(np.uint32) == ref[h].view(np.uint32), hex(h)
    # narrowing: random binary32 values, exact ties, the subnormal range and the overflow boundary
    rng = np.random.Generator(np.random.PCG64(3))
    bits = rng.integers(0, 1 << 32, size=30000, dtype=np.uint64).astype(np.uint32)
    bits[:6000] = (bits[:6000] & 0xFFFFE000) | 0x1000                  # exact ties in the dropped 13 bits
    bits[6000:9000] = (bits[6000:9000] & 0xFFFFE000) | 0x0FFF
    bits[9000:12000] = (bits[9000:12000] & 0x807FFFFF) | (rng.integers(100, 116, size=3000).astype(np.uint32) << 23)  # 2^-27..2^-12
    bits[12000:15000] = (bits[12000:15000] & 0x807FFFFF) | (rng.integers(140, 145, size=3000).astype(np.uint32) << 23)  # near 2^16
    extra = np.array([65504.0, 65519.996, 65520.0, 65536.0, 2.0 ** -24, 2.0 ** -25, 1.5 * 2.0 ** -25, 2.0 ** -14,
                      0.999999 * 2.0 ** -14, -65520.0, 5.9604645e-08], dtype=np.float32)
    x = np.concatenate([bits.view(np.float32), extra])
    ref = torch.from_numpy(x.copy()).to(torch.float16).view(torch.int16).numpy().view(np.uint16)
    for xi, ri in zip(x, ref):
        got = oracle.rne_f16(float(xi))
        if np.isnan(xi):
            assert exact_model.is_nan_fmt(got, "f16")
        else:
            assert got == int(ri), (float(xi), hex(got), hex(int(ri)))


def _patterns16():
    pats = set()
    for e in (0, 1, 2, 4, 14, 15, 16, 25, 29, 30, 31):
        for m in (0, 1, 2, 0x1FF, 0x200, 0x201, 0x3FE, 0x3FF):
            for s in (0, 1):
                pats.add((s << 15) | (e << 10) | m)
    return sorted(pats)


def test_f16_two_ranks_equal_one_torch_add():
    pats = np.array(_patterns16(), dtype=np.uint16)
    a, b = np.meshgrid(pats, pats, indexing="ij")
    a, b = a.ravel().copy(), b.ravel().copy()
    got = oracle.allreduce([a, b], dtype="f16")[0]
    ta = torch.from_numpy(a.view(np.int16)).view(torch.float16).float()
    tb = torch.from_numpy(b.view(np.int16)).view(torch.float16).float()
    ref = (ta + tb).to(torch.float16).view(torch.int16).numpy().view(np.uint16)
    nan = torch.isnan(ta + tb).numpy()
    assert np.array_equal(got[~nan], ref[~nan])
    assert all(exact_model.is_nan_fmt(int(g), "f16") for g in got[nan])


def test_f32_fold_equals_sequential_numpy_adds():
    src = workloads.special_values(8, 20000, seed=5, dtype="f32")
    got = oracle.allreduce(src, dtype="f32")[0]
    with np.errstate(all="ignore"):
        acc = src[0].view(np.float32).copy()
        for s in src[1:]:
            acc = (acc + s.view(np.float32)).astype(np.float32)
    nan = np.isnan(acc)
    assert np.array_equal(got[~nan], acc.view(np.uint32)[~nan])
    assert np.isnan(got.view(np.float32)[nan]).all()


@pytest.mark.parametrize("dtype", ["f16", "f32"])
@pytest.mark.parametrize("n", [2, 3, 8, 16])
def test_exact_model_random_columns(dtype, n):
    count = 400
    src = workloads.special_values(n, count, seed=7 * n, dtype=dtype)
    got = oracle.allreduce(src, dtype=dtype)[0]
    for i in range(count):
        col = [int(s[i]) for s in src]
        e = exact_model.fold_fmt(col, dtype)
        g = int(got[i])
        assert g == e or (exact_model.is_nan_fmt(e, dtype) and exact_model.is_nan_fmt(g, dtype)), (col, hex(g), hex(e))


def test_generalised_exact_model_agrees_with_the_bf16_one():
    src = workloads.special_values(5, 500, seed=1)
    for i in range(500):
        col = [int(s[i]) for s in src]
        a, b = exact_model.fold(col), exact_model.fold_fmt(col, "bf16")
        assert a == b or (exact_model.is_nan_bf16(a) and exact_model.is_nan_fmt(b, "bf16"))


@pytest.mark.parametrize("dtype", ["f16", "f32"])
def test_invariants_other_dtypes(dtype):
    n, count = 8, 8 * 513
    src = workloads.rank_buffers_typed(n, count, "normal", seed=2, dtype=dtype)
    ar = oracle.allreduce(src, nthreads=4, dtype=dtype)
    assert all(np.array_equal(ar[0], x) for x in ar[1:])
    rs = oracle.reduce_scatter(src, nthreads=1, dtype=dtype)
    assert np.array_equal(np.concatenate(rs), ar[0])                      # AR = AG(RS): shards concatenated in rank order
    ints = np.random.Generator(np.random.PCG64(1)).integers(-8, 9, size=(n, 300))
    tdt = torch.float16 if dtype == "f16" else torch.float32
    view, word = (torch.int16, np.uint16) if dtype == "f16" else (torch.int32, np.uint32)
    isrc = [torch.from_numpy(v.astype(np.float32)).to(tdt).view(view).numpy().view(word) for v in ints]
    got = oracle.allreduce(isrc, dtype=dtype)[0]
    back = torch.from_numpy(got.view(np.int16 if dtype == "f16" else np.int32)).view(tdt).float().numpy()
    assert np.array_equal(back, ints.sum(axis=0).astype(np.float32))
