"""Seeded synthetic rank buffers shaped like the paper's inference collectives.

This module is shared by the CPU oracle's tests and by the CUDA path's tests
and benchmark.  It holds none of the method's arithmetic: values are drawn by
torch's CPU generator and narrowed to bf16 by torch's own conversion, and the
result is handed out as raw 16-bit patterns (numpy ``uint16``).  Neither the
oracle nor the CUDA library is imported here.

Workload shapes follow the paper's characterisation of tensor-parallel
inference traffic (Section 2.2: decode collectives are KB-range, prefill ones
reach tens of MB; Section 6.7: Llama-70B-class, eight-way tensor parallelism):
a rank buffer is one partial activation of ``tokens x hidden`` bf16 values.
Sizes quoted in KB/MB are binary (KiB/MiB).
"""
from __future__ import annotations

import dataclasses
from typing import List

import numpy as np
import torch

HIDDEN = 8192  # Llama-70B-class hidden size used by the decode-step configurations


@dataclasses.dataclass(frozen=True)
class Workload:
    """One collective call: ``nranks`` rank buffers of ``count`` bf16 elements."""
    name: str
    op: str            # "allreduce" | "allgather" | "reduce_scatter"
    nranks: int
    count: int         # elements per *source* rank buffer
    dist: str          # "uniform" (U[-1,1)) or "normal" (N(0,1))
    seed: int

    @property
    def bytes_per_rank(self) -> int:
        return 2 * self.count


def _draw(count: int, dist: str, gen: torch.Generator) -> torch.Tensor:
    if dist == "uniform":
        x = torch.rand(count, generator=gen, dtype=torch.float32) * 2.0 - 1.0
    elif dist == "normal":
        x = torch.randn(count, generator=gen, dtype=torch.float32)
    else:
        raise ValueError(f"unknown distribution {dist!r}")
    return x.to(torch.bfloat16)


def rank_buffers(nranks: int, count: int, dist: str, seed: int) -> List[np.ndarray]:
    """``nranks`` arrays of ``count`` bf16 bit patterns (uint16), one generator stream per rank."""
    out = []
    for r in range(nranks):
        gen = torch.Generator(device="cpu")
        gen.manual_seed((int(seed) << 20) + r)
        t = _draw(count, dist, gen)
        out.append(t.view(torch.int16).numpy().view(np.uint16).copy())
    return out


def make(w: Workload) -> List[np.ndarray]:
    return rank_buffers(w.nranks, w.count, w.dist, w.seed)


# ---- the five benchmark configurations -------------------------------------------------

def config_small_oneshot() -> Workload:
    """Two ranks, 4096 bf16 each (8 KiB), U[-1,1), seed 0."""
    return Workload("ar_n2_8KiB", "allreduce", 2, 4096, "uniform", 0)


def config_decode_activation() -> Workload:
    """Eight ranks, batch 32 x hidden 8192 bf16 (512 KiB per rank), N(0,1), seed 1."""
    return Workload("ar_n8_512KiB", "allreduce", 8, 32 * HIDDEN, "normal", 1)


def config_size_sweep(min_log2: int = 13, max_log2: int = 26) -> List[Workload]:
    """Eight ranks, 8 KiB ... 64 MiB per rank in powers of two, N(0,1), seed 2+log2(bytes)."""
    return [Workload(f"ar_n8_2^{k}B", "allreduce", 8, (1 << k) // 2, "normal", 2 + k)
            for k in range(min_log2, max_log2 + 1)]


def config_allgather16() -> Workload:
    """Sixteen ranks, 64 KiB shard per rank, U[-1,1), seed 3."""
    return Workload("ag_n16_64KiB", "allgather", 16, 32768, "uniform", 3)


def config_alltoall8() -> Workload:
    """Expert token routing: eight ranks, 64 KiB per (sender, receiver) pair, 512 KiB per rank, N(0,1)."""
    return Workload("a2a_n8_64KiB", "alltoall", 8, 8 * 32768, "normal", 6)


def config_decode_chain(tokens: int) -> Workload:
    """One node of the decode-step chain: eight ranks, tokens x 8192 bf16, N(0,1)."""
    k = {1: 0, 8: 1, 64: 2, 256: 3}.get(tokens, 4)
    return Workload(f"chain_n8_t{tokens}", "allreduce", 8, tokens * HIDDEN, "normal", 40 + k)


CHAIN_NODES = 160          # 2 allreduces per layer x 80 layers
CHAIN_TOKENS = (1, 8, 64, 256)


# ---- adversarial value mixes for parity (not benchmark inputs) --------------------------

def special_values(nranks: int, count: int, seed: int, dtype: str = "bf16") -> List[np.ndarray]:
    """Random bit patterns biased towards the awkward corners of the element type.

    A third of the elements are arbitrary bit patterns (NaN, Inf, subnormals
    included), a third are small integers whose sums are exact, the rest are
    values with mantissa ties around 1.0 so that round-to-nearest-even matters.
    Returned as raw storage words: uint16 for bf16 / f16, uint32 for f32.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    tdt = {"bf16": torch.bfloat16, "f16": torch.float16, "f32": torch.float32}[dtype]
    if dtype == "f32":
        word, view, bits = np.uint32, torch.int32, 32
        one, tiny = 0x3F800000, 0x33800000            # 1.0 and 2^-24 (half an ulp of 1.0)
    elif dtype == "f16":
        word, view, bits = np.uint16, torch.int16, 16
        one, tiny = 0x3C00, 0x1000                    # 1.0 and 2^-11
    else:
        word, view, bits = np.uint16, torch.int16, 16
        one, tiny = 0x3F80, 0x3B80                    # 1.0 and 2^-8
    out = []
    for _ in range(nranks):
        kind = rng.integers(0, 3, size=count)
        raw = rng.integers(0, 1 << bits, size=count, dtype=np.uint64).astype(word)
        ints = torch.from_numpy(rng.integers(-8, 9, size=count).astype(np.float32)) \
            .to(tdt).view(view).numpy().view(word)
        # 1.0 + k ulp and +-(half an ulp of 1.0): sums of these land on rounding ties
        ties = np.where(rng.integers(0, 2, size=count) == 0,
                        (one + rng.integers(0, 4, size=count)).astype(word),
                        (tiny + rng.integers(0, 2, size=count) * (1 << (bits - 1))).astype(word))
        buf = np.where(kind == 0, raw, np.where(kind == 1, ints, ties)).astype(word)
        out.append(buf)
    return out


def rank_buffers_typed(nranks: int, count: int, dist: str, seed: int, dtype: str) -> List[np.ndarray]:
    """Like rank_buffers, for any element type (raw storage words)."""
    tdt = {"bf16": torch.bfloat16, "f16": torch.float16, "f32": torch.float32}[dtype]
    view, word = (torch.int32, np.uint32) if dtype == "f32" else (torch.int16, np.uint16)
    out = []
    for r in range(nranks):
        gen = torch.Generator(device="cpu")
        gen.manual_seed((int(seed) << 20) + r)
        x = torch.randn(count, generator=gen) if dist == "normal" else torch.rand(count, generator=gen) * 2.0 - 1.0
        out.append(x.to(tdt).view(view).numpy().view(word).copy())
    return out
