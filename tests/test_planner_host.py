"""The library's host planner (nuna_plan_placement) against the Python restatement of Algorithm 1."""
import os

import numpy as np
import pytest

from oracle import nap_planner as nap
from paper_2608_00867_b200 import binding as nb
from paper_2608_00867_b200 import build as nbuild

from test_oracle_planner import load_figure_example


@pytest.fixture(scope="module", autouse=True)
def built_library():
    nbuild.build()


def to_oracle_topology(cu_domain, cu_rank, cu_stack, num_stacks, nar_max):
    doms = [[] for _ in range(nar_max)]
    for cu, d in enumerate(cu_domain):
        doms[d].append(cu)
    doms = [sorted(d, key=lambda c: (cu_rank[c], c)) for d in doms]
    stacks = {cu: [cu_stack[cu]] + [s for s in range(num_stacks) if s != cu_stack[cu]] for cu in range(len(cu_domain))}
    return {"domain_cus": doms, "cu_stacks": stacks}


def run_both(tb_gpu, tb_chunks, chunk_bytes, cu_domain, cu_rank, cu_stack, num_stacks, r_cu, r_stack, nar_max):
    mc, mm, td, tg = nb.nuna_plan_placement(tb_gpu, tb_chunks, chunk_bytes, cu_domain, cu_rank, cu_stack, num_stacks,
                                            r_cu, r_stack, nar_max)
    W = [(g, t, [(c, "b", 0) for c in cs]) for t, (g, cs) in enumerate(zip(tb_gpu, tb_chunks))]
    cb = {(c, "b", 0): b for c, b in enumerate(chunk_bytes)}
    topo = to_oracle_topology(cu_domain, cu_rank, cu_stack, num_stacks, nar_max)
    M_compute, M_memory, dom = nap.nuna_aware_placement(topo, r_cu, r_stack, nar_max, W, cb)
    for t, g in enumerate(tb_gpu):
        assert mc[t] == M_compute[(g, t)], ("M_compute", t)
        assert td[t] == dom[(g, t)], ("domain", t)
    for c in range(len(chunk_bytes)):
        assert mm[c] == M_memory.get((c, "b", 0), -1), ("M_memory", c)
    return mc, mm, td, tg


def test_figure_example_through_the_library():
    W, chunk_bytes, nar_max, expect = load_figure_example()
    ids = {c: i for i, c in enumerate(sorted(chunk_bytes))}
    tb_gpu = [g for g, _, _ in W]
    tb_chunks = [[ids[c] for c in cs] for _, _, cs in W]
    cb = [chunk_bytes[c] for c in sorted(chunk_bytes)]
    cu_domain = [0, 0, 1, 1, 2, 2, 3, 3]
    mc, mm, td, tg = nb.nuna_plan_placement(tb_gpu, tb_chunks, cb, cu_domain, [0] * 8, [d % 2 for d in cu_domain], 2,
                                            1 << 20, 1 << 20, nar_max)
    assert td == [expect[(g, name)] for g, name, _ in W]          # w, x, y, z -> domains 0, 1, 2, 3
    assert tg == [0, 1, 2, 3]
    assert [cu_domain[c] for c in mc] == td


@pytest.mark.parametrize("seed", range(12))
def test_random_workloads_match_the_oracle(seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    nar_max = int(rng.integers(1, 5))
    num_cus = int(rng.integers(nar_max, 24))
    num_stacks = int(rng.integers(1, 5))
    cu_domain = [int(x) for x in rng.integers(0, nar_max, size=num_cus)]
    for d in range(nar_max):
        cu_domain[d] = d                                          # every domain has a CU
    cu_rank = [int(x) for x in rng.integers(0, 4, size=num_cus)]
    cu_stack = [int(x) for x in rng.integers(0, num_stacks, size=num_cus)]
    num_chunks = int(rng.integers(1, 40))
    chunk_bytes = [int(x) for x in rng.integers(1, 9, size=num_chunks) * 512]
    num_tbs = int(rng.integers(0, 60))
    tb_gpu = [int(x) for x in rng.integers(0, 3, size=num_tbs)]
    tb_chunks = [[int(c) for c in rng.integers(0, num_chunks, size=int(rng.integers(0, 5)))] for _ in range(num_tbs)]
    r_cu = int(rng.integers(1, 12)) * 1024
    r_stack = int(rng.integers(1, 30)) * 1024
    run_both(tb_gpu, tb_chunks, chunk_bytes, cu_domain, cu_rank, cu_stack, num_stacks, r_cu, r_stack, nar_max)


def test_oneshot_workload_groups_are_tiles_dealt_round_robin():
    """The closed form the launch code relies on: for the one-shot's regular workload the N items of a
    tile form one group and tile t lands in domain t mod nar_max."""
    n, tiles, nar_max, cus_per_dom = 8, 10, 2, 4
    tb_chunks, chunk_bytes = [], [4096] * (2 * n * tiles)
    for t in range(tiles):
        for d in range(n):
            tb_chunks.append([r * tiles + t for r in range(n)] + [(n + d) * tiles + t])
    cu_domain = [c // cus_per_dom for c in range(nar_max * cus_per_dom)]
    budget = 9 * 4096 * n * 2                                     # two groups per CU
    mc, _, td, tg = run_both([0] * len(tb_chunks), tb_chunks, chunk_bytes, cu_domain, [0] * len(cu_domain),
                             [0] * len(cu_domain), 1, budget, 1 << 40, nar_max)
    for t in range(tiles):
        items = range(t * n, (t + 1) * n)
        assert {tg[i] for i in items} == {t}
        assert {td[i] for i in items} == {t % nar_max}
        assert len({mc[i] for i in items}) == 1                   # a group stays on one compute unit


def test_malformed_input_is_rejected():
    ok = dict(tb_gpu=[0], tb_chunks=[[0]], chunk_bytes=[64], cu_domain=[0], cu_rank=[0], cu_stack=[0], num_stacks=1,
              r_max_cu=1, r_max_stack=1, nar_max=1)
    assert nb.nuna_plan_placement(**ok)[0] == [0]
    for key, val in (("tb_chunks", [[5]]), ("cu_domain", [3]), ("cu_stack", [2]), ("nar_max", 0), ("tb_gpu", [-1])):
        bad = dict(ok)
        bad[key] = val
        assert nb.nuna_plan_placement(check=False, **bad) == nb.NUNA_ERR_INVALID_ARG
    two = dict(ok, cu_domain=[0], nar_max=2)                      # a domain without any CU
    assert nb.nuna_plan_placement(check=False, **two) == nb.NUNA_ERR_INVALID_ARG


# ---- the per-SM work lists the library plans for its own one-shot ---------------------------------------

def fake_topology(num_sms, split=True, seed=0):
    rng = np.random.Generator(np.random.PCG64(seed))
    t = nb.NunaTopology()
    t.num_sms = num_sms
    t.sms_reported = num_sms
    t.verdict = nb.NUNA_TOPO_NONUNIFORM if split else nb.NUNA_TOPO_UNIFORM
    t.num_domains = 2 if split else 1
    for s in range(num_sms):
        t.sm_reported[s] = 1
        t.sm_domain[s] = (s // 6) % 2 if split else 0
        t.sm_lat_hit[s] = 270.0 + float(rng.integers(0, 3000)) / 100.0
    return t


@pytest.mark.parametrize("num_sms,nranks,ntiles,split", [
    (148, 8, 16, True), (148, 8, 128, True), (148, 8, 1000, True), (148, 2, 300, True),
    (148, 8, 128, False), (20, 5, 77, True), (7, 16, 40, True), (148, 8, 1, True), (148, 8, 0, True)])
def test_closed_form_lists_equal_the_general_planner(num_sms, nranks, ntiles, split):
    topo = fake_topology(num_sms, split, seed=ntiles)
    a = nb.debug_plan_oneshot(topo, num_sms, nranks, ntiles, 512, generic=True)
    b = nb.debug_plan_oneshot(topo, num_sms, nranks, ntiles, 512, generic=False)
    assert a == b
    assert sorted(t for lst in a for t in lst) == list(range(ntiles))        # every tile exactly once


def test_small_workload_goes_to_the_nearest_sms_one_group_each():
    num_sms, ntiles = 148, 16
    topo = fake_topology(num_sms, True, seed=3)
    lists = nb.debug_plan_oneshot(topo, num_sms, 8, ntiles, 512, generic=True)
    used = [s for s in range(num_sms) if lists[s]]
    assert len(used) == ntiles and all(len(lists[s]) == 1 for s in used)
    for d in (0, 1):
        dom_sms = sorted((s for s in range(num_sms) if topo.sm_domain[s] == d), key=lambda s: (topo.sm_lat_hit[s], s))
        chosen = [s for s in used if topo.sm_domain[s] == d]
        assert sorted(chosen) == sorted(dom_sms[:ntiles // 2])               # the 8 lowest-latency SMs of each domain
        assert all(lists[s][0] % 2 == d for s in chosen)                     # tile t -> domain t mod 2


def test_lists_agree_with_the_python_oracle():
    num_sms, nranks, ntiles, tile_bytes = 12, 4, 30, 1024
    topo = fake_topology(num_sms, True, seed=9)
    lists = nb.debug_plan_oneshot(topo, num_sms, nranks, ntiles, tile_bytes, generic=True)
    # the same workload through the oracle
    W, cb = [], {}
    for t in range(ntiles):
        for d in range(nranks):
            cs = [(("src", r, t), "b", 0) for r in range(nranks)] + [(("dst", d, t), "b", 0)]
            W.append((0, (t, d), cs))
            for c in cs:
                cb[c] = tile_bytes
    doms = [[], []]
    for s in sorted(range(num_sms), key=lambda s: (topo.sm_lat_hit[s], s)):
        doms[topo.sm_domain[s]].append(s)
    smallest = min(len(doms[0]), len(doms[1]))
    budget = -(-(-(-ntiles // 2)) // smallest)
    otopo = {"domain_cus": doms, "cu_stacks": {s: [0] for s in range(num_sms)}}
    M, _, _ = nap.nuna_aware_placement(otopo, budget * nranks * (nranks + 1) * tile_bytes, 1 << 60, 2, W, cb)
    want = [[] for _ in range(num_sms)]
    for t in range(ntiles):
        assert len({M[(0, (t, d))] for d in range(nranks)}) == 1
        want[M[(0, (t, 0))]].append(t)
    assert lists == want


def test_no_probe_means_one_domain_in_sm_order():
    lists = nb.debug_plan_oneshot(None, 10, 8, 25, 512, generic=True)
    assert lists == [[0, 1, 2], [3, 4, 5], [6, 7, 8], [9, 10, 11], [12, 13, 14], [15, 16, 17], [18, 19, 20], [21, 22, 23], [24], []]


@pytest.mark.parametrize("domains", [1, 2, 4, 8, 16])
@pytest.mark.parametrize("split", [True, False])
def test_more_domains_than_probed_are_latency_quantiles(domains, split):
    """NUNA_OPT_DOMAINS (the paper's sweep over the number of routing domains, Section 6.5): each probed
    domain is cut into equal latency quantiles; group t goes to domain t mod D; closed form = general planner."""
    num_sms, nranks, ntiles = 148, 8, 592
    topo = fake_topology(num_sms, split, seed=11)
    a = nb.debug_plan_oneshot(topo, num_sms, nranks, ntiles, 512, generic=True, domains=domains)
    b = nb.debug_plan_oneshot(topo, num_sms, nranks, ntiles, 512, generic=False, domains=domains)
    assert a == b
    assert sorted(t for lst in a for t in lst) == list(range(ntiles))        # every tile exactly once
    base = 2 if (split and domains != 1) else 1
    D = max(base, domains // base * base) if domains > base else base
    # an SM serves tiles of exactly one residue class mod D, and every class is served
    classes = set()
    for lst in a:
        if lst:
            assert len({t % D for t in lst}) == 1
            classes.add(lst[0] % D)
    assert classes == set(range(D))
    # quantiles: inside a probed domain, the SMs of a faster class are never slower than those of a slower class
    if D > base:
        sub = D // base
        for bdom in range(base):
            by_class = {}
            for s, lst in enumerate(a):
                if lst and (topo.sm_domain[s] if base == 2 else 0) == bdom:
                    by_class.setdefault(lst[0] % D, []).append(topo.sm_lat_hit[s])
            keys = sorted(by_class)
            assert len(keys) == sub
            for lo, hi in zip(keys, keys[1:]):
                assert max(by_class[lo]) <= min(by_class[hi])
