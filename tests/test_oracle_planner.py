"""Pins for the Python restatement of the paper's placement algorithm (Algorithm 1)."""
import os

import pytest

from oracle import nap_planner as nap

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "alloc_figure_example.txt")


def load_figure_example():
    W, expect, nar_max, cb = [], {}, None, None
    for line in open(GOLDEN):
        line = line.split("#")[0].split()
        if not line:
            continue
        if line[0] == "nar_max":
            nar_max = int(line[1])
        elif line[0] == "chunk_bytes":
            cb = int(line[1])
        elif line[0] == "tb":
            chunks = [(c.split("@")[0], "buffer", int(c.split("@")[1])) for c in line[3:]]
            W.append((int(line[1]), line[2], chunks))
        elif line[0] == "expect":
            expect[(int(line[1]), line[2])] = int(line[3])
    chunk_bytes = {c: cb for _, _, cs in W for c in cs}
    return W, chunk_bytes, nar_max, expect


def flat_topology(ndomains, cus_per_domain, nstacks=2):
    doms = [[d * cus_per_domain + i for i in range(cus_per_domain)] for d in range(ndomains)]
    stacks = {c: [(c // cus_per_domain) % nstacks] + [s for s in range(nstacks) if s != (c // cus_per_domain) % nstacks]
              for dom in doms for c in dom}
    return {"domain_cus": doms, "cu_stacks": stacks}


def test_figure_example_groups_and_domains():
    W, chunk_bytes, nar_max, expect = load_figure_example()
    L = nap.logical_allocation(W, chunk_bytes)
    assert len(L) == 4                                   # four disjoint singleton groups
    assert all(len(g["tbs"]) == 1 and len(g["chunks"]) == 2 for g in L)
    seen = [c for g in L for c in g["chunks"]]
    assert len(seen) == len(set(seen)) == 8
    topo = flat_topology(nar_max, 2)
    M_compute, M_memory, dom = nap.nuna_aware_placement(topo, 1 << 20, 1 << 20, nar_max, W, chunk_bytes)
    assert dom == expect                                 # dealt to domains 0,1,2,3; w uses domain 0
    for key, d in dom.items():
        assert M_compute[key] in topo["domain_cus"][d]
    # both copies of a chunk pair sit on the stack nearest the chosen CU
    for (gpu, tb, cs) in W:
        cu = M_compute[(gpu, tb)]
        assert all(M_memory[c] == topo["cu_stacks"][cu][0] for c in cs)


def test_blocks_sharing_chunks_join_one_group():
    # one-shot allreduce shape: N readers of the same source tile
    n, tiles = 4, 6
    W, cb = [], {}
    for t in range(tiles):
        for d in range(n):
            cs = [("src", r, t) for r in range(n)] + [("dst", d, t)]
            W.append((0, (t, d), [(c, "buf", 0) for c in cs]))
            for c in cs:
                cb[(c, "buf", 0)] = 4096
    L = nap.logical_allocation(W, cb)
    assert len(L) == tiles
    for g in L:
        assert len({tb[0] for _, tb, _ in g["tbs"]}) == 1 and len(g["tbs"]) == n
    _, _, dom = nap.nuna_aware_placement(flat_topology(2, 8), 10 ** 9, 10 ** 9, 2, W, cb)
    for t in range(tiles):
        assert {dom[(0, (t, d))] for d in range(n)} == {t % 2}


def test_most_shared_group_wins_and_ties_go_to_the_oldest():
    cb = {(c, "b", 0): 100 for c in "abcdef"}
    ch = lambda s: [(c, "b", 0) for c in s]
    W = [(0, "t0", ch("ab")), (0, "t1", ch("cd")), (0, "t2", ch("acd")), (0, "t3", ch("bc")), (0, "t4", ch("ef"))]
    L = nap.logical_allocation(W, cb)
    where = {tb: i for i, g in enumerate(L) for _, tb, _ in g["tbs"]}
    assert where["t2"] == where["t1"]        # shares 2 chunks with t1's group, 1 with t0's
    assert where["t3"] == where["t0"]        # one each: tie -> group created first
    assert where["t4"] not in (where["t0"], where["t1"])
    # chunk ownership is first come, first served: every chunk in exactly one group
    allc = [c for g in L for c in g["chunks"]]
    assert sorted(allc) == sorted(cb)


def test_groups_sorted_by_decreasing_bytes_stable():
    cb = {("a", "b", 0): 10, ("b", "b", 0): 30, ("c", "b", 0): 30, ("d", "b", 0): 5}
    W = [(0, i, [c]) for i, c in enumerate(cb)]
    L = nap.logical_allocation(W, cb)
    assert [g["size"] for g in L] == [30, 30, 10, 5]
    assert [g["tbs"][0][1] for g in L] == [1, 2, 0, 3]


def test_budget_first_fit_then_least_loaded():
    topo = flat_topology(1, 3, nstacks=1)
    cb = {(i, "b", 0): 60 for i in range(7)}
    W = [(0, i, [(i, "b", 0)]) for i in range(7)]
    M, _, _ = nap.nuna_aware_placement(topo, 100, 10 ** 6, 1, W, cb)
    # budget 100 holds one 60-byte block per CU; the 4th.. fall back to the least-loaded CU
    assert [M[(0, i)] for i in range(3)] == [0, 1, 2]
    counts = [sum(1 for v in M.values() if v == c) for c in range(3)]
    assert sorted(counts) == [2, 2, 3]
    assert len(M) == 7


def test_every_block_placed_once_and_deterministic():
    W, cb = [], {}
    for i in range(50):
        cs = [((i * 7 + k) % 23, "b", 0) for k in range(1 + i % 3)]
        W.append((0, i, cs))
        for c in cs:
            cb[c] = 256 * (1 + c[0] % 4)
    topo = flat_topology(3, 5)
    a = nap.nuna_aware_placement(topo, 4096, 1 << 20, 3, W, cb)
    b = nap.nuna_aware_placement(topo, 4096, 1 << 20, 3, W, cb)
    assert a == b
    assert set(a[0]) == {(0, i) for i in range(50)}
    assert set(a[1]) == set(cb)


def test_one_domain_and_round_robin_baseline():
    W = [(0, i, [(i, "b", 0)]) for i in range(10)]
    assert nap.round_robin_placement(W, [5, 6, 7]) == {(0, i): [5, 6, 7][i % 3] for i in range(10)}
