"""NUNA-aware placement (Algorithm 1) restated in Python -- TEST INFRASTRUCTURE ONLY.

Follows Section 4.2 in the paper's order and notation:

* ``W`` is the workload, a list of ``(gpu, tb, C_tb)``; ``C_tb`` is the list of
  chunks thread block ``tb`` touches, each chunk a tuple
  ``(chunk_id, buffer_type, gpu_id)``; ``chunk_bytes`` gives each chunk's size.
* ``logical_allocation`` (Section 4.2.1) walks the thread blocks in order.  A
  block none of whose chunks is assigned yet opens a new logical group;
  otherwise block and still-unassigned chunks join the existing group that
  already holds most of its chunks.  Groups are returned sorted by decreasing
  size.
* The main loop (Algorithm 1) hands the groups to the ``nar_max`` domains in
  round-robin order and calls ``physical_placement`` (Section 4.2.2) for every
  thread block of the group: the first CU of that domain whose remaining budget
  ``R[cu]`` covers the block's chunk bytes ``cs``, and an HBM stack, preferring
  that CU's nearest stack.  Budgets are decremented after every decision.

Readings where the text leaves a choice (all deterministic):

* The domain counter is used, then advanced, so the first group lands in
  domain 0 as in the worked figure (the listing increments first).
* "Shares the most chunks": ties go to the group created first.  A chunk that is
  already in a group stays there (first come, first served).
* "Size" of a group is the total bytes of its chunks; the sort is stable.
* If no CU of the domain has budget left, the CU of that domain with the most
  budget remaining takes the block (the paper's fall-back to default dispatch);
  likewise for stacks.
* A chunk that already has a stack keeps it (page-level first come, first
  served); only still-unplaced chunks of the block get the chosen stack.
"""
from __future__ import annotations

from typing import Dict, Hashable, List, Sequence, Tuple

Chunk = Tuple[Hashable, Hashable, int]          # (chunk_id, buffer_type, gpu_id)
Work = Tuple[int, Hashable, Sequence[Chunk]]    # (gpu, tb, C_tb)


def logical_allocation(W: Sequence[Work], chunk_bytes: Dict[Chunk, int]) -> List[dict]:
    groups: List[dict] = []                     # {"tbs": [(gpu, tb, C_tb)], "chunks": [chunk, ...]}
    owner: Dict[Chunk, int] = {}                # chunk -> index of its group (creation order)
    for gpu, tb, C_tb in W:
        shared: Dict[int, int] = {}
        for c in C_tb:
            if c in owner:
                shared[owner[c]] = shared.get(owner[c], 0) + 1
        if not shared:
            g = len(groups)
            groups.append({"tbs": [], "chunks": []})
        else:
            most = max(shared.values())
            g = min(i for i, k in shared.items() if k == most)
        groups[g]["tbs"].append((gpu, tb, tuple(C_tb)))
        for c in C_tb:
            if c not in owner:
                owner[c] = g
                groups[g]["chunks"].append(c)
    for grp in groups:
        grp["size"] = sum(chunk_bytes[c] for c in grp["chunks"])
    order = sorted(range(len(groups)), key=lambda i: -groups[i]["size"])   # stable
    return [groups[i] for i in order]


def physical_placement(nar: int, cs: int, R_cu: Dict, R_stack: Dict, topology: dict, gpu: int):
    """First CU of domain ``nar`` with budget for ``cs`` bytes, and a stack near it."""
    cus = topology["domain_cus"][nar]
    cu = next((c for c in cus if R_cu[(gpu, c)] >= cs), None)
    if cu is None:
        cu = max(cus, key=lambda c: (R_cu[(gpu, c)], -cus.index(c)))
    prefs = topology["cu_stacks"][cu]            # stacks in order of distance from this CU
    stack = next((s for s in prefs if R_stack[(gpu, s)] >= cs), None)
    if stack is None:
        stack = max(prefs, key=lambda s: (R_stack[(gpu, s)], -prefs.index(s)))
    return cu, stack


def nuna_aware_placement(topology: dict, R_max_cu: int, R_max_stack: int, nar_max: int,
                         W: Sequence[Work], chunk_bytes: Dict[Chunk, int]):
    """Algorithm 1.  Returns ``(M_compute, M_memory, tb_domain)``.

    ``topology`` = {"domain_cus": [[cu, ...] per domain, nearest first],
                    "cu_stacks": {cu: [stack, ...] nearest first}}.
    ``M_compute[(gpu, tb)] = cu``; ``M_memory[chunk] = stack``;
    ``tb_domain[(gpu, tb)]`` = the domain its group was dealt to.
    """
    gpus = sorted({gpu for gpu, _, _ in W})
    all_cus = [c for dom in topology["domain_cus"] for c in dom]
    all_stacks = sorted({s for prefs in topology["cu_stacks"].values() for s in prefs})
    R_cu = {(g, c): R_max_cu for g in gpus for c in all_cus}
    R_stack = {(g, s): R_max_stack for g in gpus for s in all_stacks}
    M_compute: Dict = {}
    M_memory: Dict = {}
    tb_domain: Dict = {}
    nar = 0
    L = logical_allocation(W, chunk_bytes)
    for L_i in L:
        for gpu, tb_j, C_j in L_i["tbs"]:
            cs = sum(chunk_bytes[c] for c in C_j)
            cu, stack = physical_placement(nar, cs, R_cu, R_stack, topology, gpu)
            R_cu[(gpu, cu)] -= cs
            R_stack[(gpu, stack)] -= cs
            M_compute[(gpu, tb_j)] = cu
            tb_domain[(gpu, tb_j)] = nar
            for c in C_j:
                M_memory.setdefault(c, stack)
        nar = (nar + 1) % nar_max
    return M_compute, M_memory, tb_domain


def round_robin_placement(W: Sequence[Work], cus: Sequence[int]):
    """The locality-unaware baseline (Section 5.3): thread block i goes to CU i mod |CUs|."""
    return {(gpu, tb): cus[i % len(cus)] for i, (gpu, tb, _) in enumerate(W)}
