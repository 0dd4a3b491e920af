"""Host-side parts of the topology probe: chain construction and the domain / verdict logic."""
import numpy as np
import pytest

from paper_2608_00867_b200 import binding as nb
from paper_2608_00867_b200 import build as nbuild


@pytest.fixture(scope="module", autouse=True)
def built_library():
    nbuild.build()


@pytest.mark.parametrize("n,seed", [(2, 1), (3, 2), (64, 3), (4096, 4), (32768, 0x70726F6265)])
def test_chain_is_one_cycle_over_every_node(n, seed):
    nxt, _ = nb.debug_chain(n, seed, 0, 0)
    assert sorted(nxt.tolist()) == list(range(n))          # a permutation
    assert not np.any(nxt == np.arange(n))                 # no fixed point
    i, seen = 0, 0
    while True:
        i = int(nxt[i])
        seen += 1
        if i == 0:
            break
    assert seen == n                                       # one single cycle through all nodes


def test_chain_walk_matches_python_walk():
    nxt, end = nb.debug_chain(1000, 99, 17, 48)
    i = 17
    for _ in range(48):
        i = int(nxt[i])
    assert end == i
    nxt2, _ = nb.debug_chain(1000, 99, 0, 0)
    assert np.array_equal(nxt, nxt2)                       # deterministic in the seed


def synthetic(num_sms, nlines, gap, noise, seed, split=None):
    rng = np.random.Generator(np.random.PCG64(seed))
    dom = np.zeros(num_sms, int) if split is None else np.asarray(split)
    home = rng.integers(0, 2, size=nlines)
    base = 280.0 + rng.normal(0, 4.0, size=(num_sms, 1)) + rng.normal(0, 3.0, size=(1, nlines))
    far = (dom[:, None] != home[None, :]).astype(float)
    clean = base + gap * far
    return (clean + rng.normal(0, noise, clean.shape), clean + rng.normal(0, noise, clean.shape), dom, home)


def test_uniform_matrix_gives_uniform_verdict():
    a, b, _, _ = synthetic(148, 300, gap=0.0, noise=1.0, seed=1)
    t = nb.debug_analyse_topology(a, b)
    assert t.verdict == nb.NUNA_TOPO_UNIFORM and t.num_domains == 1
    assert all(d == 0 for d in t.sm_domain[:148])
    assert sum(t.hist_near[:]) == 148 * 300 and sum(t.hist_far[:]) == 0


def test_two_clusters_are_recovered_exactly():
    split = np.array([(s // 8) % 2 for s in range(148)])
    a, b, dom, home = synthetic(148, 400, gap=30.0, noise=1.0, seed=2, split=split)
    t = nb.debug_analyse_topology(a, b)
    assert t.verdict == nb.NUNA_TOPO_NONUNIFORM and t.num_domains == 2
    got = np.array(t.sm_domain[:148])
    assert np.array_equal(got, dom)                         # SM 0 is in domain 0 by construction
    assert np.array_equal(np.array(t.line_home[:400]), home)
    assert 27.0 < t.domain_gap < 33.0
    near, far = np.array(t.hist_near[:]), np.array(t.hist_far[:])
    assert near.sum() + far.sum() == 148 * 400 and near.sum() > 0 and far.sum() > 0
    centre = lambda h: (h * (nb.NUNA_HIST_FIRST + nb.NUNA_HIST_STEP * (np.arange(len(h)) + 0.5))).sum() / h.sum()
    assert 25.0 < centre(far) - centre(near) < 35.0          # the histograms show the same gap
    assert 0.5 < t.noise < 2.5
    assert t.far_lat > t.near_lat


def test_gap_hidden_in_noise_stays_uniform():
    split = np.array([s % 2 for s in range(64)])
    a, b, _, _ = synthetic(64, 200, gap=2.0, noise=6.0, seed=3, split=split)
    t = nb.debug_analyse_topology(a, b)
    assert t.verdict == nb.NUNA_TOPO_UNIFORM                # 2 cycles is below both 3 x noise and 3 % of 280


def test_small_but_clean_gap_below_three_percent_stays_uniform():
    split = np.array([s % 2 for s in range(64)])
    a, b, _, _ = synthetic(64, 200, gap=5.0, noise=0.2, seed=4, split=split)
    t = nb.debug_analyse_topology(a, b)
    assert t.verdict == nb.NUNA_TOPO_UNIFORM                # 5 < 0.03 * 280


def test_probe_argument_errors_need_no_gpu():
    topo = nb.NunaTopology()
    import ctypes
    L = nb.lib()
    sizes = (ctypes.c_size_t * 1)(4096)
    assert L.nuna_probe_topology(None, sizes, 1, ctypes.byref(topo), None) == nb.NUNA_ERR_INVALID_ARG
    assert L.nuna_probe_topology(nb.ptr_table([4096]), sizes, 0, ctypes.byref(topo), None) == nb.NUNA_ERR_INVALID_ARG
    assert L.nuna_probe_topology(nb.ptr_table([4096]), sizes, 1, None, None) == nb.NUNA_ERR_INVALID_ARG
    assert L.nuna_probe_topology(nb.ptr_table([4100]), sizes, 1, ctypes.byref(topo), None) == nb.NUNA_ERR_ALIGNMENT
    small = (ctypes.c_size_t * 1)(64)
    assert L.nuna_probe_topology(nb.ptr_table([4096]), small, 1, ctypes.byref(topo), None) == nb.NUNA_ERR_INVALID_ARG
