"""The topology probe on a real device.  Latency values are hardware facts (no parity claim);
pinned here: coverage, self-consistency, repeatability and that buffers come back untouched."""
import numpy as np
import pytest
import torch

from paper_2608_00867_b200 import binding as nb

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def probed():
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    bufs = [torch.randint(-30000, 30000, (1 << 18,), generator=gen, device="cuda", dtype=torch.int16) for _ in range(16)]
    before = [b.clone() for b in bufs]
    t1 = nb.nuna_probe_topology(bufs)
    t2 = nb.nuna_probe_topology(bufs)
    torch.cuda.synchronize()
    return bufs, before, t1, t2


def test_buffers_are_restored_bit_for_bit(probed):
    bufs, before, _, _ = probed
    for a, b in zip(bufs, before):
        assert torch.equal(a, b)


def test_every_sm_reports_and_walks_check_out(probed):
    _, _, t, _ = probed
    props = torch.cuda.get_device_properties(0)
    assert t.num_sms == props.multi_processor_count
    assert t.sms_reported == t.num_sms and all(t.sm_reported[s] for s in range(t.num_sms))
    assert t.self_pointer_mismatches == 0
    assert t.chain_walk_ok == 1 and t.chain_steps > 0 and t.chain_nodes >= 4096
    assert t.num_bufs == 16 and t.num_lines > 500


def test_latencies_are_physical(probed):
    _, _, t, _ = probed
    hit = np.array(t.sm_lat_hit[:t.num_sms])
    miss = np.array(t.sm_lat_miss[:t.num_sms])
    assert (hit > 50).all() and (hit < 2000).all()
    assert (miss > hit).all()                                # DRAM is further away than L2 from every SM
    assert 0.0 <= t.nonuniformity < 1.0


def test_solo_read_rate_of_every_sm(probed):
    _, _, t1, t2 = probed
    a, b = np.array(t1.sm_read_gbs[:t1.num_sms]), np.array(t2.sm_read_gbs[:t2.num_sms])
    assert (a > 10.0).all() and (a < 5000.0).all()              # every SM measured, physically plausible GB/s
    assert np.median(np.abs(a - b) / a) < 0.10                  # the second probe agrees
    assert a.max() / a.min() < 3.0                              # no SM is starved of bandwidth


def test_repeatable_within_noise(probed):
    _, _, t1, t2 = probed
    a, b = np.array(t1.sm_lat_hit[:t1.num_sms]), np.array(t2.sm_lat_hit[:t2.num_sms])
    assert np.median(np.abs(a - b)) <= max(3.0 * t1.noise, 3.0)
    assert t1.verdict == t2.verdict
    if t1.verdict == nb.NUNA_TOPO_NONUNIFORM:
        assert np.array_equal(np.array(t1.sm_domain[:t1.num_sms]), np.array(t2.sm_domain[:t2.num_sms]))


def test_verdict_is_consistent_with_its_own_numbers(probed):
    _, _, t, _ = probed
    if t.verdict == nb.NUNA_TOPO_NONUNIFORM:
        assert t.num_domains == 2 and t.domain_gap > 3 * t.noise and t.far_lat > t.near_lat
        doms = np.array(t.sm_domain[:t.num_sms])
        assert 0 < doms.sum() < t.num_sms and doms[0] == 0
    else:
        assert t.num_domains == 1 and not any(t.sm_domain[:t.num_sms])


def test_granularity_scan_is_self_consistent_and_repeatable(probed):
    """The consecutive-line scan of buffer 0: runs add up to the window, the histogram and the longest run
    agree with the per-line homes, the block shares are shares, and a second probe maps the lines the same way."""
    _, _, t1, t2 = probed
    if t1.verdict != nb.NUNA_TOPO_NONUNIFORM:
        assert t1.scan_lines == 0 and all(s == -1.0 for s in t1.scan_level_spread)
        return
    W = t1.scan_lines
    assert W == min(nb.NUNA_SCAN_LINES, (1 << 19) // 128)       # buffer 0 is 512 KiB
    homes = np.array(t1.scan_home[:W])
    assert set(np.unique(homes)) <= {0, 1}
    # run lengths recomputed from the homes
    edges = np.flatnonzero(np.diff(homes)) + 1
    runs = np.diff(np.concatenate([[0], edges, [W]]))
    assert runs.sum() == W and runs.max() == t1.scan_longest_run
    hist = np.bincount(np.floor(np.log2(runs)).astype(int), minlength=nb.NUNA_SCAN_RUN_BINS)     # power-of-two bins
    assert np.array_equal(hist, np.array(t1.scan_run_hist[:]))
    # block shares: 4 KiB and 64 KiB blocks fit in a 512 KiB buffer, 2 MiB blocks do not
    for g, expect_blocks in ((0, 8), (1, 8), (2, 0)):
        shares = [t1.scan_level_share[g][b] for b in range(nb.NUNA_SCAN_BLOCKS)]
        got = [s for s in shares if s >= 0.0]
        assert len(got) == expect_blocks and all(0.0 <= s <= 1.0 for s in got)
        assert (t1.scan_level_spread[g] >= 0.0) == (expect_blocks >= 2)
    # repeatable: the second probe puts (nearly) every line of the window in the same domain
    assert t2.scan_lines == W
    agree = (homes == np.array(t2.scan_home[:W])).mean()
    assert agree >= 0.95, agree


def test_probe_refuses_a_capturing_stream():
    buf = torch.zeros(4096, dtype=torch.int16, device="cuda")
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            st = nb.nuna_probe_topology([buf], stream=s, check=False)
    assert st == nb.NUNA_ERR_CAPTURING
