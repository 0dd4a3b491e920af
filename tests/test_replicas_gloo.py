"""The N > 1 path of the benchmark (independent replicas: barrier + slowest rank's time), run as
two gloo ranks on CPU."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2608_00867_b200.replicas import Replicas
    rep = Replicas(backend="gloo")
    assert rep.world == world and rep.rank == rank and not rep.cuda
    rep.barrier()
    slow = rep.max_over_ranks(10.0 + 5.0 * rank)           # rank 1 is the slow one
    total = rep.sum_over_ranks(1000.0)                     # every replica does 1000 steps
    rep.barrier()
    out.put((rank, slow, total))
    rep.close()


def test_two_replicas_agree_on_the_slowest_time_and_total_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results == [(0, 15.0, 2000.0), (1, 15.0, 2000.0)]


def test_single_process_needs_no_process_group(monkeypatch):
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        monkeypatch.delenv(k, raising=False)
    from paper_2608_00867_b200.replicas import Replicas
    rep = Replicas(backend="gloo")
    assert rep.world == 1 and rep.max_over_ranks(3.5) == 3.5 and rep.sum_over_ranks(2.0) == 2.0
    rep.barrier()
    rep.close()
