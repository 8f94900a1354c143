"""Multi-rank plumbing on CPU (gloo, world_size 2): the barrier / sum / max helpers that
bench.py uses to turn per-rank device times into whole-job throughput."""
import os
import socket

import pytest
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2404_04793_b200 import dist_util
    r, lr, w = dist_util.init("gloo")
    assert (r, lr, w) == (rank, rank, world)
    dist_util.barrier()
    # rank 0 processed 1024 tokens in 40 ms, rank 1 1024 tokens in 50 ms
    tok_s, ms = dist_util.aggregate_throughput(1024, 40.0 + 10.0 * rank)
    mx = dist_util.max_over_ranks(float(rank))
    dist_util.barrier()
    dist_util.shutdown()
    q.put((rank, tok_s, ms, mx))


def test_aggregate_throughput_two_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, tok_s, ms, mx in res:
        assert ms == 50.0                       # the slowest rank sets the time
        assert tok_s == pytest.approx(2048 / 0.050)
        assert mx == 1.0


def test_single_process_helpers_need_no_group():
    from paper_2404_04793_b200 import dist_util
    assert dist_util.max_over_ranks(3.5) == 3.5
    assert dist_util.aggregate_throughput(100, 20.0) == (5000.0, 20.0)
