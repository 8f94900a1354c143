"""Multi-rank plumbing on CPU (gloo, world_size 2): the launcher that `bench.py --gpus N` uses to
start its ranks, and the barrier / sum / max helpers that turn per-rank device times into
whole-job throughput."""
import json
import sys
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


class _FakeCtx:
    """Stands in for a context of one rank: holds the per-layer cosine sums and token counts that
    rank accumulated over its share of the batch."""

    def __init__(self, sums, counts):
        self.sums, self.counts = list(sums), list(counts)

    def get_importance_state(self):
        return list(self.sums), list(self.counts)

    def set_importance_state(self, sums, counts):
        self.sums, self.counts = list(sums), list(counts)


def _exchange_worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2404_04793_b200 import dist_util
    dist_util.init("gloo")
    # rank r holds 3 + r sequences of 100 tokens; three layers
    ctx = _FakeCtx([10.0 + rank, 20.5 * (rank + 1), 0.125], [(3 + rank) * 100] * 3)
    dist_util.exchange_importance(ctx)
    dist_util.barrier()
    dist_util.shutdown()
    q.put((rank, ctx.sums, ctx.counts))


def test_importance_exchange_of_a_batch_sharded_over_two_ranks():
    """The one exchange of the path: the per-layer cosine sums and token counts of a batch whose
    sequences are spread over the ranks are summed over all ranks, and every rank ends up with
    the same totals (then the allocator, deterministic, gives every rank the same budgets)."""
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_exchange_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, sums, counts in res:
        assert sums == [21.0, 61.5, 0.25]
        assert counts == [700, 700, 700]


def test_single_process_helpers_need_no_group():
    from paper_2404_04793_b200 import dist_util
    assert dist_util.max_over_ranks(3.5) == 3.5
    assert dist_util.aggregate_throughput(100, 20.0) == (5000.0, 20.0)


STUB = os.path.join(os.path.dirname(os.path.abspath(__file__)), "rank_stub_job.py")


def test_launcher_starts_two_ranks_and_rank0_reports():
    """The launcher bench.py calls for --gpus 2, driving a stub job over gloo: both ranks run,
    meet in the barrier and the reductions, and rank 0 prints the whole-job line."""
    from paper_2404_04793_b200 import dist_util
    rc, text = dist_util.spawn_ranks(2, [sys.executable, STUB], capture_rank0=True, timeout=240)
    assert rc == 0, text
    line = json.loads(text.strip().splitlines()[-1])
    assert line["n_gpus"] == 2
    assert line["ms_per_step"] == 50.0                       # the slowest rank sets the time
    assert line["value"] == pytest.approx(2048 / 0.050)      # tokens of both ranks


def test_launcher_reports_a_failed_rank_and_stops_the_rest():
    from paper_2404_04793_b200 import dist_util
    rc = dist_util.spawn_ranks(2, [sys.executable, STUB, "--fail-rank", "1"], timeout=240,
                               extra_env={"TORCH_GLOO_TIMEOUT": "20"})
    assert rc != 0


def test_bench_spawns_ranks_itself_when_asked_for_several_gpus(monkeypatch):
    """`python bench.py --gpus 2` without RANK in the environment must go through the launcher
    with its own command line; under a launcher (RANK set) it must not spawn again."""
    import importlib
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    bench = importlib.import_module("bench")
    calls = []
    from paper_2404_04793_b200 import dist_util
    monkeypatch.setattr(dist_util, "spawn_ranks", lambda n, argv, **kw: calls.append((n, list(argv))) or 0)
    monkeypatch.delenv("RANK", raising=False)
    assert bench.maybe_spawn(["--gpus", "2", "--steps", "1"], 2) == 0
    assert calls and calls[0][0] == 2 and calls[0][1][-4:] == ["--gpus", "2", "--steps", "1"]
    monkeypatch.setenv("RANK", "0")
    assert bench.maybe_spawn(["--gpus", "2"], 2) is None and len(calls) == 1
    assert bench.maybe_spawn(["--gpus", "1"], 1) is None
