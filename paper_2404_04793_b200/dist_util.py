"""Multi-GPU runs: starting one rank per GPU and the process-group plumbing between them.
The hot path shards by independent sequence batches (one batch per rank, no data-path
collective); the only exchanges are a barrier around the timed region and a max / sum
reduction of each rank's device time and token count."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init(backend: str):
    rank, local_rank, world_size = world()
    if world_size > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend, rank=rank, world_size=world_size)
    return rank, local_rank, world_size


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def exchange_importance(ctx, device="cpu"):
    """One batch sharded over the ranks (each holds some of its sequences): sums the per-layer
    cosine sums and token counts of Section 3's layer average over all ranks (one all-reduce of
    2 * n_layer numbers) and puts the totals back into this rank's context, so that
    allocate_budgets gives every rank the batch's budgets.  Call after the last layer_importance."""
    sums, counts = ctx.get_importance_state()
    if dist.is_initialized():
        t = torch.tensor(list(sums) + [float(c) for c in counts], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        v = t.cpu().tolist()
        n = len(sums)
        sums, counts = v[:n], [int(round(x)) for x in v[n:]]
    ctx.set_importance_state(sums, counts)
    return sums, counts


def aggregate_throughput(units_this_rank: float, ms_this_rank: float, device="cpu"):
    """Whole-job throughput: units processed by all ranks / the slowest rank's time.
    Returns (units_per_second, max_ms)."""
    total = sum_over_ranks(units_this_rank, device)
    ms = max_over_ranks(ms_this_rank, device)
    return total / (ms * 1e-3), ms


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()


def _free_port() -> int:
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def spawn_ranks(n: int, argv, capture_rank0: bool = False, timeout: float | None = None, extra_env=None):
    """Starts `argv` (a command list) n times as ranks 0..n-1 of one node, one process per GPU:
    RANK = LOCAL_RANK = rank, WORLD_SIZE = n, rendezvous on 127.0.0.1 at a free port.  The path
    shards by independent sequence batches, so the ranks only meet in the barrier and the max /
    sum of their device times; rank 0 reports.  Waits for all ranks; if one fails the others are
    terminated (by their own PIDs).  Returns the first non-zero exit code (0 if none), and with
    capture_rank0 also rank 0's standard output."""
    import subprocess
    import time

    port = _free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ)
        env.update(RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        if extra_env:
            env.update(extra_env)
        out = subprocess.PIPE if (capture_rank0 and r == 0) else None
        procs.append(subprocess.Popen(list(argv), env=env, stdout=out, text=True if out else None))
    rc, t0, text = 0, time.time(), ""
    live = set(range(n))
    while live:
        for r in sorted(live):
            code = procs[r].poll()
            if code is not None:
                live.discard(r)
                if code != 0 and rc == 0:
                    rc = code
        if (rc != 0 or (timeout is not None and time.time() - t0 > timeout)) and live:
            for r in live:
                procs[r].terminate()
            for r in live:
                try:
                    procs[r].wait(timeout=10)
                except subprocess.TimeoutExpired:
                    procs[r].kill()
            rc = rc or 124
            break
        if capture_rank0 and 0 in live:
            # drain rank 0's pipe so that it cannot fill up; communicate() waits for its exit
            try:
                text, _ = procs[0].communicate(timeout=0.2)
            except subprocess.TimeoutExpired:
                pass
        else:
            time.sleep(0.05)
    if capture_rank0 and not text and procs[0].stdout is not None:
        try:
            text = procs[0].stdout.read() or ""
        except ValueError:
            pass
    return (rc, text) if capture_rank0 else rc
