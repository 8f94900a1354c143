"""A stand-in for a benchmark rank, used by tests/test_dist_gloo.py: takes part in the same
barrier and reductions over gloo that a GPU rank runs over NCCL and lets rank 0 print one JSON
line.  Rank r pretends to have generated 1024 tokens in (40 + 10 r) ms."""
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from paper_2404_04793_b200 import dist_util  # noqa: E402


def main():
    rank, local_rank, world = dist_util.init("gloo")
    assert local_rank == rank
    if "--fail-rank" in sys.argv and rank == int(sys.argv[sys.argv.index("--fail-rank") + 1]):
        sys.exit(3)                                   # a rank that dies before the first barrier
    dist_util.barrier()
    tok_s, ms = dist_util.aggregate_throughput(1024, 40.0 + 10.0 * rank)
    dist_util.barrier()
    if rank == 0:
        print(json.dumps({"n_gpus": world, "value": tok_s, "ms_per_step": ms}), flush=True)
    dist_util.shutdown()


if __name__ == "__main__":
    main()
