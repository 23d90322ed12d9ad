"""Helper of test_bench_host: one rank of a job started by the command line that bench.py builds for
`--gpus N` without torchrun.  Joins a gloo group from the environment torchrun sets, aggregates
like bench.py does and lets rank 0 print the result."""
import json
import os
import sys

import torch
import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402


def main():
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")

    def reduce(op):
        def f(v):
            t = torch.tensor([v], dtype=torch.float64)
            dist.all_reduce(t, op=op)
            return float(t.item())
        return f

    ms, work = bench.aggregate_over_ranks(10.0 + rank, 7.0, world, reduce(dist.ReduceOp.MAX), reduce(dist.ReduceOp.SUM))
    dist.barrier()
    if rank == 0:
        print(json.dumps({"ms": ms, "work": work, "world": world, "argv": sys.argv[1:]}))
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
