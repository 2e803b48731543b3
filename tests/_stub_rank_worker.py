"""A stand-in for one rank of the benchmark, for the launcher test: joins a gloo process group
from the environment torchrun sets, sums the ranks' numbers as the benchmark's reductions do,
and lets rank 0 print one JSON line."""
import json
import os
import sys

import torch
import torch.distributed as dist


def main():
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    assert rank == int(os.environ["RANK"]) and world == int(os.environ["WORLD_SIZE"])
    t = torch.tensor([1.0, float(rank + 1)], dtype=torch.float64)
    units, slowest = t[0:1].clone(), t[1:2].clone()
    dist.all_reduce(units, op=dist.ReduceOp.SUM)
    dist.all_reduce(slowest, op=dist.ReduceOp.MAX)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"n_gpus": world, "units": float(units), "slowest": float(slowest), "argv": sys.argv[1:],
                          "parallelism": f"rows sharded x{world}, no collective"}), flush=True)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
