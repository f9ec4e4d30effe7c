"""Stand-in for the benchmark's timed step, used by the CPU test of the rank launcher: every rank joins a gloo
group from the environment torch.distributed.run gives it, "measures" a step time that depends on its rank, and
rank 0 prints the whole-job line that bench.job_throughput forms from the slowest rank."""
import json
import os
import sys

import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402

if __name__ == "__main__":
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    ms_local = 10.0 + 15.0 * rank
    ms_per_step, units_per_s = bench.job_throughput(ms_local, steps=5, units_per_step_per_rank=1000.0, world=world, dist=dist)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"n_gpus": world, "ms_per_step": ms_per_step, "value": units_per_s, "argv": sys.argv[1:]}))
    dist.destroy_process_group()
