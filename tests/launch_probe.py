"""Started by tests/test_launch.py through the benchmark's own launch command: joins the process group on CPU
(gloo) and prints what rank 0 of the benchmark would report as its GPU count."""
import json

from paper_2605_16154_b200 import dist_util, launch

if __name__ == "__main__":
    import torch.distributed as dist
    rank, world, local = launch.init_process_group("gloo")
    slowest = dist_util.max_over_ranks(float(rank), "cpu")
    if rank == 0:
        print(json.dumps({"n_gpus": world, "slowest": slowest}))
    if world > 1:
        dist.destroy_process_group()
