"""Multi-process host logic of the replica launch (world size 2, gloo, CPU): every rank draws its own
batch, the timed region takes the slowest rank's time, and throughput is the whole-job aggregate."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_16154_b200 import dist_util, synth


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.WORKLOADS["C0"]
    rb = synth.make_rollouts(w, dist_util.replica_seed(w.seed, rank))
    dist.barrier()
    slowest = dist_util.max_over_ranks(10.0 + 5.0 * rank, "cpu")          # rank 1 is the slow one
    out[rank] = (int(rb["tok"].astype(np.int64).sum()), slowest)
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_take_the_slowest_time_and_distinct_batches():
    mgr = mp.Manager()
    out = mgr.dict()
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0][1] == out[1][1] == 15.0                                # max over ranks on every rank
    assert out[0][0] != out[1][0]                                        # different rollouts per replica
    assert dist_util.aggregate_throughput(24, 10, 15.0, 2) == 2 * 24 * 10 / 0.015
    assert dist_util.max_over_ranks(3.5, "cpu") == 3.5                   # no process group: identity
