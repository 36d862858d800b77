"""Starting one process per GPU on a single node, and the run-length defaults of the benchmark.

`python bench.py --gpus N` with N > 1 and no launcher environment re-executes itself through
`torch.distributed.run` with N processes (rendezvous on 127.0.0.1); under a launcher (RANK / WORLD_SIZE set)
it runs as the rank it was given.  No torch import here: the relaunch decision is taken before anything heavy
is loaded.
"""
from __future__ import annotations

import os
import socket
import sys
from typing import List, Mapping, Optional, Sequence, Tuple


def needs_relaunch(gpus: int, env: Mapping[str, str]) -> bool:
    """True when N > 1 ranks were asked for and this process was not started by a launcher."""
    return gpus > 1 and "WORLD_SIZE" not in env and "RANK" not in env


def free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return int(s.getsockname()[1])


def torchrun_command(n: int, script: str, argv: Sequence[str], port: Optional[int] = None) -> List[str]:
    """Command line that runs `script argv...` as n ranks of one node, one process per GPU."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={int(n)}",
            "--master-addr", "127.0.0.1", "--master-port", str(port if port is not None else free_port()),
            script, *argv]


def rank_world_local(env: Mapping[str, str] = os.environ) -> Tuple[int, int, int]:
    return int(env.get("RANK", "0")), int(env.get("WORLD_SIZE", "1")), int(env.get("LOCAL_RANK", "0"))


def init_process_group(backend: str, device=None):
    """Joins the launcher's process group when there is more than one rank; returns (rank, world, local_rank)."""
    rank, world, local = rank_world_local()
    if world > 1:
        import torch.distributed as dist
        kw = {"device_id": device} if device is not None else {}
        dist.init_process_group(backend, **kw)
    return rank, world, local


def default_steps(workload: str, impl: str = "cuda") -> int:
    """Timed steps when --steps is not given: 10 steps over a resident batch; the ragged workload runs its
    50 consecutive iterations; the CPU arm times 3 bounded samples."""
    if impl == "reference":
        return 3
    return 50 if workload == "C4" else 10
