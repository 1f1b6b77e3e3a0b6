"""Process-group plumbing of the multi-GPU benchmark: batch shards, no collective on the data path.

Every rank serves its own batch on its own GPU; ranks only meet to (a) start and stop the timed
region together and (b) agree on the slowest rank's time.  Works with NCCL (GPU runs) and gloo
(CPU tests)."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, local_rank: int = 0):
    """Joins the process group described by MASTER_ADDR / MASTER_PORT / RANK / WORLD_SIZE."""
    if dist.is_initialized():
        return
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    else:
        dist.init_process_group(backend)


def barrier(sync_cuda: bool = True):
    if dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
    if sync_cuda and torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """The slowest rank's value (a time), identical on every rank afterwards."""
    if not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: int, ms_slowest: float) -> float:
    """Whole-job units per second: every rank processed `units_per_rank` in `ms_slowest`."""
    world = dist.get_world_size() if dist.is_initialized() else 1
    return world * units_per_rank / (ms_slowest * 1e-3)


def shard_seed(rank: int) -> int:
    """Distinct input streams per rank (each rank's batch is its own shard of the job)."""
    return 1000 * rank
