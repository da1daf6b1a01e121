"""Batch-sharded replicas: the only multi-GPU form of this path.

The merge and the merged network's forward have no exchange step between images, so N GPUs run N
independent replicas, each on its own batch (weak scaling).  Nothing here touches the data path:
these helpers cover the rendezvous, the per-rank input seed, and the timing reduction (the job's
step time is the slowest rank's).
"""
import os
from typing import Tuple


def env_rank_world() -> Tuple[int, int, int]:
    """(rank, world size, local rank) from the launcher's environment; (0, 1, 0) when run alone."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def replica_seed(base_seed: int, rank: int) -> int:
    """Seed of a rank's batch: replicas draw different images from the same generator."""
    return int(base_seed) + int(rank)


def init_group(backend: str, world: int, device=None):
    """Join the process group (no-op for one process). Returns True when a group was created."""
    if world <= 1:
        return False
    import torch.distributed as dist
    if device is not None:
        dist.init_process_group(backend, device_id=device)
    else:
        dist.init_process_group(backend)
    return True


def max_over_ranks(times, world: int):
    """In-place MAX all-reduce of a tensor of per-rank times (device or CPU); identity for one rank."""
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    return times


def job_throughput(units_per_rank: int, world: int, seconds: float) -> float:
    """Whole-job units per second: every rank processed `units_per_rank` in the slowest rank's time."""
    return world * units_per_rank / seconds
