"""Host-side logic for running the library on several GPUs of one node.

The five programs are independent problems, so the multi-GPU form is N replicas, one process per
GPU, each with its own seeded inputs: no data-path collective exists.  What the ranks share is
host plumbing only, and that plumbing lives here so that it can be exercised with the ``gloo``
backend on CPUs: the rank/world/local-rank environment, the replica's input seed, the barrier
that brackets a timed region, the max-over-ranks reduction of a device time, and the whole-job
aggregate.
"""
from __future__ import annotations

import os
from dataclasses import dataclass


@dataclass(frozen=True)
class RankInfo:
    rank: int
    world: int
    local: int

    @property
    def is_root(self) -> bool:
        return self.rank == 0


def rank_info(env=None) -> RankInfo:
    """Rank, world size and local rank as the launcher exports them (single process if absent)."""
    env = os.environ if env is None else env
    rank = int(env.get("RANK", "0"))
    world = int(env.get("WORLD_SIZE", "1"))
    local = int(env.get("LOCAL_RANK", str(rank)))
    if world < 1 or not 0 <= rank < world:
        raise ValueError(f"inconsistent launcher environment: RANK={rank} WORLD_SIZE={world}")
    return RankInfo(rank, world, local)


def replica_seed(info: RankInfo, base_seed: int = 0) -> int:
    """Every replica draws its own inputs: seed = base + rank."""
    return int(base_seed) + info.rank


def init_process_group(info: RankInfo, backend: str, device=None):
    """Join the job's process group (no-op for a single process).  Returns True if one was made."""
    if info.world == 1:
        return False
    import torch.distributed as dist

    kwargs = {}
    if device is not None and backend == "nccl":
        kwargs["device_id"] = device
    dist.init_process_group(backend, rank=info.rank, world_size=info.world, **kwargs)
    return True


def barrier(info: RankInfo, device_sync=None):
    """Device sync, job-wide barrier, device sync: brackets a timed region on both sides."""
    if device_sync is not None:
        device_sync()
    if info.world > 1:
        import torch.distributed as dist

        dist.barrier()
    if device_sync is not None:
        device_sync()


def max_over_ranks(info: RankInfo, value: float, device="cpu") -> float:
    """The slowest rank's time: a job of replicas is as fast as its slowest member."""
    if info.world == 1:
        return float(value)
    import torch
    import torch.distributed as dist

    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rate(info: RankInfo, units_per_rank_per_step: float, ms_per_step: float) -> float:
    """Whole-job rate in units per second: every rank processed the same number of units in the
    (max-over-ranks) step time."""
    return info.world * units_per_rank_per_step / (ms_per_step * 1e-3)


def destroy_process_group(info: RankInfo):
    if info.world > 1:
        import torch.distributed as dist

        if dist.is_initialized():
            dist.destroy_process_group()
