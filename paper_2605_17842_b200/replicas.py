"""Host-side plumbing of the multi-GPU benchmark: independent replicas, one process per GPU.

The hot path does not shard (one GPU holds the model, the trace and the cache; there is no exchange step), so N GPUs
run N replicas of the same job.  What the ranks share is only the timing protocol: a barrier on both sides of the timed
region, the maximum of the per-rank device times, and a whole-job value = units processed by all ranks / that time.
Nothing here touches CUDA, so the same code runs over `gloo` on CPU in the tests and over `nccl` in bench.py.
"""
from __future__ import annotations

import os
from dataclasses import dataclass


@dataclass
class Ranks:
    rank: int
    world: int
    local: int

    @property
    def is_root(self) -> bool:
        return self.rank == 0


def ranks_from_env(env=None) -> Ranks:
    """RANK / WORLD_SIZE / LOCAL_RANK as set by torch.distributed.run (single process: 0 / 1 / 0)."""
    env = os.environ if env is None else env
    return Ranks(int(env.get("RANK", "0")), int(env.get("WORLD_SIZE", "1")), int(env.get("LOCAL_RANK", "0")))


def init(ranks: Ranks, backend: str, device=None):
    """Join the process group (rendezvous from MASTER_ADDR / MASTER_PORT); no-op for a single process."""
    if ranks.world <= 1:
        return
    import torch.distributed as dist
    kw = {"device_id": device} if device is not None else {}
    dist.init_process_group(backend, rank=ranks.rank, world_size=ranks.world, **kw)
    dist.barrier()


def barrier(ranks: Ranks):
    if ranks.world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(ranks: Ranks, value: float, device="cpu") -> float:
    """The slowest rank's figure: a multi-GPU time is the maximum of the per-rank device times."""
    if ranks.world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(ranks: Ranks, units_per_rank: float, ms: float) -> float:
    """Units per second of the whole job: every replica processes `units_per_rank` in `ms` (max over ranks)."""
    return ranks.world * units_per_rank * 1e3 / ms


def finish(ranks: Ranks):
    if ranks.world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
