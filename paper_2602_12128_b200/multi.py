"""Host-side logic of the multi-GPU benchmark: one process per GPU, each running the
whole operator on its own seeded batch.  Heads and batches are independent in every
equation of the operator, so the data path has no collective; the only exchange is the
maximum over ranks of the measured device time.  Works on any torch.distributed backend
(NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

import torch


def rank_seed(base: int, rank: int) -> int:
    """Seed of a rank's synthetic batch: distinct per rank, reproducible."""
    return base + 7919 * rank


def max_over_ranks(ms: float, dist=None, device="cpu") -> float:
    """The slowest rank's time; `dist` is torch.distributed (initialised) or None for one process."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, ms: float) -> float:
    """Units per second of the whole job: every rank processed `units_per_rank` in `ms` (the slowest rank's time)."""
    return world * units_per_rank / (ms * 1e-3)
