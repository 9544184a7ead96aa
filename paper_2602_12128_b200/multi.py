"""Host-side logic of the multi-GPU modes.

Replicas (the benchmark): one process per GPU, each running the whole operator on its own seeded batch.  Heads and
batches are independent in every equation of the operator, so the data path has no collective; the only exchange is the
maximum over ranks of the measured device time.

Sequence sharding (optional): the N tokens of every head are split over the ranks.  The state of Theorem 4.2 is a sum
over tokens, so each pass needs one all-reduce (sum) of the fp32 state between its key half and its query half
(`sharded_forward`, `sharded_backward`: the library's half-pass entry points with `all_reduce_sum` in between; the
library itself never communicates).  With the causal mask (Section 4.4) a rank's tokens see the tokens of the lower
ranks only: instead of the sum, every rank needs the state of everything before its shard - an exclusive prefix over
the ranks (`exclusive_prefix_state`) - which it hands to its causal pass as the carried-in state of Eq. "seq.updates"
(`sharded_causal_forward`; forward only).

Works on any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests)."""
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


def shard_bounds(n_tokens: int, world: int, rank: int):
    """[first, last) token of a rank's contiguous share of a sequence: shares differ by at most one token."""
    base, extra = divmod(n_tokens, world)
    first = rank * base + min(rank, extra)
    return first, first + base + (1 if rank < extra else 0)


def all_reduce_sum(t, dist=None):
    """Sum of a tensor over the ranks, in place (a no-op for one process)."""
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t


def sharded_forward(op, Q, K, V, O, dist=None, stream=None):
    """Forward of one rank's shard of the tokens: key half, sum of the state over the ranks, query half.  `op` is a
    binding.Hla created with the shard's own N."""
    from . import binding
    binding.hla_forward_keys(op.ctx, K, V, op.workspace, stream)
    all_reduce_sum(op.state_region(), dist)
    binding.hla_forward_queries(op.ctx, Q, O, op.workspace, stream)
    return O


def sharded_backward(op, Q, K, V, O, dO, dQ, dK, dV, dist=None, stream=None):
    """Backward of one rank's shard: query half, sum of the gradient state over the ranks, key half."""
    from . import binding
    binding.hla_backward_queries(op.ctx, Q, K, V, O, dO, dQ, dK, dV, op.workspace, stream)
    all_reduce_sum(op.state_region(gradient=True), dist)
    binding.hla_backward_keys(op.ctx, Q, K, V, O, dO, dQ, dK, dV, op.workspace, stream)
    return dQ, dK, dV


def exclusive_prefix_state(local, dist=None):
    """Sum of `local` over the ranks below this one, added in rank order (zeros on rank 0): the state of all tokens
    before this rank's shard when `local` is the state of the shard."""
    out = torch.zeros_like(local)
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return out
    parts = [torch.empty_like(local) for _ in range(dist.get_world_size())]
    dist.all_gather(parts, local.contiguous())
    for r in range(dist.get_rank()):
        out += parts[r]
    return out


def sharded_causal_forward(op_causal, op_plain, Q, K, V, O, dist=None, stream=None):
    """Causal forward of one rank's shard of the tokens.  `op_plain` (causal=False) and `op_causal` (causal=True) are
    binding.Hla objects for the shard's own N with the same feature maps.  The key half of the unmasked operator gives
    the state of the shard, the exclusive prefix over the ranks is the state of the tokens before it, and the causal
    pass starts from that state (hla_set_carry)."""
    from . import binding
    binding.hla_forward_keys(op_plain.ctx, K, V, op_plain.workspace, stream)
    before = exclusive_prefix_state(op_plain.state_region(), dist)
    op_causal.state_region().copy_(before)
    op_causal.set_carry(True)
    op_causal.forward(Q, K, V, O, stream)
    return O
