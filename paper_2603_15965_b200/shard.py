"""Token-parallel sharding of the routed-LoRA path over ranks (one process per GPU).

Rows are independent in Eq. 2, so the path shards by token with the adapter stacks replicated and NO
collective on the data path: every rank routes, groups and applies its own tokens.  The only communication
is the benchmark's bookkeeping -- a barrier around the timed region and the maximum of the per-rank times.
These helpers hold that host-side logic so that it can be exercised with the gloo backend on CPU.
"""
from __future__ import annotations

from typing import List, Tuple


def token_range(n_tokens: int, rank: int, world: int) -> Tuple[int, int]:
    """[begin, end) of the tokens rank `rank` owns when one batch of n_tokens is split over `world` ranks
    (strong scaling): contiguous, disjoint, covering, sizes differing by at most one."""
    if not (0 <= rank < world) or n_tokens < 0:
        raise ValueError("bad rank / world / token count")
    base, extra = divmod(n_tokens, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def rank_batches(rank: int, world: int, n_sets: int) -> List[int]:
    """Indices of the activation batches rank `rank` draws under weak scaling (every rank processes full-size
    batches of its own): disjoint across ranks, n_sets per rank."""
    if not (0 <= rank < world) or n_sets < 1:
        raise ValueError("bad rank / world / n_sets")
    return [rank * n_sets + b for b in range(n_sets)]


def max_over_ranks(value: float, dist=None, device: str = "cpu") -> float:
    """Maximum of a per-rank scalar over the process group (the step time of a multi-GPU run)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput: every rank processed tokens_per_rank tokens per step of ms_per_step (max over ranks)."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)
