"""Host-side helpers for running independent replicas on several GPUs.

Weight tensors (layers) are independent units of the optimizer step, so ranks
share no data: each rank owns its own tensors and the only cross-rank steps are
a barrier and a max-reduction of the measured time.
"""
from __future__ import annotations

from typing import List


def tensor_ids_for_rank(rank: int, world: int, tensors_per_rank: int) -> List[int]:
    """Global tensor ids owned by a rank (contiguous blocks, no overlap)."""
    if not (0 <= rank < world) or tensors_per_rank < 1:
        raise ValueError("bad rank / world / tensors_per_rank")
    return list(range(rank * tensors_per_rank, (rank + 1) * tensors_per_rank))


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Max of a per-rank scalar over the process group (identity without a group)."""
    if dist is None or not dist.is_initialized():
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    if t.device.type == "cuda":
        t = t.float()
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, world: int, max_seconds: float) -> float:
    """Whole-job throughput: all ranks' units over the slowest rank's time."""
    return units_per_rank * world / max_seconds
