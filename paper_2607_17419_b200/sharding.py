"""Host-side helpers for running the forward on several GPUs of one node.

(batch, head) pairs are independent units of the KATA forward, so a job is split over ranks by giving each
rank a contiguous range of the B*H pairs; no collective is needed in the data path.  Timing is reduced with
a MAX over ranks.
"""
from __future__ import annotations


def pair_range(n_pairs: int, rank: int, world: int) -> tuple[int, int]:
    """[begin, end) of the (batch*head) pairs owned by `rank`: balanced, contiguous, covering, disjoint."""
    if not (0 <= rank < world) or n_pairs < 0:
        raise ValueError("bad rank/world/n_pairs")
    base, extra = divmod(n_pairs, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(values, device=None):
    """Element-wise MAX of a list of floats over all ranks of the default process group (identity if none)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_rate(units_per_rank: float, world: int, ms_max: float) -> float:
    """Units per second of the whole job when every rank processed `units_per_rank` in `ms_max` ms."""
    return world * units_per_rank / (ms_max * 1e-3)
