"""Multi-GPU plumbing: candidates are independent, so a batch shards by candidate range with no
data-path collective.  Each rank evaluates its own range on its own GPU (one process per GPU);
the only communication is the max-over-ranks of the measured time (and whatever reduction a
search driver adds on the K makespans afterwards)."""
import torch
import torch.distributed as dist


def shard_range(num_candidates: int, world_size: int, rank: int):
    """Contiguous candidate range [first, first + count) of `rank`; sizes differ by at most one."""
    base, extra = divmod(int(num_candidates), int(world_size))
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def weak_scaling_first(candidates_per_rank: int, rank: int) -> int:
    """Weak scaling: every rank draws its own `candidates_per_rank` candidates; index of the first."""
    return int(rank) * int(candidates_per_rank)


def max_over_ranks(value: float, device=None) -> float:
    """MAX all-reduce of one number (the timing convention: the slowest rank decides)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
