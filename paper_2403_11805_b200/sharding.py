"""How the path spreads over several GPUs: contexts are independent (Sec. 3.1), so each rank owns whole contexts and
nothing of the data path crosses ranks.  Only the timing is reduced (maximum over ranks)."""
import torch


def contexts_of_rank(n_contexts: int, rank: int, world: int):
    """Round-robin ownership: context c belongs to rank c % world."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    return list(range(rank, n_contexts, world))


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()
