"""Chain sharding across ranks: chains are independent and the generator is keyed by the global
chain id, so a rank needs only its id range. No collective touches the data path; ranks exchange
only timings and, if wanted, the final samples."""
from __future__ import annotations


def chain_range(rank: int, world: int, total_chains: int):
    """Contiguous [begin, end) of global chain ids for `rank` when `total_chains` are split as
    evenly as possible (the first total % world ranks get one more)."""
    if not (0 <= rank < world) or total_chains < 0:
        raise ValueError("bad rank/world/total")
    base, extra = divmod(total_chains, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def weak_offset(rank: int, chains_per_rank: int) -> int:
    """Global id of a rank's first chain when every rank runs the same number of chains."""
    return rank * chains_per_rank


def max_over_ranks(values, dist=None, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return [float(v) for v in values]
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def gather_rows(local, dist=None):
    """All ranks' [n_i, d] arrays stacked in rank order (numpy in, numpy out; off the timed path)."""
    import numpy as np
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return np.asarray(local)
    out = [None] * dist.get_world_size()
    dist.all_gather_object(out, np.asarray(local))
    return np.concatenate(out, axis=0)
