"""Data-parallel plumbing: the encoder layer never mixes batch entries, so N GPUs run N
independent replicas on disjoint slices of the global batch (weights replicated, no collective
on the data path).  Only the bookkeeping lives here: which sequences a rank owns, and the
max-over-ranks reduction of the device timings."""
from __future__ import annotations


def shard_range(global_batch: int, world: int, rank: int) -> tuple[int, int]:
    """[first, last) sequence indices of `rank`: contiguous blocks, remainders to the low ranks."""
    if world < 1 or not 0 <= rank < world or global_batch < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(global_batch, world)
    first = rank * base + min(rank, extra)
    return first, first + base + (1 if rank < extra else 0)


def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks of the default process group
    (identity when torch.distributed is not initialised)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]
