"""Batch sharding for multi-GPU runs: images are independent, so every rank takes a contiguous
slice of the batch with a replica of the packed weights; there is no collective on the data path.
Only timing is reduced (maximum over ranks)."""


def shard_range(n_items, rank, world):
    """[begin, end) of the items rank `rank` of `world` processes owns; sizes differ by at most 1."""
    if world <= 0 or not (0 <= rank < world) or n_items < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_items, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]
