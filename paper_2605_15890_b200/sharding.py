"""Host-side helpers for running the path on several GPUs.

Every bucket of coordinates is independent (its own norm, random draws keyed by message
position), so a gradient is sharded by contiguous, pack-block-aligned coordinate ranges,
one per rank, with no exchange on the data path. Only timings are reduced across ranks.
"""
BLOCK = 512


def coordinate_range(d_total, rank, world, align=BLOCK):
    """[start, stop) of rank's shard: whole pack blocks, as equal as possible, the last
    shard taking the ragged tail. Shards of ranks 0..world-1 tile [0, d_total). With buckets of
    more than 512 coordinates pass the bucket size as `align`: a shard starts at a bucket."""
    if not (0 <= rank < world) or d_total < 0:
        raise ValueError("bad rank / size")
    nblk = (d_total + align - 1) // align
    base, extra = divmod(nblk, world)
    b0 = rank * base + min(rank, extra)
    b1 = b0 + base + (1 if rank < extra else 0)
    return min(b0 * align, d_total), min(b1 * align, d_total)


def first_block(d_total, rank, world, align=BLOCK):
    """Pack-block index of the shard's first coordinate (for agc_plan_set_first_block)."""
    return coordinate_range(d_total, rank, world, align)[0] // BLOCK


def max_over_ranks(values, device=None):
    """Element-wise maximum over all ranks of a list of floats (a step time is the slowest
    rank's). Without an initialised process group the values come back unchanged."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]
