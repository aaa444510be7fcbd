"""Host-side helpers for running the path on several GPUs.

Every bucket of coordinates is independent (its own norm, random draws keyed by message
position), so a gradient is sharded by contiguous, pack-block-aligned coordinate ranges,
one per rank, with no exchange on the data path. The one exception is the global norm
(one l2 norm per worker over the whole vector): between its two passes the shards exchange
n floats (`global_norm_sums`). Timings are reduced across ranks as well.
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


def power_of_two_range(d_total, rank, world):
    """[start, stop) of rank's shard when every shard but the last covers the same power-of-two
    number of pack blocks (the smallest that covers the vector with `world` shards): the split
    for which the sharded global-norm encoder equals the unsplit one bit for bit. Trailing
    shards may be empty for short vectors."""
    if not (0 <= rank < world) or d_total < 0:
        raise ValueError("bad rank / size")
    nblk = (d_total + BLOCK - 1) // BLOCK
    per = 1
    while per * world < nblk:
        per *= 2
    return min(rank * per * BLOCK, d_total), min((rank + 1) * per * BLOCK, d_total)


def global_norm_sums(local_sums, combine):
    """The exchange between the two passes of the sharded global-norm encoder: every rank
    contributes its n sums of squares (a float32 tensor on the CPU or on its GPU), all ranks
    get the ranges' sums in rank order and combine them with `combine` (the library's
    agc_combine_norm_sums): the same tree on every rank, so all ranks hold identical norms.
    Returns a float32 numpy array [n]."""
    import numpy as np
    import torch
    import torch.distributed as dist
    t = local_sums if isinstance(local_sums, torch.Tensor) else torch.from_numpy(np.asarray(local_sums, np.float32))
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return combine(t.detach().cpu().numpy()[None, :])
    parts = [torch.empty_like(t) for _ in range(dist.get_world_size())]
    dist.all_gather(parts, t.contiguous())
    return combine(np.stack([x.detach().cpu().numpy() for x in parts]))


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
