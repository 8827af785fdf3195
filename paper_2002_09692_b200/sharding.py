"""Host-side helpers for running the gossip round on several GPUs, one process per GPU.

The round acts column by column (the mask depends on the column only, the average mixes
rows), so a model can be cut into column shards, one per GPU, and a round needs NO exchange
between the shards: every rank derives the same matching from the same (seed, t, bandwidth)
and the same mask from the global column index (saps_set_column_offset).  The only
cross-rank step is optional: placing the per-shard wire buffers in one globally contiguous
buffer needs the exclusive scan of one count per rank.
"""
from __future__ import annotations

TILE_COLS = 2048          # column tile of the kernels; shard boundaries are multiples of it
MAX_COLUMNS = 1 << 32


def column_shard(n_total: int, world: int, rank: int, align: int = TILE_COLS):
    """Strong scaling: cut n_total columns into `world` contiguous shards whose boundaries are
    multiples of `align`.  Returns (begin, end); trailing ranks may get an empty shard."""
    if not (0 <= rank < world) or n_total < 1:
        raise ValueError("bad rank/world/n_total")
    tiles = (n_total + align - 1) // align
    per, extra = divmod(tiles, world)
    first_tile = rank * per + min(rank, extra)
    ntile = per + (1 if rank < extra else 0)
    begin = min(first_tile * align, n_total)
    end = min((first_tile + ntile) * align, n_total)
    return begin, end


def weak_shard(n_per_rank: int, world: int, rank: int):
    """Weak scaling: every rank holds n_per_rank columns of a model with world * n_per_rank
    columns.  Returns (column offset, columns)."""
    if not (0 <= rank < world):
        raise ValueError("bad rank/world")
    if world * n_per_rank > MAX_COLUMNS:
        raise ValueError("global column index must stay below 2^32")
    return rank * n_per_rank, n_per_rank


def exclusive_offsets(counts):
    """[c0, c1, ...] -> ([0, c0, c0+c1, ...], total)."""
    out, run = [], 0
    for c in counts:
        out.append(run)
        run += int(c)
    return out, run


def global_pack_offset(local_count: int, group=None):
    """Offset of this rank's packed entries in the globally contiguous wire buffer, and the
    global count: one all-gather of a single integer per rank."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    dev = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    mine = torch.tensor([int(local_count)], dtype=torch.int64, device=dev)
    every = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(every, mine, group=group)
    offsets, total = exclusive_offsets([int(t.item()) for t in every])
    return offsets[dist.get_rank(group)], total


def max_over_ranks(value: float, group=None) -> float:
    """A multi-GPU time is the slowest rank's."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    dev = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())
