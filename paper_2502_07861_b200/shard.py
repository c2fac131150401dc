"""Multi-GPU layout of the BalanceKV path: one process per GPU, streams sharded, no exchange.

Every (sequence, layer, KV head) stream is compressed and decoded on its own (Algorithm 3 runs
per stream; the estimator of Theorem 3.3 sums over that stream's sets only), so ranks never
exchange cache data.  A rank owns a contiguous range of sequences; the only collective is the
max-over-ranks of a timing or the gather of outputs that a caller may want on one rank.
"""
from __future__ import annotations


def shard_range(n_items: int, world: int, rank: int) -> range:
    """Contiguous balanced split of n_items over `world` ranks (earlier ranks take the extra one)."""
    if world < 1 or not 0 <= rank < world or n_items < 0:
        raise ValueError("bad shard arguments")
    base, extra = divmod(n_items, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def owner_of(item: int, n_items: int, world: int) -> int:
    """Rank whose shard_range holds `item`."""
    if not 0 <= item < n_items:
        raise ValueError("item out of range")
    base, extra = divmod(n_items, world)
    cut = extra * (base + 1)
    return item // (base + 1) if item < cut else extra + (item - cut) // base


def walk_seed(base_seed: int, first_sequence: int) -> int:
    """Context seed of a rank: the library keys the coin of sequence s by seed + s, so a rank that
    owns global sequences [first, ...) as its local 0.. uses base_seed + first."""
    return base_seed + first_sequence


def max_over_ranks(value: float, device=None) -> float:
    """Max of a scalar over the default process group (identity without one)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
