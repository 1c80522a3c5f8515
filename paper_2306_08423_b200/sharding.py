"""Host-side helpers for running on several GPUs (one process per GPU).

Candidates are independent, so the path shards without any exchange on the data path: either
every rank runs its own search (weak scaling, what ``bench.py --gpus N`` does), or the ranks
split one candidate range into contiguous slices and merge their 16-byte (time, index) winners
at the end.  The merge is a host-side gather of two integers per rank, not a data-path
collective; it works on any ``torch.distributed`` backend (``gloo`` on CPU in the tests).
"""
from __future__ import annotations


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the search a rank runs in weak-scaling mode."""
    return base_seed + rank


def shard_range(n: int, rank: int, world: int):
    """Contiguous slice [first, first + count) of n candidates for this rank; slices differ in
    size by at most one and cover [0, n) exactly once."""
    if world < 1 or not 0 <= rank < world or n < 0:
        raise ValueError("bad shard arguments")
    base, extra = divmod(n, world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def merge_argmin(best_index: int, best_batch_ns: int, group=None):
    """Global (index, batch_ns) winner from every rank's local winner: smallest time, ties to
    the smallest index.  A rank with an empty slice passes index -1."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    mine = torch.tensor([best_batch_ns, best_index], dtype=torch.int64)
    gathered = [torch.zeros(2, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(gathered, mine, group=group)
    pairs = [(int(g[0]), int(g[1])) for g in gathered if int(g[1]) >= 0]
    if not pairs:
        return -1, 0
    t, i = min(pairs)
    return i, t


def gather_topk_lists(local_times, local_indices, group=None):
    """Every rank's (times, indices) top-k list, concatenated in rank order on every rank.  The
    lists are torch tensors of equal length on all ranks (CPU tensors under gloo, device tensors
    under NCCL); a rank with fewer than k candidates pads with (INT64_MAX, INT64_MAX) pairs.
    The k smallest of the result (smallest time, ties to the smallest index) are the global
    top-k: every global winner is a winner of its own rank's slice."""
    import torch
    import torch.distributed as dist
    if not dist.is_available() or not dist.is_initialized():
        return local_times, local_indices
    world = dist.get_world_size(group)
    pair = torch.stack([local_times, local_indices])                 # [2, k]
    out = [torch.empty_like(pair) for _ in range(world)]
    dist.all_gather(out, pair, group=group)
    both = torch.cat(out, dim=1)
    return both[0].contiguous(), both[1].contiguous()


def max_over_ranks(value: float, device=None, group=None) -> float:
    """Largest value over the ranks (used for device-timed durations)."""
    import torch
    import torch.distributed as dist
    if not dist.is_available() or not dist.is_initialized():
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())
