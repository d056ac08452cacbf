"""Assignment of independent sequences (images) to ranks.

Images are independent (the paper decodes batch size 1; Sec. 5.1), all state is per sequence and
every random number is a function of the *global* sequence id, so the path shards by sequence with
no collective on the data path: each rank holds a full replica of the weights, runs a contiguous
block of sequences and passes the id of its first one as `seq_base`.  Results are identical
whatever the number of ranks.  The only communication is a host-side gather of token ids.
"""
from __future__ import annotations


def shard_sequences(n_sequences: int, world_size: int, rank: int):
    """Contiguous block partition: returns (first global sequence id, count) of `rank`."""
    if world_size < 1 or not 0 <= rank < world_size or n_sequences < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_sequences, world_size)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)


def gather_token_lists(local, group=None):
    """Host-side gather of this rank's per-sequence token lists into global sequence order
    (torch.distributed must be initialised; any backend)."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    parts = [None] * world
    dist.all_gather_object(parts, list(local), group=group)
    return [seq for part in parts for seq in part]


def max_over_ranks(value: float, device=None, group=None) -> float:
    """Slowest rank's time: the figure a multi-GPU run reports."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())
