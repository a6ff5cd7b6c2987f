"""Row sharding for multi-GPU runs.

Positions are independent, so a batch is split into contiguous row ranges, one per rank, with
no exchange on the data path.  Each rank passes `row_offset` = the global id of its first row:
the random streams are keyed by global row, so the sharded run reproduces the single-GPU run
bit for bit.  The only cross-rank quantities of the objective (the number of valid positions
and the summed loss) are two scalars the caller all-reduces.  Block verification shards by
sequence in the same way (`seq_offset`)."""
from __future__ import annotations


def shard_rows(n_rows: int, rank: int, world_size: int):
    """Contiguous, balanced partition of range(n_rows): returns (first_row, n_local)."""
    if not (0 <= rank < world_size):
        raise ValueError("rank outside [0, world_size)")
    base, extra = divmod(n_rows, world_size)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def global_grad_scale(n_valid_local: int, group=None) -> float:
    """1 / N_valid over all ranks (the normaliser of the objective); all-reduces one integer."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([n_valid_local], dtype=torch.int64)
    if dist.is_available() and dist.is_initialized():
        if dist.get_backend(group) == "nccl":
            t = t.cuda()
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    n = int(t.item())
    return 1.0 / n if n > 0 else 0.0
