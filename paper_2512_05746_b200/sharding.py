"""Row sharding of the quantized-layer forward across GPUs (one process per GPU).

Every step of the path treats rows (tokens, pixels) independently and the weights are small, so a multi-GPU run
replicates the weights and gives each rank a contiguous range of rows (whole images for a convolution, so that no
window crosses a shard boundary).  Nothing is exchanged on the data path; the only collective is the reduction of
the step time over ranks that the benchmark reports.
"""
from __future__ import annotations


def shard_rows(rows: int, rank: int, world: int) -> tuple[int, int]:
    """(first row, row count) of `rank`: contiguous, sizes differ by at most one, the union is [0, rows)."""
    if world <= 0 or not (0 <= rank < world):
        raise ValueError("rank / world out of range")
    base, extra = divmod(int(rows), world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def shard_images(batch: int, rank: int, world: int) -> tuple[int, int]:
    """(first image, image count) of `rank` for an NHWC batch: images are never split."""
    return shard_rows(batch, rank, world)


def max_over_ranks(value: float, device=None) -> float:
    """Largest `value` over all ranks of the default process group (the value itself without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])
