"""Host-side helpers for running the path on several GPUs of one node.

The operations shard with no exchange step: every output row (GEMM), image (conv) or problem (batched) is
independent, so each rank computes its own slice with the same kernels and nothing crosses NVLink on the data
path.  ``torch.distributed`` is used only to agree on a time (max over ranks) or, when a caller wants the
int8 result whole on every rank, to gather the output slices after the epilogue.
"""
from __future__ import annotations

from typing import Tuple


def row_shard(total: int, world: int, rank: int, align: int = 128) -> Tuple[int, int]:
    """Contiguous slice [start, start + count) of `total` rows for `rank`: slices are multiples of `align`
    (the tile height) except the last non-empty one, cover every row once, and differ by at most one block."""
    assert world >= 1 and 0 <= rank < world and total >= 0 and align >= 1
    blocks = (total + align - 1) // align
    base, extra = divmod(blocks, world)
    my_blocks = base + (1 if rank < extra else 0)
    first_block = rank * base + min(rank, extra)
    start = min(first_block * align, total)
    end = min((first_block + my_blocks) * align, total)
    return start, end - start


def batch_shard(batch: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous slice of `batch` independent problems (pairs are kept together for the paired kernel)."""
    return row_shard(batch, world, rank, align=2)


def rank_seed(seed: int, rank: int) -> int:
    """Seed of the independent draw that `rank` benchmarks (rank 0 keeps the named configuration's seed)."""
    return seed + 1000 * rank


def max_over_ranks(value_ms: float, device=None) -> float:
    """Max of a per-rank duration over the default process group (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value_ms)
    t = torch.tensor([value_ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, max_ms: float) -> float:
    """Units per second of the whole job: every rank processed `units_per_rank` in at most `max_ms`."""
    return world * units_per_rank / (max_ms * 1e-3)


def gather_rows(local_rows, total: int, world: int, align: int = 128):
    """All-gather int8 output slices produced under row_shard into the whole [total, N] result on every rank."""
    import torch
    import torch.distributed as dist
    n = local_rows.shape[1]
    counts = [row_shard(total, world, r, align)[1] for r in range(world)]
    pad = max(counts)
    buf = torch.zeros((pad, n), dtype=local_rows.dtype, device=local_rows.device)
    buf[: local_rows.shape[0]] = local_rows
    out = [torch.empty_like(buf) for _ in range(world)]
    dist.all_gather(out, buf)
    return torch.cat([o[:c] for o, c in zip(out, counts)], dim=0)
