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


# ------------------------------------------------------------------------------------------------ sharded calls
# Each wrapper takes the WHOLE problem (every rank holds, or can view, the full operands), computes this rank's slice
# with one call into the library and returns it; with gather=True the int8 slices are all-gathered after the epilogue
# (a quarter of the bytes the int32 accumulators would be) so that every rank ends up with the whole result.
# `world`/`rank` default to the process group's; `kernel` is the library call (the binding's function by default): the
# CPU tests pass a host implementation with the same signature, so the slicing and gathering logic runs without a GPU.
def _world_rank(world, rank):
    import torch.distributed as dist
    if world is None or rank is None:
        if dist.is_available() and dist.is_initialized():
            return dist.get_world_size(), dist.get_rank()
        return 1, 0
    return int(world), int(rank)


def sharded_gemm_i8(A, B, bias, mult, shift, per_channel: int, relu: int, *, world=None, rank=None, gather=False, kernel=None,
                    out=None):
    """Rows of A and C are split across ranks (row_shard, 128-row blocks); B, bias, mult, shift are replicated.
    A: (M, K), B: (K, N) views as for ``binding.gemm_i8``.  Returns this rank's (count, N) int8 slice of C, or the
    whole (M, N) result with gather=True."""
    import torch
    from . import binding
    world, rank = _world_rank(world, rank)
    M, N = A.shape[0], B.shape[1]
    start, count = row_shard(M, world, rank)
    C = out if out is not None else torch.empty((count, N), dtype=torch.int8, device=A.device)
    if count:
        (kernel or binding.gemm_i8)(A[start:start + count], B, C, bias, mult, shift, per_channel, relu)
    return gather_rows(C, M, world) if gather and world > 1 else C


def sharded_conv2d_i8(x, w, bias, mult, shift, per_channel: int, relu: int, stride=(1, 1), pad=(0, 0), *, world=None, rank=None,
                      gather=False, kernel=None):
    """Images are split across ranks (whole images, one per block); the weights are replicated.  x: (N, H, W, C),
    w: (K, R, S, C).  Returns this rank's (count, P, Q, K) slice of y, or all N images with gather=True."""
    import torch
    from . import binding
    world, rank = _world_rank(world, rank)
    N, H, W, _ = x.shape
    K, R, S, _ = w.shape
    P = (H + 2 * pad[0] - R) // stride[0] + 1
    Q = (W + 2 * pad[1] - S) // stride[1] + 1
    start, count = row_shard(N, world, rank, align=1)
    y = torch.empty((count, P, Q, K), dtype=torch.int8, device=x.device)
    if count:
        (kernel or binding.conv2d_i8)(x[start:start + count], w, y, bias, mult, shift, per_channel, relu, stride, pad)
    if gather and world > 1:
        return gather_rows(y.reshape(count, P * Q * K), N, world, align=1).reshape(N, P, Q, K)
    return y


def sharded_batched_gemm_i8(A, B, bias, mult, shift, per_channel: int, relu: int, *, world=None, rank=None, gather=False,
                            kernel=None):
    """The batch is split across ranks (pairs of problems stay together).  A: (batch, M, K), B: (batch, K, N),
    bias: (batch, N), (N,) or None.  Returns this rank's (count, M, N) slice of C, or the whole batch with gather=True."""
    import torch
    from . import binding
    world, rank = _world_rank(world, rank)
    batch, M, _ = A.shape
    N = B.shape[2]
    start, count = batch_shard(batch, world, rank)
    C = torch.empty((count, M, N), dtype=torch.int8, device=A.device)
    if count:
        b = bias[start:start + count] if (bias is not None and bias.dim() == 2) else bias
        (kernel or binding.batched_gemm_i8)(A[start:start + count], B[start:start + count], C, b, mult, shift, per_channel, relu)
    if gather and world > 1:
        return gather_rows(C.reshape(count, M * N), batch, world, align=2).reshape(batch, M, N)
    return C
