"""Host-side helpers for running the layer on several GPUs, one process per GPU.

Every step of the path (rotation, quantization, GEMM) is independent per row (token) of X, so a
batch is split by rows, the rotations and the quantized weights are replicated, and no data moves
between ranks.  The only cross-rank operation is the reduction of timings (max over ranks) that a
benchmark needs."""
from __future__ import annotations

import torch


def row_range(M: int, rank: int, world: int) -> tuple[int, int]:
    """Half-open row interval [lo, hi) of `rank` in a balanced contiguous split of M rows: the
    first M % world ranks get one row more.  Empty when there are more ranks than rows."""
    if world < 1 or not 0 <= rank < world or M < 0:
        raise ValueError(f"bad partition request M={M} rank={rank} world={world}")
    base, extra = divmod(M, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks of the default process group
    (identity when torch.distributed is not initialised)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]
