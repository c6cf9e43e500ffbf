"""Row-block sharding of the fused operators over several GPUs (one process per GPU).

Every template is a map over independent rows (cells, stored cells) followed by a
sum, so the main input - and whatever has its row count: cell-shaped and
column-vector sides, U of the Outer template - is split into contiguous row blocks,
one per rank (for a CSR matrix: blocks holding equal shares of the stored cells);
small inputs (v, row-vector sides, V) are replicated.  Each rank runs the ordinary
single-GPU call on its block; full, column and k-vector aggregates are then summed
over the ranks with ONE all-reduce of the result (8 bytes to a few KB); per-row and
per-cell results stay partitioned by rows and need no communication.  No kernel is
ever handed memory of another GPU.

The functions here are host logic only (which rows go where, and how the pieces
combine); the single-GPU call is passed in, so the same code runs under `gloo` on
CPU in the tests and under `nccl` on GPUs.
"""
from __future__ import annotations

import numpy as np


def row_block(rows: int, rank: int, world: int):
    """[lo, hi) of the contiguous row block of `rank`: sizes differ by at most one."""
    base, extra = divmod(int(rows), int(world))
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def csr_row_blocks(rowptr, world: int):
    """Row boundaries b[0..world] of contiguous row blocks holding equal shares of the
    stored cells: block r is rows [b[r], b[r + 1]).  rowptr: rows + 1 offsets."""
    rowptr = np.asarray(rowptr, dtype=np.int64)
    rows, nnz = rowptr.size - 1, int(rowptr[-1])
    bounds = [0]
    for r in range(1, world):
        # the first row whose offset reaches the r-th share of the cells, never before the last bound
        b = int(np.searchsorted(rowptr, (nnz * r) // world, side="left"))
        bounds.append(min(max(b, bounds[-1]), rows))
    bounds.append(rows)
    return bounds


def csr_block(rowptr, colidx, vals, lo: int, hi: int):
    """The sub-matrix of rows [lo, hi) as (rowptr, colidx, vals) with offsets rebased to 0."""
    rowptr = np.asarray(rowptr)
    a, b = int(rowptr[lo]), int(rowptr[hi])
    return (rowptr[lo:hi + 1] - rowptr[lo]).astype(rowptr.dtype), colidx[a:b], vals[a:b]


# which results are sums over rows (one all-reduce) and which stay partitioned by rows
REDUCED = {
    "cell": {"full": True, "col": True, "row": False, "none": False},
    "magg": {"full": True},
    "row": {"col_t": True, "col": True, "full": True, "row": False, "none": False},
    "row_b1": {"col_t": True, "none": False},
    "outer": {"full": True, "left": True, "right": False, "none": False},
}


def combine(template: str, agg: str, local_result, group=None):
    """The job-wide result from this rank's: an all-reduce (sum) for the aggregates that
    sum over rows, the local piece unchanged for results partitioned by rows (the caller
    keeps them distributed, or gathers them by rank order)."""
    import torch
    import torch.distributed as dist
    if not REDUCED[template][agg]:
        return local_result
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        t = local_result if isinstance(local_result, torch.Tensor) \
            else torch.as_tensor(local_result, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
        return t
    return local_result


def sharded(template: str, agg: str, local_call, group=None):
    """Runs `local_call()` - the single-GPU fused operator on this rank's row block - and
    combines the result over the ranks."""
    return combine(template, agg, local_call(), group)
