"""Multi-GPU plumbing.  Every output row of the quantized linear depends only on its own input row,
its stream's table entry and the shared weight, so the path shards by rows with NO collective on the
data path: each rank runs the same kernels on its rows with replicated weights and tables.  The only
communication is the barrier and the max-over-ranks of the timing."""
from __future__ import annotations

import numpy as np


def shard_rows(M: int, seg_offsets, seg_stream, rank: int, world: int):
    """Rows [lo, hi) of rank `rank` out of `world`, and that slice's own segment arrays
    (offsets relative to lo).  Rows are split as evenly as possible; a segment that straddles a
    boundary is cut, which is exact because rows are independent."""
    assert 0 <= rank < world and M >= 1
    base, extra = divmod(M, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    off = np.asarray(seg_offsets, np.int64)
    st = np.asarray(seg_stream, np.int64)
    out_off, out_st = [0], []
    for s in range(len(st)):
        a, b = max(int(off[s]), lo), min(int(off[s + 1]), hi)
        if b > a:
            out_off.append(b - lo)
            out_st.append(int(st[s]))
    if not out_st:                      # an empty shard still needs one (empty) segment
        out_st = [int(st[0])]
        out_off = [0, 0]
    return lo, hi, np.asarray(out_off, np.int32), np.asarray(out_st, np.int32)


def max_over_ranks(value: float, device=None) -> float:
    """MAX of a scalar over all ranks of the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank: float, world: int, ms_max: float) -> float:
    """Units all ranks processed per second, given the slowest rank's time for its share."""
    return units_per_rank * world / (ms_max * 1e-3)
