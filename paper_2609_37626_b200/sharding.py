"""Host-side sharding of the decode path over ranks, one process per GPU.

The attention shard of a rank is fixed by the layout (Sec. 3 of the paper): a head
slice of H/T heads under TP / DOP, the requests it owns under DP-attention (assigned
round-robin so that counts are balanced, App. B), or a contiguous 1/T of every
request's tokens under position-sharded CP (App. E).  Head and request slices are
independent units -- no exchange happens inside attention -- so several ranks simply
run their own calls; only CP ends with one exchange (an all-gather of the per-rank
(O, LSE) partials followed by splash_lse_merge on each rank).

Nothing here touches a GPU: these helpers only compute index ranges and reduce timing
numbers over a torch.distributed process group (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import List, Tuple

import numpy as np


def head_slice(rank: int, world: int, num_heads: int) -> Tuple[int, int]:
    """[head_begin, head_end) of a rank under TP / DOP (H divisible by T)."""
    assert num_heads % world == 0, "head count must divide evenly over the ranks"
    per = num_heads // world
    return rank * per, (rank + 1) * per


def request_slice(rank: int, world: int, num_requests: int) -> np.ndarray:
    """Requests owned by a rank under DP-attention / DOP: round-robin, count-balanced."""
    return np.arange(rank, num_requests, world, dtype=np.int64)


def kv_range(rank: int, world: int, seq_lens: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Contiguous token range [begin, end) of every request held by a CP rank."""
    s = np.asarray(seq_lens, dtype=np.int64)
    return (s * rank // world).astype(np.int32), (s * (rank + 1) // world).astype(np.int32)


def max_over_ranks(values: List[float], device=None) -> List[float]:
    """Element-wise maximum of a few floats over the default process group (identity when
    torch.distributed is not initialised)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(values, dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def weak_scaling_value(units_per_rank: int, world: int, ms_max: float) -> float:
    """Whole-job throughput when every rank processes `units_per_rank` units in the time of
    the slowest rank."""
    return world * units_per_rank / (ms_max * 1e-3)
