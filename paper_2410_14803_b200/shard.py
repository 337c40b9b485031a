"""Host-side helpers for running one replay shard per GPU.

Trajectories are independent, so the hot path shards with no data-path collective: every rank owns
its own buffer (and its own sampler) and the only communication is the barrier around the timed
region and the reduction below.
"""
from __future__ import annotations

from typing import List, Sequence

import torch
import torch.distributed as dist


def max_over_ranks(values: Sequence[float], device: str = "cpu") -> List[float]:
    """Element-wise maximum of `values` over all ranks of the default process group (identity when
    torch.distributed is not initialised).  Timings of a multi-GPU run are reported this way."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]
