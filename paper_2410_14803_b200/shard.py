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


# ---------------------------------------------------------------------------------------------------
# One prioritized replay over several shards (one per GPU): the proportional draw of App. A
# ("Priority-Based Sampling": P(i) = p_i^alpha / sum_j p_j^alpha) taken over the concatenation of the
# shards' masses.  The only exchange is the list of per-shard totals (8 bytes per rank).  A draw's
# threshold y = floor(u T / 2^64) falls into exactly one shard g; inside it the draw is the local one
# with threshold y - (total of the shards before g), and that local threshold is reproduced exactly by
# the local 0.64 fixed-point uniform u' = ceil(y_local 2^64 / T_g), since then floor(u' T_g / 2^64) =
# y_local.  So every rank feeds its own distrl_sample with the routed uniforms of the draws it owns and
# the result equals one linear scan over all masses.  Integer arithmetic throughout (Python integers).
# ---------------------------------------------------------------------------------------------------

def gather_totals(local_total: int) -> List[int]:
    """Total mass of every shard, in rank order (all-gather of one 64-bit integer per rank)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [int(local_total)]
    mine = torch.tensor([int(local_total) - (1 << 63)], dtype=torch.int64)   # uint64 carried in an int64
    out = [torch.zeros(1, dtype=torch.int64) for _ in range(dist.get_world_size())]
    dist.all_gather(out, mine)
    return [int(t.item()) + (1 << 63) for t in out]


def route_draws(u_fix, totals: Sequence[int]):
    """Owner shard and local uniform of every global draw.

    u_fix: iterable of 0.64 fixed-point uniforms (integers in [0, 2^64)); totals: total mass per shard.
    Returns (owner, u_local): lists of the same length; draw j belongs to shard owner[j], which obtains
    it by sampling its own masses with the uniform u_local[j]."""
    totals = [int(t) for t in totals]
    grand = sum(totals)
    if grand <= 0:
        raise ValueError("no mass in any shard")
    before = [0]
    for t in totals:
        before.append(before[-1] + t)
    owner, u_local = [], []
    for u in u_fix:
        y = (int(u) * grand) >> 64
        g = 0
        while before[g + 1] <= y:      # few shards: a linear walk
            g += 1
        y_local = y - before[g]
        up = -((-(y_local << 64)) // totals[g])          # ceil(y_local 2^64 / T_g)
        assert up < (1 << 64) and (up * totals[g]) >> 64 == y_local
        owner.append(g)
        u_local.append(up)
    return owner, u_local


def global_weight_factor(n_local: int, total_local: int, n_global: int, total_global: int, beta: float) -> float:
    """What a shard multiplies its un-normalised local importance weights (n_local q / T_local)^-beta by to get
    the global ones (n_global q / T_global)^-beta; the batch maximum is then one all-reduce (max_over_ranks)."""
    return ((n_global / n_local) * (total_local / total_global)) ** (-beta)


def sample_over_shards(sampler, n_local: int, u_fix, beta: float, idx_out, w_out, normalise: bool = True):
    """One batch drawn over all ranks' shards, every step on the device (device tensors in and out).

    All-gathers the shards' totals and sizes, routes the draws (distrl_route_draws), samples locally with
    the routed uniforms, turns the owned draws into global indices and weights (distrl_finish_shard_draws),
    assembles the batch with one element-wise maximum over the ranks and divides by the batch maximum.
    With one rank it is distrl_sample with a detour."""
    from . import binding as b
    k = u_fix.numel()
    dev = u_fix.device
    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    rank = dist.get_rank() if world > 1 else 0
    mine_total = torch.zeros(1, dtype=torch.int64, device=dev)
    b.distrl_sampler_total(sampler, mine_total)
    sizes = torch.tensor([int(n_local)], dtype=torch.int64, device=dev)
    if world > 1:
        totals = torch.zeros(world, dtype=torch.int64, device=dev)
        all_n = torch.zeros(world, dtype=torch.int64, device=dev)
        dist.all_gather_into_tensor(totals, mine_total)
        dist.all_gather_into_tensor(all_n, sizes)
        ns = [int(x) for x in all_n.cpu()]
    else:
        totals, ns = mine_total, [int(n_local)]
    u_local = torch.empty(k, dtype=torch.int64, device=dev)
    mine = torch.empty(k, dtype=torch.uint8, device=dev)
    b.distrl_route_draws(u_fix, totals, rank, u_local, mine)
    idx_local = torch.empty(k, dtype=torch.int64, device=dev)
    w_local = torch.empty(k, dtype=torch.float32, device=dev)
    b.distrl_sample(sampler, u_local, beta, False, idx_local, w_local)
    b.distrl_finish_shard_draws(mine, idx_local, w_local, totals, rank, ns[rank], sum(ns), sum(ns[:rank]), beta,
                                idx_out, w_out)
    if world > 1:
        dist.all_reduce(idx_out, op=dist.ReduceOp.MAX)
        dist.all_reduce(w_out, op=dist.ReduceOp.MAX)
    if normalise:
        b.distrl_normalise_weights(w_out)
