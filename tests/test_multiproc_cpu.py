"""World-size-2 check, on CPU with gloo, of the host logic the multi-GPU benchmark relies on: every
rank builds its own replay shard from its rank-dependent seed (no data-path collective), and the
step time that is reported is the maximum over ranks."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from paper_2410_14803_b200 import synth
    from paper_2410_14803_b200.shard import max_over_ranks
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.make_workload(1, shard=rank)
        digest = float(np.sum(w.arrays["rewards"], dtype=np.float64) + np.sum(w.arrays["values"], dtype=np.float64))
        # every rank reports a different step time; all must agree on the maximum
        ms = max_over_ranks([10.0 + rank, 3.0 - rank])
        gathered = [None] * world
        dist.all_gather_object(gathered, (w.n, w.m, digest))
        out.put((rank, ms, gathered))
    finally:
        dist.destroy_process_group()


def test_two_ranks_build_distinct_shards_and_agree_on_the_slowest():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, gathered in results:
        assert ms == [11.0, 3.0]                       # max over ranks of each entry
        (n0, m0, d0), (n1, m1, d1) = gathered
        assert m0 == m1 == 4096                        # same shape of work per rank (weak scaling)
        assert d0 != d1                                # but different data: the shards are independent


def test_shard_zero_is_the_unsharded_workload():
    sys.path.insert(0, ROOT)
    from paper_2410_14803_b200 import synth
    a, b = synth.make_workload(0), synth.make_workload(0, shard=0)
    for k in a.arrays:
        np.testing.assert_array_equal(a.arrays[k], b.arrays[k])
    c = synth.make_workload(0, shard=3)
    assert not np.array_equal(a.arrays["values"][:50], c.arrays["values"][:50])


def _global_sampler_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import oracle
    from paper_2410_14803_b200 import shard
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        sizes = [700, 1300, 90][:world]
        qs = [np.random.default_rng(50 + r).integers(1, 2 ** 32, size=sizes[r], dtype=np.uint64).astype(np.uint32)
              for r in range(world)]                                  # every rank can rebuild all shards (for the check)
        q_local = qs[rank]
        totals = shard.gather_totals(int(q_local.sum(dtype=np.uint64)))
        assert totals == [int(q.sum(dtype=np.uint64)) for q in qs]
        u = np.random.default_rng(7).integers(0, 2 ** 64, size=400, dtype=np.uint64)   # the same draws on every rank
        u[:3] = [0, 2 ** 64 - 1, 2 ** 63]
        owner, u_local = shard.route_draws(u.tolist(), totals)
        mine = [j for j, g in enumerate(owner) if g == rank]
        idx_local = oracle.sample_linear(q_local, np.array([u_local[j] for j in mine], dtype=np.uint64))
        base = sum(sizes[:rank])
        beta = 0.4
        raw = oracle.is_weights(q_local, idx_local, beta, False) * shard.global_weight_factor(
            sizes[rank], totals[rank], sum(sizes), sum(totals), beta)
        wmax = shard.max_over_ranks([float(raw.max()) if len(mine) else 0.0])[0]
        out.put((rank, mine, (base + idx_local).tolist(), (raw / wmax).tolist()))
    finally:
        dist.destroy_process_group()


def test_draws_routed_to_their_shards_equal_one_linear_scan_over_all_masses():
    import oracle
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_global_sampler_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    sizes = [700, 1300]
    q_all = np.concatenate([np.random.default_rng(50 + r).integers(1, 2 ** 32, size=sizes[r], dtype=np.uint64).astype(np.uint32)
                            for r in range(world)])
    u = np.random.default_rng(7).integers(0, 2 ** 64, size=400, dtype=np.uint64)
    u[:3] = [0, 2 ** 64 - 1, 2 ** 63]
    want_idx = oracle.sample_linear(q_all, u)                         # one linear scan over the concatenation
    want_w = oracle.is_weights(q_all, want_idx, 0.4, True)
    got_idx = np.full(400, -1, dtype=np.int64)
    got_w = np.zeros(400)
    for rank, mine, idx, w in results:
        got_idx[mine] = idx
        got_w[mine] = w
    np.testing.assert_array_equal(got_idx, want_idx)                  # every draw owned by exactly one shard
    np.testing.assert_allclose(got_w, want_w, rtol=1e-12)


def test_routing_identity_on_extreme_totals():
    sys.path.insert(0, ROOT)
    from paper_2410_14803_b200 import shard
    rng = np.random.default_rng(3)
    for totals in ([1, 1, 1], [2 ** 63, 5, 2 ** 62], [7], [3, 2 ** 40 + 1]):
        us = [0, 2 ** 64 - 1, 2 ** 63] + [int(x) for x in rng.integers(0, 2 ** 64, size=200, dtype=np.uint64)]
        owner, ul = shard.route_draws(us, totals)
        grand = sum(totals)
        for u, g, up in zip(us, owner, ul):
            y = (u * grand) >> 64
            assert sum(totals[:g]) <= y < sum(totals[:g + 1])
            assert (up * totals[g]) >> 64 == y - sum(totals[:g])
