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
