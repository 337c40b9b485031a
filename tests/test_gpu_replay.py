"""GPU parity of the circular buffer of trajectories (App. A "Circular Replay Buffer", Section 5.3):
the CUDA ingest, called through the C ABI, against the oracle's sequential ingest on the same inputs.
Rows, masses, segment offsets, liveness flags, the write index and every partial sum of the sampler
must match bit for bit; what is computed from the wrapped buffer afterwards (Retrace targets,
priorities, draws) obeys the contracts of those entry points."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_14803_b200 as distrl
from paper_2410_14803_b200 import binding

from helpers import assert_close, dev, read_tree, sample_by_prefix, tree_from_q

pytestmark = pytest.mark.gpu

N_FIELDS = 5   # r, V, log pi, log mu, entropy


class _Pair:
    """The CUDA buffer and the oracle's, fed the same calls."""

    def __init__(self, capacity, m_capacity, with_sampler=True, n_fields=N_FIELDS):
        self.n, self.mcap = capacity, m_capacity
        self.fields = [torch.full((capacity,), float("nan"), dtype=torch.float32, device="cuda") for _ in range(n_fields)]
        self.q = torch.full((capacity,), 12345, dtype=torch.int32, device="cuda")
        self.off = torch.full((m_capacity + 1,), -7, dtype=torch.int64, device="cuda")
        self.alive = torch.full((m_capacity,), float("nan"), dtype=torch.float32, device="cuda")
        self.ws = distrl.alloc_workspace(distrl.distrl_replay_workspace_bytes(capacity))
        self.rb = distrl.distrl_replay_create(self.fields, self.q, self.off, self.alive, self.ws)
        self.sampler = None
        if with_sampler:
            self.sws = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(capacity))
            distrl.distrl_workspace_init(self.sws)
            self.sampler = distrl.distrl_build_sampler(self.q, self.sws)
        self.ring = oracle.Ring(capacity, n_fields)
        self.m_out = torch.zeros(1, dtype=torch.int64, device="cuda")
        self.ingested = False

    def ingest(self, lens, rows, q):
        off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
        d_rows = [dev(r.astype(np.float32)) for r in rows]
        distrl.distrl_replay_ingest(self.rb, self.sampler, off, dev(off), d_rows, dev(q.astype(np.uint32).view(np.int32)),
                                    self.m_out)
        assert self.ring.ingest(off, [r.astype(np.float32) for r in rows], q)
        self.ingested = True

    def check(self):
        assert distrl.distrl_get_status(self.ws) == 0
        ring = self.ring
        assert self.rb.head == ring.head
        for got, want in zip(self.fields, ring.fields):
            np.testing.assert_array_equal(got.cpu().numpy().astype(np.float64), want)
        q = self.q.cpu().numpy().view(np.uint32)
        np.testing.assert_array_equal(q, ring.q)
        seg_off, seg_alive = ring.segments()
        m = seg_alive.shape[0]
        assert m <= self.mcap and (not self.ingested or int(self.m_out.item()) == m)
        got_off = self.off.cpu().numpy()
        np.testing.assert_array_equal(got_off[:m + 1], seg_off)
        assert np.all(got_off[m:] == self.n)                       # the padding: empty segments at the end
        got_alive = self.alive.cpu().numpy()
        np.testing.assert_array_equal(got_alive[:m], seg_alive.astype(np.float32))
        assert not got_alive[m:].any()
        if self.sampler is not None:
            got, info = read_tree(self.sampler)
            for a, b in zip(got, tree_from_q(q, info)):
                np.testing.assert_array_equal(a, b)
            assert distrl.distrl_get_status(self.sws) == 0
        return q, seg_off, seg_alive

    def close(self):
        if self.sampler is not None:
            self.sampler.close()
        self.rb.close()


def _rows(rng, total):
    r = rng.normal(0, 1, total)
    V = rng.random(total)
    lm = rng.normal(-5, 2, total)
    lp = lm + rng.normal(0, 0.5, total)
    ent = rng.uniform(0, 3, total)
    return [r, V, lp, lm, ent]


def _lens_short(rng, capacity):
    return rng.integers(0, 21, size=int(rng.integers(1, 40))).tolist()


def _lens_long(rng, capacity):
    return rng.integers(1, capacity // 12, size=int(rng.integers(1, 6))).tolist()


def _lens_geometric(rng, capacity):
    return np.minimum(64, rng.geometric(1 / 12, size=int(rng.integers(50, 400)))).tolist()


@pytest.mark.parametrize("capacity,maker,calls", [
    (1000, _lens_short, 40),          # short trajectories, many laps around a small buffer
    (50_000, _lens_long, 60),         # long ones: the cut trajectories reach across many words of the bit masks
    (70_001, _lens_geometric, 60),    # capacity not a multiple of 32
    (4096 * 33 + 5, _lens_long, 45),  # more than one block of words in the compaction
], ids=["short", "long", "geometric", "large"])
@pytest.mark.parametrize("with_sampler", [True, False], ids=["tree", "plain"])
def test_ring_ingest_matches_the_oracle(capacity, maker, calls, with_sampler):
    rng = np.random.default_rng(capacity)
    pair = _Pair(capacity, capacity, with_sampler)
    pair.check()                                                       # the empty buffer: one dead segment
    laps = 0
    for call in range(calls):
        lens = maker(rng, capacity)
        while sum(lens) > capacity // 2:
            lens = lens[:-1]
        total = int(sum(lens))
        before = pair.ring.head
        pair.ingest(lens, _rows(rng, total), rng.integers(1, 2 ** 32, size=total, dtype=np.uint64))
        laps += pair.ring.head < before
        if call % 5 == 4 or call == calls - 1:
            pair.check()
    assert laps >= 2, "the sequence should wrap around more than once"
    pair.close()


def test_ring_hand_patterns_exact_fill_whole_buffer_and_cuts():
    rng = np.random.default_rng(1)

    def go(pair, lens):
        total = int(sum(lens))
        pair.ingest(lens, _rows(rng, total), rng.integers(1, 1000, size=total))
        return pair.check()

    pair = _Pair(100, 100)
    go(pair, [60, 40])                    # exactly full, the write index is back at 0
    assert pair.rb.head == 0
    go(pair, [100])                       # one trajectory as long as the buffer replaces everything
    assert pair.rb.head == 0
    go(pair, [10])                        # cuts it: slots 10..99 die
    q, off, alive = go(pair, [0, 0])      # nothing but empty trajectories: nothing changes
    assert off.tolist() == [0, 10, 100] and alive.tolist() == [1, 0]
    assert q[:10].all() and not q[10:].any()
    pair.close()
    pair = _Pair(100, 100)
    go(pair, [20, 70])                    # head 90
    q, off, alive = go(pair, [5, 8])      # 5 rows at 90..94; 8 do not fit: 95..99 retired, rows at 0..7 cut the first
    assert off.tolist() == [0, 8, 20, 90, 95, 100] and alive.tolist() == [1, 0, 1, 1, 0]
    q, off, alive = go(pair, [30])        # slots 8..37: the rest of the 70-row trajectory (38..89) dies with it
    assert off.tolist() == [0, 8, 38, 90, 95, 100] and alive.tolist() == [1, 1, 0, 1, 0]
    assert not q[38:90].any() and q[8:38].all() and q[90:95].all()
    pair.close()


def test_ring_refusals_change_nothing():
    pair = _Pair(64, 64)
    rng = np.random.default_rng(2)
    pair.ingest([20, 20], _rows(rng, 40), rng.integers(1, 99, size=40))
    state = pair.check()
    lib = binding._load()

    def raw(lens_host, lens_dev=None):
        off = np.concatenate([[0], np.cumsum(lens_host)]).astype(np.int64)
        offd = off if lens_dev is None else np.concatenate([[0], np.cumsum(lens_dev)]).astype(np.int64)
        total = int(off[-1])
        rows = [dev(x.astype(np.float32)) for x in _rows(rng, max(total, 1))]
        q = dev(rng.integers(1, 99, size=max(total, 1)).astype(np.int32))
        return lib.distrl_replay_ingest(pair.rb.handle, pair.sampler.handle, off.shape[0] - 1,
                                        off.ctypes.data_as(binding.ctypes.c_void_p), dev(offd).data_ptr(),
                                        binding._ptr_array(rows, torch.float32), q.data_ptr(), None, None)

    assert raw([65]) == binding.ERR_SIZE                  # longer than the buffer
    assert raw([30, 30]) == binding.ERR_SIZE              # 24 slots left, 30 + retired 24... the call laps itself
    off_bad = np.array([0, 5, 3], dtype=np.int64)
    assert lib.distrl_replay_ingest(pair.rb.handle, None, 2, off_bad.ctypes.data_as(binding.ctypes.c_void_p),
                                    dev(off_bad).data_ptr(), None, None, None, None) == binding.ERR_OFFSETS
    torch.cuda.synchronize()
    again = pair.check()
    for a, b in zip(state, again):
        np.testing.assert_array_equal(a, b)
    # host and device offsets that disagree are reported through the status word
    assert raw([4, 4], lens_dev=[4, 5]) == 0
    assert distrl.distrl_get_status(pair.ws) == binding.ERR_OFFSETS
    pair.close()


def test_ring_segment_capacity_overflow_is_reported():
    pair = _Pair(256, 4, with_sampler=False)
    rng = np.random.default_rng(3)
    lens = [3] * 10                                        # 10 live segments + 1 dead > 4
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    distrl.distrl_replay_ingest(pair.rb, None, off, dev(off), [dev(x.astype(np.float32)) for x in _rows(rng, 30)],
                                dev(np.ones(30, dtype=np.int32)), pair.m_out)
    assert distrl.distrl_get_status(pair.ws) == binding.ERR_SIZE
    assert int(pair.m_out.item()) == 11
    got = pair.off.cpu().numpy()
    assert got.tolist() == [0, 3, 6, 9, 256]               # clipped, still a valid CSR over the buffer
    pair.close()


def test_empty_buffer_has_nothing_to_draw():
    pair = _Pair(5000, 100)
    u = dev(np.random.default_rng(4).integers(0, 2 ** 63, size=64).astype(np.int64))
    for normalise in (True, False):
        idx = torch.zeros(64, dtype=torch.int64, device="cuda")
        w = torch.full((64,), float("nan"), dtype=torch.float32, device="cuda")
        distrl.distrl_sample(pair.sampler, u, 0.4, normalise, idx, w)
        assert distrl.distrl_get_status(pair.sws) == binding.ERR_INDEX
        assert (idx.cpu().numpy() == -1).all() and (w.cpu().numpy() == 0).all()
    # the sampler is usable afterwards
    rng = np.random.default_rng(5)
    pair.ingest([7, 9], _rows(rng, 16), rng.integers(1, 99, size=16))
    q, _, _ = pair.check()
    uu = rng.integers(0, 2 ** 64, size=64, dtype=np.uint64)
    idx = torch.zeros(64, dtype=torch.int64, device="cuda")
    w = torch.zeros(64, dtype=torch.float32, device="cuda")
    distrl.distrl_sample(pair.sampler, dev(uu.view(np.int64)), 0.4, True, idx, w)
    np.testing.assert_array_equal(idx.cpu().numpy(), oracle.sample_linear(q, uu))
    assert_close(w.cpu().numpy(), oracle.is_weights(q, idx.cpu().numpy(), 0.4, True), "is_weight")
    pair.close()


@pytest.mark.parametrize("capacity,mean_len,seed", [(30_011, 12, 7), (200_000, 40, 8), (9_000, 300, 9)])
def test_full_path_through_a_wrapped_buffer(capacity, mean_len, seed):
    # New batches go through Retrace and the priority stage on their own (their masses are what the
    # buffer stores), are ingested past the wrap-around, and the wrapped buffer then goes back through
    # distrl_retrace_targets -> distrl_compute_priorities -> distrl_filter_trajectories (dead stretches)
    # -> distrl_build_sampler -> distrl_sample, all against the oracle.
    rng = np.random.default_rng(seed)
    gamma, lam, beta = 0.99, 0.95, 0.4
    cfg = distrl.make_prio_cfg(1.0, 0.5, 0.1, 2.0, 0.5, 2.0 ** 20)
    pair = _Pair(capacity, capacity)
    laps = 0
    for call in range(40):
        per_call = max(2, capacity // (6 * mean_len))
        lens = np.minimum(capacity // 8, rng.geometric(1 / mean_len, size=int(rng.integers(per_call // 2, 2 * per_call))))
        while lens.sum() > capacity // 3:
            lens = lens[:-1]
        total = int(lens.sum())
        off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
        rows = [x.astype(np.float32) for x in _rows(rng, total)]
        d = [dev(x) for x in rows]
        d_off = dev(off)
        vt, adv, dl, mass = (torch.empty(total, dtype=torch.float32, device="cuda") for _ in range(4))
        newq = torch.empty(total, dtype=torch.int32, device="cuda")
        ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(total))
        distrl.distrl_workspace_init(ws)
        distrl.distrl_retrace_targets(distrl.make_batch(d_off, d[0], d[1], d[2], d[3]), gamma, lam, vt, adv, dl, workspace=ws)
        distrl.distrl_compute_priorities(dl, d[2], d[3], d[4], cfg, mass, newq)
        assert distrl.distrl_get_status(ws) == 0
        before = pair.ring.head
        distrl.distrl_replay_ingest(pair.rb, pair.sampler, off, d_off, d, newq, pair.m_out)
        assert pair.ring.ingest(off, rows, newq.cpu().numpy().view(np.uint32))
        laps += pair.ring.head < before
    assert laps >= 2
    q, seg_off, seg_alive = pair.check()
    live = np.repeat(seg_alive.astype(bool), np.diff(seg_off))
    assert live.any() and not live.all()
    # draws straight from the incrementally repaired tree
    u = rng.integers(0, 2 ** 64, size=2048, dtype=np.uint64)
    idx = torch.empty(2048, dtype=torch.int64, device="cuda")
    w = torch.empty(2048, dtype=torch.float32, device="cuda")
    distrl.distrl_sample(pair.sampler, dev(u.view(np.int64)), beta, True, idx, w)
    got_idx = idx.cpu().numpy()
    np.testing.assert_array_equal(got_idx, sample_by_prefix(q, u))
    np.testing.assert_array_equal(got_idx[:32], oracle.sample_linear(q, u[:32]))
    assert live[got_idx].all()                                          # no evicted transition is ever drawn
    assert_close(w.cpu().numpy(), oracle.is_weights(q, got_idx, beta, True), "is_weight")
    # the whole wrapped buffer back through the path, with the padded offsets (n_trajectories = capacity of the list)
    n = capacity
    f = pair.fields
    vt, adv, dl, mass = (torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(4))
    q2 = torch.empty(n, dtype=torch.int32, device="cuda")
    ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    distrl.distrl_retrace_targets(distrl.make_batch(pair.off, f[0], f[1], f[2], f[3]), gamma, lam, vt, adv, dl, workspace=ws)
    assert distrl.distrl_get_status(ws) == 0
    h = [x.cpu().numpy() for x in f]
    o_vt, o_adv, o_dl = oracle.retrace(seg_off, h[0], h[1], h[2], h[3], gamma, lam)
    assert_close(vt.cpu().numpy()[live], o_vt[live], "v_target of the live trajectories")
    assert_close(adv.cpu().numpy()[live], o_adv[live], "advantage of the live trajectories")
    assert_close(dl.cpu().numpy(), o_dl, "td_delta")                    # dead rows are finite numbers too
    distrl.distrl_compute_priorities(dl, f[2], f[3], f[4], cfg, mass, q2)
    kept = torch.zeros(1, dtype=torch.int64, device="cuda")
    distrl.distrl_filter_trajectories(pair.off, pair.alive, 0.5, q2, kept)
    assert int(kept.item()) == int(seg_alive.sum())
    o_mass = oracle.priority_mass(dl.cpu().numpy(), h[2], h[3], h[4], 1.0, 0.5, 0.1, 2.0, 0.5)
    assert_close(mass.cpu().numpy(), o_mass, "prio_mass")
    want_q = oracle.quantise(mass.cpu().numpy(), 2.0 ** 20)
    assert oracle.filter_trajectories(seg_off, seg_alive.astype(np.float64), 0.5, want_q) == int(seg_alive.sum())
    got_q = q2.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(got_q, want_q)
    assert not got_q[~live].any() and got_q[live].all()
    sws = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(n))
    distrl.distrl_workspace_init(sws)
    s2 = distrl.distrl_build_sampler(q2, sws)
    distrl.distrl_sample(s2, dev(u.view(np.int64)), beta, True, idx, w)
    np.testing.assert_array_equal(idx.cpu().numpy(), sample_by_prefix(got_q, u))
    assert live[idx.cpu().numpy()].all()
    assert_close(w.cpu().numpy(), oracle.is_weights(got_q, idx.cpu().numpy(), beta, True), "is_weight")
    assert distrl.distrl_get_status(sws) == 0
    s2.close()
    pair.close()
