"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle
on the same seeded inputs.  Bit-exact for masses, partial sums and indices;
max |err| <= 1e-4 (1 + |ref|) for every fp32 output."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_14803_b200 as distrl
from paper_2410_14803_b200 import synth

from helpers import (TOL, assert_close, check_retrace, dev, gpu_retrace, prio_cfg_of, random_batch, read_tree,
                     sample_by_prefix, tree_from_q)

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------ Retrace ---

@pytest.mark.parametrize("index", [0, 1, 2, 3])
def test_retrace_workloads(index):
    w = synth.make_workload(index)
    a = w.arrays
    check_retrace(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"],
                  w.gamma, w.lam)


@pytest.mark.parametrize("kind", ["single", "ones", "tile_aligned", "tile_straddle", "with_empty", "long_mixed"])
@pytest.mark.parametrize("n", [1, 5, 2048, 2049, 20000, 70001])
def test_retrace_adversarial_layouts(kind, n):
    off = synth.adversarial_offsets(kind, n)
    r, V, lp, lm = random_batch(11 + n, off)
    check_retrace(off, r, V, lp, lm, 0.99, 0.95)


def test_retrace_long_trajectory_many_tiles_on_policy():
    # One trajectory over ~150 tiles with pi = mu and lambda = gamma = 1: the carry crosses
    # every tile boundary undamped, so every look-back link matters.
    n = 300001
    off = np.array([0, n], dtype=np.int64)
    rng = np.random.default_rng(5)
    r = rng.normal(0, 0.01, n).astype(np.float32)
    V = rng.random(n, dtype=np.float32)
    lm = rng.normal(-5, 2, n).astype(np.float32)
    out = gpu_retrace(off, r, V, lm, lm, 1.0, 1.0)
    assert out["status"] == 0
    vt, adv, dl = oracle.retrace(off, r, V, lm, lm, 1.0, 1.0)
    # fp32 running sums over 3e5 terms: compare with a tolerance scaled to the sum of magnitudes
    bound = 1e-4 * (1.0 + np.abs(adv)) + 2e-7 * np.cumsum(np.abs(dl[::-1]))[::-1] * 8
    assert np.all(np.abs(out["advantage"] - adv) <= bound)


@pytest.mark.parametrize("gamma,lam", [(0.95, 0.0), (1.0, 1.0), (0.0, 0.5), (0.5, 1.0)])
def test_retrace_parameter_corners(gamma, lam):
    w = synth.make_workload(1)
    a = w.arrays
    check_retrace(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"], gamma, lam)


def test_retrace_bootstrap_values():
    off = synth.adversarial_offsets("with_empty", 9000)
    r, V, lp, lm = random_batch(3, off)
    boot = np.random.default_rng(4).random(off.shape[0] - 1, dtype=np.float32)
    check_retrace(off, r, V, lp, lm, 0.97, 0.9, boot=boot)


@pytest.mark.parametrize("kind", ["with_empty", "long_mixed", "ones", "tile_aligned", "tile_straddle", "single"])
@pytest.mark.parametrize("n", [1, 129, 2047, 2048, 2049, 2176, 2177, 100003, 700001])
def test_retrace_bootstrap_values_layouts(kind, n):
    # bootstrap values with aligned arrays go through the pipelined kernel: ends inside the 128-item halo
    # of a tile, on tile boundaries, empty trajectories in between, buffers shorter than a halo
    off = synth.adversarial_offsets(kind, n)
    r, V, lp, lm = random_batch(n + 7, off)
    boot = np.random.default_rng(n).normal(0, 2, off.shape[0] - 1).astype(np.float32)
    check_retrace(off, r, V, lp, lm, 0.97, 0.9, boot=boot)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_retrace_bootstrap_values_empty_trajectories_everywhere(seed):
    # The pipelined kernel finds the trajectory of an end from the trajectory of the lowest end in the same
    # 32-step word of the end mask; empty trajectories break that count and are resolved by a search in the
    # offsets.  Here they sit wherever the bookkeeping changes hands: at the start and the end of the buffer,
    # in runs, between ends of one word, on both sides of every 2048th trajectory (one block of the mask
    # kernel takes 2048), right after a tile boundary.
    rng = np.random.default_rng(700 + seed)
    m = 3 * 2048 + 777
    lens = rng.integers(1, 6 if seed < 2 else 40, size=m)
    lens[rng.random(m) < 0.15] = 0
    for g in (0, 1, 2, m - 1, m - 2):
        lens[g] = 0
    for c in (2048, 4096, 6144):
        lens[c - 2:c + 3] = [0, 1, 0, 0, 2][:5] if seed != 1 else [1, 0, 0, 1, 0]
    lens[100:140] = 0                                     # a long run of empty trajectories
    lens[140:200] = 1                                     # then an end at every step
    lens[200:230:2] = 0
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    r, V, lp, lm = random_batch(seed + 30, off)
    boot = rng.normal(0, 2, m).astype(np.float32)
    check_retrace(off, r, V, lp, lm, 0.97, 0.9, boot=boot)


def test_retrace_bootstrap_values_through_the_general_kernel():
    # arrays that are not 16-byte aligned; and a workspace without room for what the pipelined kernel
    # keeps of the bootstrap values (the fixed array of the workspace-free entry point is one)
    off = synth.adversarial_offsets("long_mixed", 50001)
    r, V, lp, lm = random_batch(9, off)
    boot = np.random.default_rng(5).normal(0, 2, off.shape[0] - 1).astype(np.float32)
    check_retrace(off, r, V, lp, lm, 0.97, 0.9, boot=boot, misalign=True)
    n = r.shape[0]
    t = [dev(off), dev(r), dev(V), dev(lp), dev(lm), dev(boot)]     # kept alive: the batch only holds pointers
    batch = distrl.make_batch(*t)
    out = [torch.full((n,), float("nan"), dtype=torch.float32, device="cuda") for _ in range(3)]
    status = torch.full((1,), -77, dtype=torch.int32, device="cuda")
    distrl.distrl_retrace_targets_static(batch, 0.97, 0.9, *out, status_out=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    vt, adv, dl = oracle.retrace(off, r, V, lp, lm, 0.97, 0.9, bootstrap=boot)
    assert_close(out[0].cpu().numpy(), vt, "v_target")
    assert_close(out[1].cpu().numpy(), adv, "advantage")
    assert_close(out[2].cpu().numpy(), dl, "td_delta")


def test_retrace_bootstrap_repeated_runs_agree_bit_for_bit():
    n = 500001
    off = synth.adversarial_offsets("long_mixed", n)
    r, V, lp, lm = random_batch(77, off)
    boot = np.random.default_rng(6).normal(0, 2, off.shape[0] - 1).astype(np.float32)
    t = [dev(off), dev(r), dev(V), dev(lp), dev(lm), dev(boot)]
    batch = distrl.make_batch(*t)
    ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    first = None
    for _ in range(20):
        out = [torch.full((n,), float("nan"), dtype=torch.float32, device="cuda") for _ in range(3)]
        distrl.distrl_retrace_targets(batch, 0.99, 0.95, *out, workspace=ws)
        got = [o.view(torch.int32) for o in out]
        if first is None:
            first = got
        for g, f in zip(got, first):
            assert torch.equal(g, f)
    assert distrl.distrl_get_status(ws) == 0
    vt, adv, dl = oracle.retrace(off, r, V, lp, lm, 0.99, 0.95, bootstrap=boot)
    assert_close(first[0].view(torch.float32).cpu().numpy(), vt, "v_target")
    assert_close(first[1].view(torch.float32).cpu().numpy(), adv, "advantage")
    assert_close(first[2].view(torch.float32).cpu().numpy(), dl, "td_delta")


@pytest.mark.parametrize("n", [3, 4099, 30011])
def test_retrace_unaligned_pointers_and_ragged_tail(n):
    off = synth.adversarial_offsets("long_mixed", n)
    r, V, lp, lm = random_batch(n, off)
    check_retrace(off, r, V, lp, lm, 0.99, 0.95, misalign=True)


def test_retrace_without_optional_outputs_and_copy_of_logp():
    w = synth.make_workload(1)
    a = w.arrays
    out = gpu_retrace(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"],
                      w.gamma, w.lam, want_delta=False, want_logp=True)
    vt, adv, _ = oracle.retrace(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"],
                                a["logp_behaviour"], w.gamma, w.lam)
    assert_close(out["v_target"], vt, "v_target")
    np.testing.assert_array_equal(out["logp_target"], a["logp_target"])
    np.testing.assert_array_equal(out["logp_behaviour"], a["logp_behaviour"])


def test_retrace_is_deterministic():
    w = synth.make_workload(2)
    a = w.arrays
    args = (a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"], w.gamma, w.lam)
    x, y = gpu_retrace(*args), gpu_retrace(*args)
    for key in ("v_target", "advantage", "td_delta"):
        np.testing.assert_array_equal(x[key].view(np.uint32), y[key].view(np.uint32))


@pytest.mark.parametrize("kind", ["long_mixed", "single", "ones", "with_empty"])
def test_retrace_repeated_runs_agree_bit_for_bit(kind):
    # The warps of the pipelined scan meet through flags in shared and global memory; a missed ordering
    # would show up as a run that differs from the others.  Twenty runs on the same inputs and the same
    # workspace, on a layout that keeps several hundred tiles busy, must agree bit for bit (and with
    # the oracle).
    n = 700001
    off = synth.adversarial_offsets(kind, n)
    r, V, lp, lm = random_batch(31, off)
    t = [dev(off), dev(r), dev(V), dev(lp), dev(lm)]
    batch = distrl.make_batch(*t)
    ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    first = None
    for _ in range(20):
        out = [torch.full((n,), float("nan"), dtype=torch.float32, device="cuda") for _ in range(3)]
        distrl.distrl_retrace_targets(batch, 0.999, 0.97, *out, workspace=ws)
        got = [o.cpu().numpy().view(np.uint32) for o in out]
        if first is None:
            first = got
        for g, f in zip(got, first):
            np.testing.assert_array_equal(g, f)
    assert distrl.distrl_get_status(ws) == 0
    vt, adv, dl = oracle.retrace(off, r, V, lp, lm, 0.999, 0.97)
    assert_close(first[0].view(np.float32), vt, "v_target")
    assert_close(first[1].view(np.float32), adv, "advantage")
    assert_close(first[2].view(np.float32), dl, "td_delta")


def test_two_retrace_calls_at_the_same_time_on_two_streams():
    # Trajectories far longer than the 128-step halo: almost every tile needs the value that its right
    # neighbour produces, i.e. blocks wait for other blocks.  Two such calls on two streams (own
    # workspaces) compete for the SMs; each must still finish with status 0 and the oracle's results,
    # whichever way the device interleaves them (every tile goes by ticket, so a block only waits for
    # tiles of blocks that are already running).
    def case(seed, n, boot):
        rng = np.random.default_rng(seed)
        lens = []
        while sum(lens) < n:
            lens.append(int(rng.integers(300, 6000)))
        lens[-1] -= sum(lens) - n
        off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
        r, V, lp, lm = random_batch(seed, off)
        lp = (lm + rng.normal(0, 0.05, n)).astype(np.float32)        # ratios near 1: the trace stays alive
        b = rng.random(len(lens), dtype=np.float32) if boot else None
        return off, r, V, lp, lm, b

    cases = [case(41, 600_001, False), case(42, 450_000, False), case(43, 300_000, True)]
    streams = [torch.cuda.Stream() for _ in cases]
    held = []
    for (off, r, V, lp, lm, b), st in zip(cases, streams):
        n = r.shape[0]
        t = dict(off=dev(off), r=dev(r), V=dev(V), lp=dev(lp), lm=dev(lm), b=dev(b) if b is not None else None)
        t["batch"] = distrl.make_batch(t["off"], t["r"], t["V"], t["lp"], t["lm"], t["b"])
        t["out"] = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(3)]
        t["G"] = torch.empty(n, dtype=torch.float32, device="cuda")
        t["ws"] = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
        t["ws2"] = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
        distrl.distrl_workspace_init(t["ws"])
        distrl.distrl_workspace_init(t["ws2"])
        held.append(t)
    torch.cuda.synchronize()
    for rnd in range(6):
        for t in held:
            for o in t["out"]:
                o.fill_(float("nan"))
            t["G"].fill_(float("nan"))
        torch.cuda.synchronize()
        for _ in range(3):           # several calls in flight on every stream
            for t, st in zip(held, streams):
                distrl.distrl_retrace_targets(t["batch"], 0.99, 0.95, *t["out"], workspace=t["ws"], stream=st)
                distrl.distrl_mc_returns(t["batch"], 0.99, t["G"], None, workspace=t["ws2"], stream=st)
        torch.cuda.synchronize()
        for (off, r, V, lp, lm, b), t, st in zip(cases, held, streams):
            assert distrl.distrl_get_status(t["ws"], stream=st) == 0
            assert distrl.distrl_get_status(t["ws2"], stream=st) == 0
            vt, adv, dl = oracle.retrace(off, r, V, lp, lm, 0.99, 0.95, bootstrap=b)
            assert_close(t["out"][0].cpu().numpy(), vt, "v_target")
            assert_close(t["out"][1].cpu().numpy(), adv, "advantage")
            assert_close(t["out"][2].cpu().numpy(), dl, "td_delta")
            assert_close(t["G"].cpu().numpy(), oracle.mc_return(off, r, 0.99)[0], "mc_return")


def test_retrace_bad_offsets_are_reported_not_fatal():
    off = np.array([0, 10, 7, 20], dtype=np.int64)     # decreasing
    r, V, lp, lm = random_batch(1, np.array([0, 20]))
    out = gpu_retrace(off, r, V, lp, lm, 0.9, 0.9)
    assert out["status"] == distrl.binding.ERR_OFFSETS
    off = np.array([0, 10, 19], dtype=np.int64)        # does not end at N
    out = gpu_retrace(off, r, V, lp, lm, 0.9, 0.9)
    assert out["status"] == distrl.binding.ERR_OFFSETS
    # the workspace stays usable: a valid call afterwards is correct
    check_retrace(np.array([0, 10, 20], dtype=np.int64), r, V, lp, lm, 0.9, 0.9)


def test_a_wait_that_runs_out_is_reported_not_fatal():
    # one warp waits, with a short limit, for a tile that nothing publishes: the status word must say so,
    # and the same workspace must serve an ordinary call right after
    n = 5000
    ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    distrl.distrl_selftest_bounded_wait(ws)
    assert distrl.distrl_get_status(ws) == distrl.binding.ERR_TIMEOUT
    assert distrl.distrl_get_status(ws) == 0       # reading cleared it
    off = synth.adversarial_offsets("long_mixed", n)
    r, V, lp, lm = random_batch(5, off)
    check_retrace(off, r, V, lp, lm, 0.99, 0.95)


def test_mc_returns():
    for index in (1, 2):
        w = synth.make_workload(index)
        a = w.arrays
        n = w.n
        t_off, t_r = dev(a["traj_offsets"]), dev(a["rewards"])
        batch = distrl.make_batch(t_off, t_r, None)
        G = torch.empty(n, dtype=torch.float32, device="cuda")
        lab = torch.empty(n, dtype=torch.uint8, device="cuda")
        ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
        distrl.distrl_workspace_init(ws)
        distrl.distrl_mc_returns(batch, w.gamma, G, lab, workspace=ws)
        assert distrl.distrl_get_status(ws) == 0
        Gr, labr = oracle.mc_return(a["traj_offsets"], a["rewards"], w.gamma)
        assert_close(G.cpu().numpy(), Gr, "mc_return")
        # the label is decided in fp32 on the device: it must match the sign of the device's own G,
        # and the oracle's label wherever G is not within rounding of zero
        np.testing.assert_array_equal(lab.cpu().numpy(), (G.cpu().numpy() > 0).astype(np.uint8))
        clear = np.abs(Gr) > 1e-5
        np.testing.assert_array_equal(lab.cpu().numpy()[clear], labr[clear])


# --------------------------------------------------------------- priorities ---

def _gpu_priorities(w, delta, alpha=None, with_entropy=True):
    a = w.arrays
    n = w.n
    t = [dev(delta), dev(a["logp_target"]), dev(a["logp_behaviour"]), dev(a["entropy"]) if with_entropy else None]
    mass = torch.empty(n, dtype=torch.float32, device="cuda")
    q = torch.empty(n, dtype=torch.int32, device="cuda")
    distrl.distrl_compute_priorities(t[0], t[1], t[2], t[3], prio_cfg_of(w, alpha), mass, q)
    torch.cuda.synchronize()
    return mass.cpu().numpy(), q.cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("index,alpha,with_entropy", [(0, 0.5, True), (0, 1.0, True), (1, 0.5, True), (1, 1.0, False),
                                                      (1, 0.7, True), (2, 0.5, True), (3, 0.5, True)])
def test_priorities(index, alpha, with_entropy):
    w = synth.make_workload(index)
    a = w.arrays
    _, _, dl = oracle.retrace(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"],
                              w.gamma, w.lam)
    delta = dl.astype(np.float32)
    if w.heavy_tail:
        delta = (delta * synth.heavy_tail_scale(w)).astype(np.float32)
    mass, q = _gpu_priorities(w, delta, alpha, with_entropy)
    ref = oracle.priority_mass(delta, a["logp_target"], a["logp_behaviour"], a["entropy"] if with_entropy else None,
                               w.w_td, w.w_rho, w.w_ent, w.rho_clip, alpha)
    assert_close(mass, ref, "prio_mass")
    # integer stage: the device's q is exactly Q(device's fp32 mass)
    np.testing.assert_array_equal(q, oracle.quantise(mass, w.scale))
    assert q.min() >= 1
    # informational: how often Q of the oracle's own mass differs
    q_ref = oracle.quantise(ref.astype(np.float32), w.scale)
    diff = np.abs(q.astype(np.int64) - q_ref.astype(np.int64))
    assert np.all(diff <= np.maximum(1, 4e-7 * q_ref))


def test_priority_quantiser_edges_on_device():
    # drive the device quantiser through its corner cases with alpha = 1, w = (1, 0, 0): mass = |delta|
    S = 2.0 ** 20
    vals = np.array([0.0, 2.0 ** -21, 1.5 / S, 2.5 / S, 3.5 / S, 1.0, 4095.999, 4096.0, 1e30, np.inf, np.nan,
                     -3.0, 2.0 ** -30], dtype=np.float32)
    z = torch.zeros(vals.shape[0], dtype=torch.float32, device="cuda")
    mass = torch.empty_like(z)
    q = torch.empty(vals.shape[0], dtype=torch.int32, device="cuda")
    distrl.distrl_compute_priorities(dev(vals), z, z, z, distrl.make_prio_cfg(1.0, 0.0, 0.0, 2.0, 1.0, S), mass, q)
    got = q.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(got, oracle.quantise(mass.cpu().numpy(), S))
    assert got[0] == 1 and got[2] == 2 and got[3] == 2 and got[4] == 4 and got[7] == 2 ** 32 - 1 and got[10] == 1


def test_trajectory_level_priorities():
    w = synth.make_workload(1)
    a = w.arrays
    off = np.sort(np.concatenate([a["traj_offsets"], a["traj_offsets"][[5, 5, 100]]]))   # add empty trajectories
    _, _, dl = oracle.retrace(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"],
                              w.gamma, w.lam)
    delta = dl.astype(np.float32)
    m = off.shape[0] - 1
    mass = torch.empty(m, dtype=torch.float32, device="cuda")
    q = torch.empty(m, dtype=torch.int32, device="cuda")
    distrl.distrl_compute_priorities_traj(dev(off), dev(delta), dev(a["logp_target"]), dev(a["logp_behaviour"]),
                                          dev(a["entropy"]), prio_cfg_of(w), mass, q)
    ref = oracle.priority_mass_traj(off, delta, a["logp_target"], a["logp_behaviour"], a["entropy"], w.w_td, w.w_rho,
                                    w.w_ent, w.rho_clip, w.alpha)
    assert_close(mass.cpu().numpy(), ref, "traj prio_mass")
    np.testing.assert_array_equal(q.cpu().numpy().view(np.uint32), oracle.quantise(mass.cpu().numpy(), w.scale))


def _traj_layouts():
    rng = np.random.default_rng(77)
    yield "ones", np.ones(3000, dtype=np.int64)
    yield "rows_of_32", np.full(700, 32, dtype=np.int64)
    yield "31_33", np.tile(np.array([31, 33], dtype=np.int64), 400)
    yield "window_edges", np.array([2048, 2047, 1, 2049, 4096, 5, 6000, 255, 257, 256], dtype=np.int64)
    yield "one_long", np.array([50_001], dtype=np.int64)
    yield "empties_everywhere", np.concatenate([np.zeros(600, dtype=np.int64), [7], np.zeros(300, dtype=np.int64),
                                                rng.integers(0, 4, 900), [3000], np.zeros(5, dtype=np.int64)])
    yield "geometric_mix", np.minimum(rng.geometric(1 / 12.0, 5000), 200).astype(np.int64)
    yield "long_and_short", np.where(rng.random(1500) < 0.02, rng.integers(500, 3000, 1500), rng.integers(1, 6, 1500))
    yield "all_empty", np.zeros(300, dtype=np.int64)


@pytest.mark.parametrize("name,lens", list(_traj_layouts()), ids=[nm for nm, _ in _traj_layouts()])
@pytest.mark.parametrize("with_entropy", [True, False])
def test_trajectory_level_priorities_layouts(name, lens, with_entropy):
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    n, m = int(off[-1]), lens.shape[0]
    rng = np.random.default_rng(m + n)
    delta = (rng.normal(0, 1, n) * np.exp(rng.normal(0, 1, n))).astype(np.float32)
    lm = rng.normal(-5, 2, n).astype(np.float32)
    lp = (lm + rng.normal(0, 0.7, n)).astype(np.float32)
    ent = rng.uniform(0, 3, n).astype(np.float32)
    w = synth.make_workload(0)
    mass = torch.full((m,), float("nan"), dtype=torch.float32, device="cuda")
    q = torch.zeros(m, dtype=torch.int32, device="cuda")
    one = lambda x: dev(x) if n else torch.empty(0, dtype=torch.float32, device="cuda")
    runs = []
    for _ in range(3):
        distrl.distrl_compute_priorities_traj(dev(off), one(delta), one(lp), one(lm), one(ent) if with_entropy else None,
                                              prio_cfg_of(w), mass, q)
        torch.cuda.synchronize()
        runs.append((mass.cpu().numpy().copy(), q.cpu().numpy().copy()))
    ref = oracle.priority_mass_traj(off, delta, lp, lm, ent if with_entropy else None, w.w_td, w.w_rho, w.w_ent,
                                    w.rho_clip, w.alpha)
    assert_close(runs[0][0], ref, "traj prio_mass (%s)" % name)
    np.testing.assert_array_equal(runs[0][1].view(np.uint32), oracle.quantise(runs[0][0], w.scale))
    for r in runs[1:]:                                   # every sum is formed in one fixed order
        np.testing.assert_array_equal(r[0], runs[0][0])
        np.testing.assert_array_equal(r[1], runs[0][1])


# ------------------------------------------------------------------ sampler ---

def _masses(n, seed, heavy=True):
    rng = np.random.default_rng(seed)
    if heavy:
        x = np.exp(rng.normal(0, 3, n)) * 2 ** 18
        return np.clip(np.rint(x), 1, 2 ** 32 - 1).astype(np.uint32)
    return rng.integers(1, 2 ** 32, size=n, dtype=np.uint64).astype(np.uint32)


def _build(q):
    tq = dev(q.view(np.int32))
    ws = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(q.shape[0]))
    distrl.distrl_workspace_init(ws)
    return distrl.distrl_build_sampler(tq, ws), tq, ws


def _check_tree(s, q):
    got, info = read_tree(s)
    want = tree_from_q(q, info)
    for l, (g, x) in enumerate(zip(got, want), start=1):
        np.testing.assert_array_equal(g, x, err_msg="level %d" % l)
    tot = torch.zeros(1, dtype=torch.int64, device="cuda")
    distrl.distrl_sampler_total(s, tot)
    _, total = oracle.prefix(q)
    assert int(tot.cpu().numpy().view(np.uint64)[0]) == total
    assert int(got[-1].sum(dtype=np.uint64)) == total


def _sample(s, u, beta, normalise=True):
    k = u.shape[0]
    idx = torch.full((k,), -1, dtype=torch.int64, device="cuda")
    wts = torch.full((k,), float("nan"), dtype=torch.float32, device="cuda")
    distrl.distrl_sample(s, dev(u.view(np.int64)), beta, normalise, idx, wts)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), wts.cpu().numpy()


@pytest.mark.parametrize("n", [1, 2, 127, 128, 129, 4095, 4096, 4097, 131073, 1 << 20, (1 << 22) + 5])
@pytest.mark.parametrize("heavy", [True, False])
def test_sampler_build_and_sample(n, heavy):
    q = _masses(n, n + int(heavy), heavy)
    s, tq, ws = _build(q)
    _check_tree(s, q)
    rng = np.random.default_rng(n)
    u = rng.integers(0, 1 << 64, size=513, dtype=np.uint64)
    u[:4] = [0, 2 ** 64 - 1, 2 ** 63, 1]
    idx, wts = _sample(s, u, 0.4)
    np.testing.assert_array_equal(idx, sample_by_prefix(q, u))
    sub = slice(0, 24 if n > 100000 else 513)
    np.testing.assert_array_equal(idx[sub], oracle.sample_linear(q, u[sub]))       # the definition itself
    assert_close(wts, oracle.is_weights(q, idx, 0.4, True), "is_weight")
    assert wts.max() == 1.0
    _, raw = _sample(s, u, 0.6, normalise=False)
    assert_close(raw, oracle.is_weights(q, idx, 0.6, False), "is_weight raw")
    assert distrl.distrl_get_status(ws) == 0
    s.close()


def test_normalising_draw_without_a_cooperative_launch():
    # the library option that forbids cooperative launches sends a normalising draw down the path of
    # large batches (the last block rescales): same indices, same weights
    q = _masses((1 << 20) + 3, 77)
    s, tq, ws = _build(q)
    u = np.random.default_rng(78).integers(0, 1 << 64, size=4096, dtype=np.uint64)
    old = distrl.distrl_set_cooperative_launch(False)
    try:
        assert old is True
        idx, wts = _sample(s, u, 0.4)
    finally:
        assert distrl.distrl_set_cooperative_launch(old) is False
    idx2, wts2 = _sample(s, u, 0.4)
    np.testing.assert_array_equal(idx, sample_by_prefix(q, u))
    np.testing.assert_array_equal(idx, idx2)
    assert_close(wts, oracle.is_weights(q, idx, 0.4, True), "is_weight")
    assert_close(wts2, oracle.is_weights(q, idx, 0.4, True), "is_weight")
    assert distrl.distrl_get_status(ws) == 0
    s.close()


def test_two_samplers_drawing_at_the_same_time_on_two_streams():
    # A normalising draw lets its blocks wait for one another; two such draws from different samplers
    # on different streams must not starve each other (the launch is cooperative: each grid gets the
    # SMs it needs at once, or waits as a whole).
    k = 4096
    qa, qb = _masses(1 << 20, 3), _masses((1 << 20) + 77, 4, heavy=False)
    (sa, tqa, wsa), (sb, tqb, wsb) = _build(qa), _build(qb)
    st_a, st_b = torch.cuda.Stream(), torch.cuda.Stream()
    rng = np.random.default_rng(99)
    torch.cuda.synchronize()
    for rnd in range(25):
        ua = rng.integers(0, 2 ** 64, size=k, dtype=np.uint64)
        ub = rng.integers(0, 2 ** 64, size=k, dtype=np.uint64)
        d_ua, d_ub = dev(ua.view(np.int64)), dev(ub.view(np.int64))
        ia, ib = (torch.full((k,), -1, dtype=torch.int64, device="cuda") for _ in range(2))
        wa, wb = (torch.full((k,), float("nan"), dtype=torch.float32, device="cuda") for _ in range(2))
        torch.cuda.synchronize()
        for _ in range(4):       # several draws in flight on each stream
            distrl.distrl_sample(sa, d_ua, 0.4, True, ia, wa, stream=st_a)
            distrl.distrl_sample(sb, d_ub, 0.6, True, ib, wb, stream=st_b)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(ia.cpu().numpy(), sample_by_prefix(qa, ua))
        np.testing.assert_array_equal(ib.cpu().numpy(), sample_by_prefix(qb, ub))
        assert_close(wa.cpu().numpy(), oracle.is_weights(qa, ia.cpu().numpy(), 0.4, True), "is_weight a")
        assert_close(wb.cpu().numpy(), oracle.is_weights(qb, ib.cpu().numpy(), 0.6, True), "is_weight b")
    assert distrl.distrl_get_status(wsa) == 0 and distrl.distrl_get_status(wsb) == 0
    sa.close()
    sb.close()


def test_draws_over_two_shards_through_the_ordinary_entry_point():
    # one replay over two shards (two samplers, as two GPUs would hold them): the draws routed to their owner
    # with the exact local uniform come out of distrl_sample as one linear scan over all masses would give them
    from paper_2410_14803_b200 import shard
    qa, qb = _masses(300_001, 31), _masses(123_457, 32, heavy=False)
    (sa, tqa, wsa), (sb, tqb, wsb) = _build(qa), _build(qb)
    totals = [int(qa.sum(dtype=np.uint64)), int(qb.sum(dtype=np.uint64))]
    u = np.random.default_rng(33).integers(0, 2 ** 64, size=3000, dtype=np.uint64)
    owner, u_local = shard.route_draws(u.tolist(), totals)
    got = np.full(3000, -1, dtype=np.int64)
    for g, (s, base) in enumerate(((sa, 0), (sb, qa.shape[0]))):
        mine = np.array([j for j, o in enumerate(owner) if o == g])
        ul = np.array([u_local[j] for j in mine], dtype=np.uint64)
        idx, _ = _sample(s, ul, 0.4)
        got[mine] = base + idx
    np.testing.assert_array_equal(got, sample_by_prefix(np.concatenate([qa, qb]), u))
    sa.close()
    sb.close()


def test_draws_routed_on_the_device_over_three_shards():
    # the same routing done by distrl_route_draws from a device array of the shards' totals: every shard samples
    # all k positions with what the call gives it and keeps the ones it owns; together they are one linear scan
    # over the concatenated masses.  The local uniforms equal the host routine's, the owners the plain definition.
    from paper_2410_14803_b200 import shard, binding
    qs = [_masses(200_001, 41), np.array([7], dtype=np.uint32), _masses(123_457, 42, heavy=False)]
    built = [_build(q) for q in qs]
    totals = [int(q.sum(dtype=np.uint64)) for q in qs]
    d_tot = torch.zeros(3, dtype=torch.int64, device="cuda")
    for g, (s, _, _) in enumerate(built):
        distrl.distrl_sampler_total(s, d_tot[g:g + 1])
    torch.cuda.synchronize()
    assert [int(x) for x in d_tot.cpu().numpy().view(np.uint64)] == totals
    k = 5000
    u = np.random.default_rng(43).integers(0, 2 ** 64, size=k, dtype=np.uint64)
    u[:4] = [0, 2 ** 64 - 1, 1, 2 ** 63]
    grand = sum(totals)
    ys = [(int(x) * grand) >> 64 for x in u]
    u[4] = -((-(totals[0] << 64)) // grand)                    # the first threshold of the one-mass shard ...
    u[5] = -((-((totals[0] + 6) << 64)) // grand)              # ... and its last
    u[6] = -((-((totals[0] + 7) << 64)) // grand)              # the first of the third shard
    ys = [(int(x) * grand) >> 64 for x in u]
    assert ys[4] == totals[0] and ys[5] == totals[0] + 6 and ys[6] == totals[0] + 7
    d_u = dev(u.view(np.int64))
    owner_host, ul_host = shard.route_draws(u.tolist(), totals)
    before = np.concatenate([[0], np.cumsum(np.array(totals, dtype=object))])
    got = np.full(k, -1, dtype=np.int64)
    base, n_all, parts_i, parts_w = 0, sum(q.shape[0] for q in qs), [], []
    for g, (s, _, ws) in enumerate(built):
        ul = torch.empty(k, dtype=torch.int64, device="cuda")
        mine = torch.empty(k, dtype=torch.uint8, device="cuda")
        owner = torch.empty(k, dtype=torch.int32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        distrl.distrl_route_draws(d_u, d_tot, g, ul, mine, owner, status)
        idx = torch.empty(k, dtype=torch.int64, device="cuda")
        wts = torch.empty(k, dtype=torch.float32, device="cuda")
        distrl.distrl_sample(s, ul, 0.4, False, idx, wts)
        torch.cuda.synchronize()
        assert status.item() == 0 and distrl.distrl_get_status(ws) == 0
        m = mine.cpu().numpy().astype(bool)
        ow = owner.cpu().numpy()
        assert ow.tolist() == owner_host
        assert [bool(x) for x in m] == [o == g for o in owner_host]
        assert all(before[o] <= y < before[o + 1] for o, y in zip(ow, ys))
        ulh = ul.cpu().numpy().view(np.uint64)
        assert [int(x) for x in ulh[m]] == [ul_host[j] for j in np.nonzero(m)[0]]
        assert np.all(ulh[~m] == 0)
        got[m] = base + idx.cpu().numpy()[m]
        # the shard's contribution to the batch: global indices and un-normalised global weights, -1 / 0 elsewhere
        gi = torch.empty(k, dtype=torch.int64, device="cuda")
        gw = torch.empty(k, dtype=torch.float32, device="cuda")
        distrl.distrl_finish_shard_draws(mine, idx, wts, d_tot, g, qs[g].shape[0], n_all, base, 0.4, gi, gw)
        torch.cuda.synchronize()
        parts_i.append(gi.cpu().numpy())
        parts_w.append(gw.cpu().numpy())
        assert np.all(parts_i[-1][~m] == -1) and np.all(parts_w[-1][~m] == 0)
        base += qs[g].shape[0]
    q_all = np.concatenate(qs)
    np.testing.assert_array_equal(got, sample_by_prefix(q_all, u))
    # an element-wise maximum over the shards (what one all-reduce does) assembles the batch
    all_i, all_w = np.maximum.reduce(parts_i), np.maximum.reduce(parts_w)
    np.testing.assert_array_equal(all_i, got)
    assert_close(all_w, oracle.is_weights(q_all, got, 0.4, False), "global un-normalised weights")
    d_w = dev(all_w)
    distrl.distrl_normalise_weights(d_w)
    torch.cuda.synchronize()
    assert_close(d_w.cpu().numpy(), oracle.is_weights(q_all, got, 0.4, True), "global weights / batch maximum")
    assert d_w.max().item() == 1.0
    # totals that do not fit 64 bits, or no mass at all: reported, nothing owned
    for bad in ([2 ** 63, 2 ** 63, 5], [0, 0, 0]):
        d_bad = dev(np.array(bad, dtype=np.uint64).view(np.int64))
        ul = torch.full((k,), 9, dtype=torch.int64, device="cuda")
        mine = torch.full((k,), 9, dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        distrl.distrl_route_draws(d_u, d_bad, 1, ul, mine, None, status)
        torch.cuda.synchronize()
        assert status.item() == binding.ERR_SIZE
        assert int(ul.abs().sum().item()) == 0 and int(mine.sum().item()) == 0
    lib = binding._load()
    assert lib.distrl_route_draws(d_u.data_ptr(), k, d_tot.data_ptr(), 0, 0, ul.data_ptr(), mine.data_ptr(), None, None, None) == binding.ERR_PARAM
    assert lib.distrl_route_draws(d_u.data_ptr(), k, d_tot.data_ptr(), 3, 3, ul.data_ptr(), mine.data_ptr(), None, None, None) == binding.ERR_PARAM
    assert lib.distrl_route_draws(d_u.data_ptr(), k, None, 3, 0, ul.data_ptr(), mine.data_ptr(), None, None, None) == binding.ERR_NULL
    assert lib.distrl_route_draws(None, 0, None, 3, 0, None, None, None, None, None) == binding.OK
    for s, _, _ in built:
        s.close()


def test_sample_over_shards_with_one_rank_is_the_ordinary_draw():
    from paper_2410_14803_b200 import shard
    q = _masses(77_777, 51)
    s, tq, ws = _build(q)
    u = np.random.default_rng(52).integers(0, 2 ** 64, size=2000, dtype=np.uint64)
    idx = torch.empty(2000, dtype=torch.int64, device="cuda")
    wts = torch.empty(2000, dtype=torch.float32, device="cuda")
    shard.sample_over_shards(s, q.shape[0], dev(u.view(np.int64)), 0.4, idx, wts)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(idx.cpu().numpy(), sample_by_prefix(q, u))
    assert_close(wts.cpu().numpy(), oracle.is_weights(q, idx.cpu().numpy(), 0.4, True), "weights")
    assert distrl.distrl_get_status(ws) == 0
    s.close()


@pytest.mark.parametrize("k", [1, 2, 3, 255, 4096, 100_003])
def test_stratified_uniforms_and_a_stratified_batch(k):
    rng = np.random.default_rng(k)
    u = rng.integers(0, 2 ** 64, size=k, dtype=np.uint64)
    u[0], u[-1] = 0, 2 ** 64 - 1
    d_u = dev(u.view(np.int64))
    out = torch.empty_like(d_u)
    distrl.distrl_stratify_uniforms(d_u, out)
    want = oracle.stratify(u)
    np.testing.assert_array_equal(out.cpu().numpy().view(np.uint64), want)
    distrl.distrl_stratify_uniforms(d_u, d_u)                                    # in place
    np.testing.assert_array_equal(d_u.cpu().numpy().view(np.uint64), want)
    q = _masses(50_000, 5)
    s, tq, ws = _build(q)
    idx, wts = _sample(s, want, 0.4)
    np.testing.assert_array_equal(idx, sample_by_prefix(q, want))
    assert np.all(np.diff(idx) >= 0)                                             # one draw per stratum, in order
    s.close()


def test_sampling_brute_force_on_device():
    # every threshold y in [0, total) must land on index i exactly q_i times
    q = np.array([3, 1, 7, 1, 1, 12, 5] * 40, dtype=np.uint32)
    total = int(q.sum())
    u = np.array([-((-y * (1 << 64)) // total) for y in range(total)], dtype=np.uint64)
    s, tq, ws = _build(q)
    idx, _ = _sample(s, u, 0.4)
    np.testing.assert_array_equal(np.bincount(idx, minlength=q.shape[0]), q)
    s.close()


def _update(s, w_cfg, idx, nd, lp, lm, ent):
    k = idx.shape[0]
    mass = torch.full((k,), float("nan"), dtype=torch.float32, device="cuda")
    distrl.distrl_update_priorities(s, dev(idx), dev(nd), lp, lm, ent, w_cfg, mass)
    torch.cuda.synchronize()
    return mass.cpu().numpy()


@pytest.mark.parametrize("index,k", [(0, 32), (1, 256), (1, 9000), (2, 1024), (2, 20000)])
def test_update_equals_rebuild(index, k):
    w = synth.make_workload(index)
    a = w.arrays
    cfg = prio_cfg_of(w)
    _, _, dl = oracle.retrace(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"],
                              w.gamma, w.lam)
    mass0 = oracle.priority_mass(dl, a["logp_target"], a["logp_behaviour"], a["entropy"], w.w_td, w.w_rho, w.w_ent,
                                 w.rho_clip, w.alpha)
    q = oracle.quantise(mass0.astype(np.float32), w.scale)
    s, tq, ws = _build(q)
    lp, lm, ent = dev(a["logp_target"]), dev(a["logp_behaviour"]), dev(a["entropy"])
    for rnd in range(3):
        u = synth.uniforms(w, rnd, k)
        idx, wts = _sample(s, u, w.beta)
        np.testing.assert_array_equal(idx, sample_by_prefix(q, u))
        assert_close(wts, oracle.is_weights(q, idx, w.beta, True), "is_weight")
        if rnd == 0:   # force duplicates, also across the chunk boundary of large batches
            idx[k // 2:k // 2 + 5] = idx[0]
            idx[-1] = idx[1]
        nd = synth.fresh_abs_delta(w, rnd, k)
        gmass = _update(s, cfg, idx, nd, lp, lm, ent)
        q_ref = q.copy()
        omass = oracle.update(q_ref, idx, nd, a["logp_target"], a["logp_behaviour"], a["entropy"], w.w_td, w.w_rho,
                              w.w_ent, w.rho_clip, w.alpha, w.scale)
        assert_close(gmass, omass, "update mass")
        # integer stage: sequential requantisation of the device's own masses
        oracle.update_from_mass(q, idx, gmass, w.scale)
        np.testing.assert_array_equal(tq.cpu().numpy().view(np.uint32), q)
        assert np.all(np.abs(q.astype(np.int64) - q_ref.astype(np.int64)) <= np.maximum(1, 4e-7 * q_ref))
        _check_tree(s, q)                      # incremental repair == rebuild from scratch
    assert distrl.distrl_get_status(ws) == 0
    s.close()


def test_update_rejects_bad_index_but_applies_the_rest():
    q = _masses(5000, 1)
    s, tq, ws = _build(q)
    z = torch.zeros(5000, dtype=torch.float32, device="cuda")
    idx = np.array([7, 5000, -1, 9], dtype=np.int64)
    nd = np.array([4.0, 1.0, 1.0, 9.0], dtype=np.float32)
    _update(s, distrl.make_prio_cfg(1.0, 0.0, 0.0, 2.0, 0.5, 2.0 ** 20), idx, nd, z, z, z)
    assert distrl.distrl_get_status(ws) == distrl.binding.ERR_INDEX
    q[7] = 2 << 20
    q[9] = 3 << 20
    np.testing.assert_array_equal(tq.cpu().numpy().view(np.uint32), q)
    _check_tree(s, q)
    assert distrl.distrl_get_status(ws) == 0       # reading cleared it
    s.close()


def test_full_path_rounds_config3():
    """Workload 3 end to end at full size in the call sequence the benchmark times."""
    w = synth.make_workload(3)
    a = w.arrays
    n = w.n
    out = check_retrace(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"],
                        w.gamma, w.lam)
    delta = (out["td_delta"] * synth.heavy_tail_scale(w)).astype(np.float32)
    cfg = prio_cfg_of(w)
    lp, lm, ent = dev(a["logp_target"]), dev(a["logp_behaviour"]), dev(a["entropy"])
    mass = torch.empty(n, dtype=torch.float32, device="cuda")
    tq = torch.empty(n, dtype=torch.int32, device="cuda")
    distrl.distrl_compute_priorities(dev(delta), lp, lm, ent, cfg, mass, tq)
    q = oracle.quantise(mass.cpu().numpy(), w.scale)
    np.testing.assert_array_equal(tq.cpu().numpy().view(np.uint32), q)
    ws = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    s = distrl.distrl_build_sampler(tq, ws)
    _check_tree(s, q)
    for rnd in range(w.rounds):
        u = synth.uniforms(w, rnd)
        idx, wts = _sample(s, u, w.beta)
        np.testing.assert_array_equal(idx, sample_by_prefix(q, u))
        if rnd in (0, 57):
            np.testing.assert_array_equal(idx[:6], oracle.sample_linear(q, u[:6]))
        assert_close(wts, oracle.is_weights(q, idx, w.beta, True), "is_weight")
        nd = synth.fresh_abs_delta(w, rnd)
        gmass = _update(s, cfg, idx, nd, lp, lm, ent)
        oracle.update_from_mass(q, idx, gmass, w.scale)
    np.testing.assert_array_equal(tq.cpu().numpy().view(np.uint32), q)
    _check_tree(s, q)
    assert distrl.distrl_get_status(ws) == 0
    s.close()


# -------------------------------------------------------------- token level ---

def _token_case(off, sto, tok_p, tok_m, seed, gamma=0.99, lam=0.95, **kw):
    n = int(off[-1])
    rng = np.random.default_rng(seed)
    r = rng.normal(0, 1, n).astype(np.float32)
    V = rng.random(n, dtype=np.float32)
    lp = oracle.token_logp(sto, oracle.bf16_bits_to_f64(tok_p))
    lm = oracle.token_logp(sto, oracle.bf16_bits_to_f64(tok_m))
    out = gpu_retrace(off, r, V, None, None, gamma, lam, tokens=(sto, tok_p, tok_m), want_logp=True, **kw)
    assert out["status"] == 0
    vt, adv, dl = oracle.retrace(off, r, V, lp, lm, gamma, lam)
    assert_close(out["logp_target"], lp, "token logp_target")
    assert_close(out["logp_behaviour"], lm, "token logp_behaviour")
    assert_close(out["v_target"], vt, "v_target")
    assert_close(out["advantage"], adv, "advantage")
    assert_close(out["td_delta"], dl, "td_delta")


@pytest.mark.parametrize("n", [1000, 50000, 300001])
def test_token_level_workload(n):
    w = synth.make_workload(4, n_override=n)
    a = w.arrays
    _token_case(a["traj_offsets"], a["step_token_offsets"], a["tok_logp_target"], a["tok_logp_behaviour"], n,
                w.gamma, w.lam)


@pytest.mark.parametrize("counts", ["all32", "zeros_and_ones", "one_huge", "wide"])
def test_token_level_count_extremes(counts):
    # all32: every tile owns more tokens than one staging pass holds (18432); zeros_and_ones: empty steps;
    # one_huge: a single step with 70,000 tokens; wide: counts up to 200.
    n = 5000
    rng = np.random.default_rng(17)
    cnt = {"all32": np.full(n, 32), "zeros_and_ones": rng.integers(0, 2, n),
           "one_huge": np.where(np.arange(n) == 2500, 70000, 1), "wide": rng.integers(0, 201, n)}[counts]
    sto = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int64)
    nt = int(sto[-1])
    shrink = np.float32(max(1, cnt.max() // 32))     # keep the per-step sums in a sane range
    tok_m = synth.f32_to_bf16_bits((rng.standard_normal(nt) * 0.3 - 0.3).astype(np.float32) / shrink)
    tok_p = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(tok_m) +
                                   (rng.standard_normal(nt) * 0.05).astype(np.float32) / shrink)
    off = synth.adversarial_offsets("long_mixed", n, tile=1024)
    _token_case(off, sto, tok_p, tok_m, 3)


@pytest.mark.parametrize("n", [1, 2, 511, 512, 513, 544, 545, 546, 1023, 1024, 1025, 1057, 1569, 4097])
@pytest.mark.parametrize("kind", ["single", "ones", "tile_straddle", "long_mixed"])
def test_token_level_tile_edges(n, kind):
    # sizes around the 512-step tiles and the 32-step halo of the pipelined token kernel: which tiles are
    # staged, which are taken straight from global memory, where the buffer ends inside a halo
    rng = np.random.default_rng(1000 + n)
    cnt = rng.integers(1, 33, n)
    sto = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int64)
    nt = int(sto[-1])
    tok_m = synth.f32_to_bf16_bits((rng.standard_normal(nt) * 0.3 - 0.3).astype(np.float32))
    tok_p = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(tok_m) + (rng.standard_normal(nt) * 0.05).astype(np.float32))
    off = synth.adversarial_offsets(kind, n, tile=512)
    _token_case(off, sto, tok_p, tok_m, n)


@pytest.mark.parametrize("n", [1, 2, 31, 32, 33, 511, 512, 513, 544, 545, 546, 1023, 1024, 1025, 1057, 1569, 4097, 40001])
@pytest.mark.parametrize("kind", ["single", "ones", "tile_straddle", "long_mixed"])
def test_token_level_tile_edges_dense_instance(n, kind):
    # the same sizes with 18 to 40 tokens per step: the instance with one step per lane and sixteen token warps
    rng = np.random.default_rng(2000 + n)
    cnt = rng.integers(18, 41, n)
    cnt[rng.random(n) < 0.05] = 0
    sto = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int64)
    nt = int(sto[-1])
    tok_m = synth.f32_to_bf16_bits((rng.standard_normal(nt) * 0.3 - 0.3).astype(np.float32) / np.float32(2))
    tok_p = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(tok_m) + (rng.standard_normal(nt) * 0.05).astype(np.float32))
    off = synth.adversarial_offsets(kind, n, tile=512)
    _token_case(off, sto, tok_p, tok_m, n)


@pytest.mark.parametrize("counts", ["first_vector_only", "sparse", "near_capacity", "over_capacity_some"])
def test_token_level_staging_corners(counts):
    # first_vector_only: all tokens of a tile inside one 16-byte vector; sparse: most steps empty;
    # near_capacity: tiles just below what a stage holds; over_capacity_some: staged and direct tiles mixed
    n = 6000
    rng = np.random.default_rng(23)
    cnt = {"first_vector_only": (np.arange(n) % 512 == 3).astype(np.int64) * 5,
           "sparse": (rng.random(n) < 0.03).astype(np.int64) * rng.integers(1, 33, n),
           "near_capacity": np.full(n, 18),
           "over_capacity_some": np.where((np.arange(n) // 700) % 2 == 0, 8, 31)}[counts]
    sto = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int64)
    nt = int(sto[-1])
    tok_m = synth.f32_to_bf16_bits((rng.standard_normal(nt) * 0.3 - 0.3).astype(np.float32))
    tok_p = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(tok_m) + (rng.standard_normal(nt) * 0.05).astype(np.float32))
    off = synth.adversarial_offsets("long_mixed", n, tile=512)
    _token_case(off, sto, tok_p, tok_m, 5)


@pytest.mark.parametrize("lo,hi", [(20, 33), (17, 19), (16, 18), (32, 36), (34, 36), (36, 48), (0, 70)])
def test_token_level_dense_buffers(lo, hi):
    # mean token counts around and above what a stage of the pipelined kernel holds (about 17 per step) and what
    # a stage of its instance for dense buffers holds (about 34): the mask kernel's verdict on the mean sends the
    # call to one of them or to the general kernel; whichever it is, the results are the oracle's
    n = 120001
    rng = np.random.default_rng(lo * 100 + hi)
    cnt = rng.integers(lo, hi, n)
    sto = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int64)
    nt = int(sto[-1])
    tok_m = synth.f32_to_bf16_bits((rng.standard_normal(nt) * 0.3 - 0.3).astype(np.float32) / np.float32(2))
    tok_p = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(tok_m) + (rng.standard_normal(nt) * 0.05).astype(np.float32))
    off = synth.adversarial_offsets("long_mixed", n, tile=512)
    _token_case(off, sto, tok_p, tok_m, 11)


def test_token_level_bad_step_offsets_are_reported_not_fatal():
    n = 3000
    rng = np.random.default_rng(3)
    cnt = rng.integers(1, 33, n)
    sto = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int64)
    nt = int(sto[-1])
    tok = synth.f32_to_bf16_bits((rng.standard_normal(nt) * 0.3 - 0.3).astype(np.float32))
    bad = sto.copy()
    bad[700] = bad[699] - 40          # a decreasing pair inside a staged tile
    bad[2900] = bad[2899] - 3         # and one inside the last, direct tile
    off = synth.adversarial_offsets("long_mixed", n, tile=512)
    r = rng.normal(0, 1, n).astype(np.float32)
    V = rng.random(n, dtype=np.float32)
    out = gpu_retrace(off, r, V, None, None, 0.99, 0.95, tokens=(bad, tok, tok))
    assert out["status"] == distrl.binding.ERR_OFFSETS
    good = gpu_retrace(off, r, V, None, None, 0.99, 0.95, tokens=(sto, tok, tok))
    assert good["status"] == 0


@pytest.mark.parametrize("pattern", ["workload", "alternating", "dense_alternating"])
def test_token_level_repeated_runs_agree_bit_for_bit(pattern):
    # The token kernel's warps hand data to one another through shared-memory buffers guarded by
    # mbarriers, and drift apart by up to a tile: forty runs on the same inputs and workspace must
    # agree bit for bit.  "alternating": tiles of one token per step alternate with tiles of 17, so
    # that the same shared-memory positions belong to different warps in consecutive tiles;
    # "dense_alternating": tiles of 12 and of 36 tokens per step, which the instance for dense buffers takes.
    if pattern == "workload":
        w = synth.make_workload(4, n_override=1500001)
        a = w.arrays
        n, off, sto, tp, tm = w.n, a["traj_offsets"], a["step_token_offsets"], a["tok_logp_target"], a["tok_logp_behaviour"]
    else:
        n = 1200000 if pattern == "alternating" else 600000
        rng = np.random.default_rng(12)
        cnt = np.where((np.arange(n) // 512) % 2 == 0, 1, 17) if pattern == "alternating" else \
            np.where((np.arange(n) // 512) % 2 == 0, 12, 36)
        sto = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int64)
        nt = int(sto[-1])
        tm = synth.f32_to_bf16_bits((rng.standard_normal(nt) * 0.3 - 0.3).astype(np.float32) / np.float32(2))
        tp = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(tm) + (rng.standard_normal(nt) * 0.05).astype(np.float32))
        off = synth.adversarial_offsets("long_mixed", n, tile=512)
    rng = np.random.default_rng(8)
    t_off, t_r, t_V = dev(off), dev(rng.normal(0, 1, n).astype(np.float32)), dev(rng.random(n, dtype=np.float32))
    t_sto, t_tp, t_tm = dev(sto), dev(tp, torch.bfloat16), dev(tm, torch.bfloat16)
    batch = distrl.make_batch(t_off, t_r, t_V, None, None, None, t_sto, t_tp, t_tm)
    ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    first = None
    for _ in range(40):
        out = [torch.full((n,), float("nan"), dtype=torch.float32, device="cuda") for _ in range(5)]
        distrl.distrl_retrace_targets(batch, 0.99, 0.95, *out, workspace=ws)
        got = [o.view(torch.int32) for o in out]
        if first is None:
            first = got
        for g, f in zip(got, first):
            assert torch.equal(g, f)                  # compared on the device: bit patterns
    assert distrl.distrl_get_status(ws) == 0
    lp = oracle.token_logp(sto, oracle.bf16_bits_to_f64(tp))
    assert_close(first[3].view(torch.float32).cpu().numpy(), lp, "token logp_target")


def test_token_level_single_token_steps_equal_plain_logp():
    # one token per step: the token path must agree with the fp32-logp path on the same numbers
    n = 30000
    rng = np.random.default_rng(21)
    off = synth.adversarial_offsets("long_mixed", n)
    tok_m = synth.f32_to_bf16_bits(rng.normal(-5, 2, n).astype(np.float32))
    tok_p = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(tok_m) + rng.normal(0, 0.5, n).astype(np.float32))
    sto = np.arange(n + 1, dtype=np.int64)
    r = rng.normal(0, 1, n).astype(np.float32)
    V = rng.random(n, dtype=np.float32)
    a = gpu_retrace(off, r, V, None, None, 0.99, 0.95, tokens=(sto, tok_p, tok_m))
    b = gpu_retrace(off, r, V, synth.bf16_bits_to_f32(tok_p), synth.bf16_bits_to_f32(tok_m), 0.99, 0.95)
    # the token path takes step sums as differences of short running sums: a few ulp of the 16-token sums
    for key in ("v_target", "advantage", "td_delta"):
        assert_close(a[key], b[key].astype(np.float64), key, tol=1e-5)


def test_token_level_unaligned_token_arrays():
    w = synth.make_workload(4, n_override=20000)
    a = w.arrays
    sto, tp, tm = a["step_token_offsets"], a["tok_logp_target"], a["tok_logp_behaviour"]
    n = w.n
    rng = np.random.default_rng(2)
    r = rng.normal(0, 1, n).astype(np.float32)
    V = rng.random(n, dtype=np.float32)
    t_off, t_r, t_V, t_sto = dev(a["traj_offsets"]), dev(r), dev(V), dev(sto)
    bufp = torch.empty(tp.shape[0] + 1, dtype=torch.bfloat16, device="cuda")
    bufm = torch.empty(tp.shape[0] + 1, dtype=torch.bfloat16, device="cuda")
    bufp[1:].copy_(torch.from_numpy(tp).view(torch.bfloat16))
    bufm[1:].copy_(torch.from_numpy(tm).view(torch.bfloat16))
    batch = distrl.make_batch(t_off, t_r, t_V, None, None, None, t_sto, bufp[1:], bufm[1:])
    vt = torch.empty(n, dtype=torch.float32, device="cuda")
    adv = torch.empty(n, dtype=torch.float32, device="cuda")
    ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    distrl.distrl_retrace_targets(batch, w.gamma, w.lam, vt, adv, workspace=ws)
    assert distrl.distrl_get_status(ws) == 0
    lp = oracle.token_logp(sto, oracle.bf16_bits_to_f64(tp))
    lm = oracle.token_logp(sto, oracle.bf16_bits_to_f64(tm))
    o_vt, o_adv, _ = oracle.retrace(a["traj_offsets"], r, V, lp, lm, w.gamma, w.lam)
    assert_close(vt.cpu().numpy(), o_vt, "v_target")
    assert_close(adv.cpu().numpy(), o_adv, "advantage")


# ------------------------------------------------------- circular overwrite ---

@pytest.mark.parametrize("n,head,k", [(100, 90, 30), (100, 0, 100), (5000, 4990, 4000), (5000, 17, 12000),
                                      (1 << 20, (1 << 20) - 5, 4096), (300001, 123, 70000)])
def test_replay_overwrite_equals_rebuild(n, head, k):
    q = _masses(n, 5)
    s, tq, ws = _build(q)
    new_q = _masses(k, 6, heavy=False)
    distrl.distrl_replay_overwrite(s, head, dev(new_q.view(np.int32)))
    torch.cuda.synchronize()
    oracle.replay_overwrite(q, head, new_q)
    np.testing.assert_array_equal(tq.cpu().numpy().view(np.uint32), q)
    _check_tree(s, q)
    u = np.random.default_rng(n).integers(0, 1 << 64, size=200, dtype=np.uint64)
    idx, _ = _sample(s, u, 0.4)
    np.testing.assert_array_equal(idx, sample_by_prefix(q, u))
    assert distrl.distrl_get_status(ws) == 0
    s.close()


# ---------------------------------------------------------------- fused pass ---

@pytest.mark.parametrize("index,with_ent,with_scale,n_over", [(0, True, False, None), (1, True, True, None),
                                                              (1, False, False, None), (2, True, True, None),
                                                              (3, True, True, 3000001)])
def test_fused_retrace_priorities_build(index, with_ent, with_scale, n_over):
    w = synth.make_workload(index, n_override=n_over)
    a = w.arrays
    n = w.n
    cfg = prio_cfg_of(w)
    scale = synth.heavy_tail_scale(w) if with_scale else None
    t = [dev(a["traj_offsets"]), dev(a["rewards"]), dev(a["values"]), dev(a["logp_target"]), dev(a["logp_behaviour"])]
    batch = distrl.make_batch(*t)
    t_ent = dev(a["entropy"]) if with_ent else None
    t_sc = dev(scale) if with_scale else None
    vt, adv, dl, mass = (torch.full((n,), float("nan"), dtype=torch.float32, device="cuda") for _ in range(4))
    tq = torch.zeros(n, dtype=torch.int32, device="cuda")
    ws_r = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    ws_s = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(n))
    distrl.distrl_workspace_init(ws_r)
    distrl.distrl_workspace_init(ws_s)
    s = distrl.distrl_retrace_priorities_build(batch, w.gamma, w.lam, t_ent, t_sc, cfg, vt, adv, dl, tq, mass,
                                               retrace_workspace=ws_r, sampler_workspace=ws_s)
    assert distrl.distrl_get_status(ws_r) == 0
    o_vt, o_adv, o_dl = oracle.retrace(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"],
                                       a["logp_behaviour"], w.gamma, w.lam)
    assert_close(vt.cpu().numpy(), o_vt, "v_target")
    assert_close(adv.cpu().numpy(), o_adv, "advantage")
    assert_close(dl.cpu().numpy(), o_dl, "td_delta")
    d_in = o_dl * scale.astype(np.float64) if with_scale else o_dl
    o_mass = oracle.priority_mass(d_in, a["logp_target"], a["logp_behaviour"], a["entropy"] if with_ent else None,
                                  w.w_td, w.w_rho, w.w_ent, w.rho_clip, w.alpha)
    assert_close(mass.cpu().numpy(), o_mass, "prio_mass")
    q = tq.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(q, oracle.quantise(mass.cpu().numpy(), w.scale))
    _check_tree(s, q)
    u = synth.uniforms(w, 0)
    idx, wts = _sample(s, u, w.beta)
    np.testing.assert_array_equal(idx, sample_by_prefix(q, u))
    assert_close(wts, oracle.is_weights(q, idx, w.beta, True), "is_weight")
    # a refresh round on the fused sampler keeps the tree exact
    nd = synth.fresh_abs_delta(w, 0)
    gm = _update(s, cfg, idx, nd, t[3], t[4], t_ent if with_ent else None)
    oracle.update_from_mass(q, idx, gm, w.scale)
    np.testing.assert_array_equal(tq.cpu().numpy().view(np.uint32), q)
    _check_tree(s, q)
    assert distrl.distrl_get_status(ws_s) == 0
    s.close()


def test_fused_pass_quantiser_edges():
    # one-step trajectories with V = 0, weights (1, 0, 0), alpha = 0.5: the priority is |r| itself, so the
    # rewards below walk the fused epilogue through zero, a denormal, the ties of the quantiser, values
    # that saturate it, infinity and NaN.  Whatever mass the device reports, its mass must be Q of it.
    special = np.array([0.0, 1e-45, 1e-38, 2.0 ** -42, (1.5 * 2.0 ** -20) ** 2, (2.5 * 2.0 ** -20) ** 2, 1.0, 4096.0 ** 2,
                        1.7e7, 3e38, np.inf, np.nan, -3.0], dtype=np.float32)
    n = 5000
    rng = np.random.default_rng(4)
    r = (rng.random(n, dtype=np.float32) * 4).astype(np.float32)
    r[:special.shape[0]] = special
    r[2048:2048 + special.shape[0]] = special[::-1]
    off = np.arange(n + 1, dtype=np.int64)
    z = np.zeros(n, dtype=np.float32)
    t = [dev(off), dev(r), dev(z), dev(z), dev(z)]
    vt, adv, mass = (torch.full((n,), float("nan"), dtype=torch.float32, device="cuda") for _ in range(3))
    tq = torch.zeros(n, dtype=torch.int32, device="cuda")
    ws_r = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    ws_s = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(n))
    distrl.distrl_workspace_init(ws_r)
    distrl.distrl_workspace_init(ws_s)
    cfg = distrl.make_prio_cfg(1.0, 0.0, 0.0, 2.0, 0.5, 2.0 ** 20)
    s = distrl.distrl_retrace_priorities_build(distrl.make_batch(*t), 0.9, 0.9, None, None, cfg, vt, adv, None, tq, mass,
                                               retrace_workspace=ws_r, sampler_workspace=ws_s)
    assert distrl.distrl_get_status(ws_r) == 0
    q = tq.cpu().numpy().view(np.uint32)
    m = mass.cpu().numpy()
    np.testing.assert_array_equal(q, oracle.quantise(m, 2.0 ** 20))
    assert q.min() >= 1
    finite = np.isfinite(r) & (r >= 0)
    assert_close(m[finite], np.sqrt(r[finite].astype(np.float64)), "mass of the finite rewards")
    assert q[0] == 1 and q[6] == 1 << 20 and q[7] == 4294967295 and q[10] == 4294967295 and q[11] == 1
    _check_tree(s, q)
    s.close()


def test_fused_pass_refuses_what_it_does_not_serve():
    w = synth.make_workload(0)
    a = w.arrays
    n = w.n
    t = [dev(a["traj_offsets"]), dev(a["rewards"]), dev(a["values"]), dev(a["logp_target"]), dev(a["logp_behaviour"])]
    boot = torch.zeros(w.m, dtype=torch.float32, device="cuda")
    batch = distrl.make_batch(*t, boot)
    out = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(2)]
    tq = torch.zeros(n, dtype=torch.int32, device="cuda")
    ws_r = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    ws_s = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(n))
    with pytest.raises(distrl.DistrlError) as e:
        distrl.distrl_retrace_priorities_build(batch, 0.9, 0.9, None, None, prio_cfg_of(w), out[0], out[1], None, tq,
                                               None, retrace_workspace=ws_r, sampler_workspace=ws_s)
    assert e.value.code == distrl.binding.ERR_PARAM


def test_rounds_replayed_from_a_cuda_graph_match_the_oracle():
    """The benchmark records the sample -> refresh rounds once into a CUDA graph and replays it; the
    replayed launches must leave exactly the state the oracle reaches by running the rounds in order."""
    w = synth.make_workload(2)
    a = w.arrays
    n, k, R = w.n, w.batch, 6
    cfg = prio_cfg_of(w)
    _, _, dl = oracle.retrace(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"],
                              w.gamma, w.lam)
    mass0 = oracle.priority_mass(dl, a["logp_target"], a["logp_behaviour"], a["entropy"], w.w_td, w.w_rho, w.w_ent,
                                 w.rho_clip, w.alpha)
    q = oracle.quantise(mass0.astype(np.float32), w.scale)
    s, tq, ws = _build(q)
    lp, lm, ent = dev(a["logp_target"]), dev(a["logp_behaviour"]), dev(a["entropy"])
    us = np.stack([synth.uniforms(w, r) for r in range(R)])
    nds = np.stack([synth.fresh_abs_delta(w, r) for r in range(R)])
    d_u, d_nd = dev(us.view(np.int64)), dev(nds)
    idx = torch.empty((R, k), dtype=torch.int64, device="cuda")
    wts = torch.empty((R, k), dtype=torch.float32, device="cuda")
    mass = torch.empty((R, k), dtype=torch.float32, device="cuda")

    def rounds():
        for r in range(R):
            distrl.distrl_sample(s, d_u[r], w.beta, True, idx[r], wts[r])
            distrl.distrl_update_priorities(s, idx[r], d_nd[r], lp, lm, ent, cfg, mass[r])

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        rounds()                                   # first use outside capture
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    # oracle: the same six rounds, in order, from the device's own masses
    def oracle_rounds(qq):
        for r in range(R):
            np.testing.assert_array_equal(idx[r].cpu().numpy(), sample_by_prefix(qq, us[r]))
            assert_close(wts[r].cpu().numpy(), oracle.is_weights(qq, idx[r].cpu().numpy(), w.beta, True), "is_weight")
            oracle.update_from_mass(qq, idx[r].cpu().numpy(), mass[r].cpu().numpy(), w.scale)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        rounds()
    torch.cuda.synchronize()
    # state now: rounds ran once (eagerly; capture itself launches nothing)
    q1 = q.copy()
    # replay twice; after each replay the recorded outputs describe that replay
    for _ in range(2):
        q_before = tq.cpu().numpy().view(np.uint32).copy()
        graph.replay()
        torch.cuda.synchronize()
        qq = q_before.copy()
        oracle_rounds(qq)
        np.testing.assert_array_equal(tq.cpu().numpy().view(np.uint32), qq)
        _check_tree(s, qq)
    assert distrl.distrl_get_status(ws) == 0
    del q1
    s.close()


# ------------------------------------------------- what a drawn batch carries ---

def _policy_arrays(n, seed):
    rng = np.random.default_rng(seed)
    lm = rng.normal(-5, 2, n).astype(np.float32)
    lp = (lm + rng.normal(0, 0.7, n)).astype(np.float32)
    adv = rng.normal(0, 2, n).astype(np.float32)
    return lp, lm, adv


@pytest.mark.parametrize("n", [1, 3, 4, 1023, 1024, 1025, 303_107, (1 << 21) + 3])
@pytest.mark.parametrize("weights", [False, True])
@pytest.mark.parametrize("misalign", [False, True])
def test_actor_coefficients_whole_buffer(n, weights, misalign):
    from helpers import dev_misaligned
    up = dev_misaligned if misalign else dev
    lp, lm, adv = _policy_arrays(n, n)
    w = np.random.default_rng(n + 1).uniform(0.01, 1.0, n).astype(np.float32) if weights else None
    coef = torch.full((n + 1,), float("nan"), dtype=torch.float32, device="cuda")
    out = coef[1:] if misalign else coef[:n]
    distrl.distrl_actor_coefficients(up(lp), up(lm), up(adv), out, is_weight=up(w) if weights else None)
    torch.cuda.synchronize()
    assert_close(out.cpu().numpy(), oracle.actor_coefficients(lp, lm, adv, None, w), "actor coefficient", tol=1e-5)
    if not misalign:
        assert np.isnan(coef[n].item())                                   # nothing written past the end


@pytest.mark.parametrize("index", [1, 2])
def test_actor_coefficients_of_a_prioritised_draw(index):
    # the whole chain: Retrace advantages -> priorities -> draw -> coefficients of the drawn batch
    w = synth.make_workload(index)
    a = w.arrays
    g = gpu_retrace(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"], w.gamma, w.lam)
    adv = g["advantage"]
    mass, q = _gpu_priorities(w, g["td_delta"])
    s, tq, ws = _build(q)
    u = synth.uniforms(w, 0)
    idx, wts = _sample(s, u, w.beta)
    coef = torch.full((idx.shape[0],), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    distrl.distrl_actor_coefficients(dev(a["logp_target"]), dev(a["logp_behaviour"]), dev(adv), coef, idx=dev(idx),
                                     is_weight=dev(wts), status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    ref = oracle.actor_coefficients(a["logp_target"], a["logp_behaviour"], adv, idx, wts)
    assert_close(coef.cpu().numpy(), ref, "actor coefficient of the batch", tol=1e-5)
    s.close()


def test_actor_coefficients_edges():
    lp, lm, adv = _policy_arrays(100, 3)
    t = [dev(lp), dev(lm), dev(adv)]
    # empty batch: nothing launched, nothing written
    distrl.distrl_actor_coefficients(*t, torch.empty(0, dtype=torch.float32, device="cuda"),
                                     idx=torch.empty(0, dtype=torch.int64, device="cuda"))
    # indices outside the buffer: flagged, NaN, neighbours untouched and correct
    idx = np.array([5, -1, 99, 100, 0, 1 << 40], dtype=np.int64)
    coef = torch.zeros(idx.shape[0], dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    distrl.distrl_actor_coefficients(*t, coef, idx=dev(idx), status=status)
    torch.cuda.synchronize()
    c = coef.cpu().numpy()
    good = np.array([0, 2, 4])
    assert np.all(np.isnan(c[[1, 3, 5]]))
    assert_close(c[good], oracle.actor_coefficients(lp, lm, adv, idx[good]), "in-range entries", tol=1e-5)
    from paper_2410_14803_b200 import binding
    assert status.item() == binding.ERR_INDEX
    # whole-buffer form needs k == n; required pointers are checked on the host
    lib = binding._load()
    p = [x.data_ptr() for x in t]
    assert lib.distrl_actor_coefficients(100, None, 7, p[0], p[1], p[2], None, coef.data_ptr(), None, None) == binding.ERR_SIZE
    assert lib.distrl_actor_coefficients(100, None, 100, p[0], None, p[2], None, coef.data_ptr(), None, None) == binding.ERR_NULL
    assert lib.distrl_actor_coefficients(100, None, 100, p[0], p[1] + 2, p[2], None, coef.data_ptr(), None, None) == binding.ERR_ALIGN


def test_trajectory_level_draw_returns_transition_ranges():
    w = synth.make_workload(1)
    a = w.arrays
    off = np.sort(np.concatenate([a["traj_offsets"], a["traj_offsets"][[7, 7, 300]]]))   # with empty trajectories
    m = off.shape[0] - 1
    delta = np.random.default_rng(4).normal(0, 1, w.n).astype(np.float32)
    q = torch.empty(m, dtype=torch.int32, device="cuda")
    distrl.distrl_compute_priorities_traj(dev(off), dev(delta), dev(a["logp_target"]), dev(a["logp_behaviour"]),
                                          dev(a["entropy"]), prio_cfg_of(w), None, q)
    qh = q.cpu().numpy().view(np.uint32)
    s, tq, ws = _build(qh)
    u = np.random.default_rng(9).integers(0, 1 << 64, size=777, dtype=np.uint64)
    idx, _ = _sample(s, u, w.beta)
    np.testing.assert_array_equal(idx, sample_by_prefix(qh, u))
    b = torch.full((777,), -7, dtype=torch.int64, device="cuda")
    e = torch.full((777,), -7, dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    distrl.distrl_trajectory_ranges(dev(off), dev(idx), b, e, status=status)
    torch.cuda.synchronize()
    rb, re = oracle.trajectory_ranges(off, idx)
    np.testing.assert_array_equal(b.cpu().numpy(), rb)
    np.testing.assert_array_equal(e.cpu().numpy(), re)
    assert status.item() == 0
    bad = np.array([0, m, -1, m - 1], dtype=np.int64)
    b2 = torch.zeros(4, dtype=torch.int64, device="cuda")
    e2 = torch.zeros(4, dtype=torch.int64, device="cuda")
    distrl.distrl_trajectory_ranges(dev(off), dev(bad), b2, e2, status=status)
    torch.cuda.synchronize()
    assert b2.cpu().tolist() == [int(off[0]), -1, -1, int(off[m - 1])]
    assert e2.cpu().tolist() == [int(off[1]), -1, -1, int(off[m])]
    assert status.item() != 0
    s.close()


# ------------------------------------------------------------ trajectory filter ---

@pytest.mark.parametrize("name,lens", list(_traj_layouts()), ids=[nm for nm, _ in _traj_layouts()])
def test_filter_trajectories_layouts(name, lens):
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    n, m = int(off[-1]), lens.shape[0]
    rng = np.random.default_rng(n + 3 * m)
    q = rng.integers(1, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32)
    score = rng.uniform(0, 1, m).astype(np.float32)
    score[rng.random(m) < 0.05] = np.float32(0.5)          # exactly at the threshold: retained
    score[rng.random(m) < 0.02] = np.nan                   # not retained
    tq = dev(q.view(np.int32)) if n else torch.empty(0, dtype=torch.int32, device="cuda")
    kept = torch.full((1,), -1, dtype=torch.int64, device="cuda")
    distrl.distrl_filter_trajectories(dev(off), dev(score), 0.5, tq, kept)
    torch.cuda.synchronize()
    ref = q.copy()
    kept_ref = oracle.filter_trajectories(off, score, 0.5, ref)
    np.testing.assert_array_equal(tq.cpu().numpy().view(np.uint32), ref)
    assert kept.item() == kept_ref


def test_no_draw_returns_a_filtered_transition():
    w = synth.make_workload(2)
    a = w.arrays
    off, n, m = a["traj_offsets"], w.n, w.m
    g = gpu_retrace(off, a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"], w.gamma, w.lam)
    _, q = _gpu_priorities(w, g["td_delta"])
    score = np.random.default_rng(21).uniform(0, 1, m).astype(np.float32)   # stands in for V_traj's outputs
    tq = dev(q.view(np.int32))
    distrl.distrl_filter_trajectories(dev(off), dev(score), 0.6, tq)
    ref = q.copy()
    oracle.filter_trajectories(off, score, 0.6, ref)
    np.testing.assert_array_equal(tq.cpu().numpy().view(np.uint32), ref)
    ws = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    s = distrl.distrl_build_sampler(tq, ws)
    _check_tree(s, ref)
    u = np.random.default_rng(22).integers(0, 1 << 64, size=20000, dtype=np.uint64)
    u[:3] = [0, (1 << 64) - 1, 1 << 63]
    idx, wts = _sample(s, u, w.beta)
    np.testing.assert_array_equal(idx, sample_by_prefix(ref, u))
    traj_of = np.searchsorted(off, idx, side="right") - 1
    assert np.all(score[traj_of] >= 0.6) and np.all(ref[idx] > 0)
    assert_close(wts, oracle.is_weights(ref, idx, w.beta), "IS weights after filtering")
    assert distrl.distrl_get_status(ws) == 0
    s.close()


@pytest.mark.parametrize("lead", [1, 2, 3])
def test_filter_trajectories_mass_array_off_a_16_byte_boundary(lead):
    # the sweep stores 16 bytes where four neighbouring steps go: the array may start anywhere on a 4-byte boundary,
    # and nothing before or after it may be touched
    rng = np.random.default_rng(50 + lead)
    lens = rng.integers(0, 40, size=3000)
    lens[::97] = 5000                                       # longer than a window
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    n, m = int(off[-1]), lens.shape[0]
    q = rng.integers(1, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32)
    score = rng.uniform(0, 1, m).astype(np.float32)
    score[0] = score[-1] = 0.0                              # the first and the last trajectory go
    guard = 8
    whole = torch.full((lead + n + guard,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    tq = whole[lead:lead + n]
    tq.copy_(dev(q.view(np.int32)))
    assert tq.data_ptr() % 16 == 4 * lead
    kept = torch.zeros(1, dtype=torch.int64, device="cuda")
    distrl.distrl_filter_trajectories(dev(off), dev(score), 0.5, tq, kept)
    torch.cuda.synchronize()
    ref = q.copy()
    kept_ref = oracle.filter_trajectories(off, score, 0.5, ref)
    np.testing.assert_array_equal(tq.cpu().numpy().view(np.uint32), ref)
    assert kept.item() == kept_ref
    h = whole.cpu().numpy()
    assert np.all(h[:lead] == 0x5A5A5A5A) and np.all(h[lead + n:] == 0x5A5A5A5A)


def test_filter_trajectories_edges():
    from paper_2410_14803_b200 import binding
    off = np.array([0, 3, 3, 8], dtype=np.int64)
    q = np.arange(1, 9, dtype=np.uint32)
    tq = dev(q.view(np.int32))
    kept = torch.zeros(1, dtype=torch.int64, device="cuda")
    distrl.distrl_filter_trajectories(dev(off), dev(np.array([1, 1, 1], dtype=np.float32)), 0.0, tq, kept)   # all retained
    torch.cuda.synchronize()
    np.testing.assert_array_equal(tq.cpu().numpy().view(np.uint32), q)
    assert kept.item() == 3
    distrl.distrl_filter_trajectories(dev(off), dev(np.array([0, 5, 5], dtype=np.float32)), 1.0, tq, kept)   # first dropped
    torch.cuda.synchronize()
    np.testing.assert_array_equal(tq.cpu().numpy().view(np.uint32), [0, 0, 0, 4, 5, 6, 7, 8])
    assert kept.item() == 2
    with pytest.raises(distrl.DistrlError):
        distrl.distrl_filter_trajectories(dev(off), dev(np.zeros(3, dtype=np.float32)), float("nan"), tq)
    lib = binding._load()
    assert lib.distrl_filter_trajectories(8, 0, None, None, 0.5, None, None, None) == binding.OK            # no trajectories
    assert lib.distrl_filter_trajectories(8, 3, None, None, 0.5, tq.data_ptr(), None, None) == binding.ERR_NULL
