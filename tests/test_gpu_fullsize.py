"""Full-size parity cases: the workloads at their real sizes.  The token-level workload is checked twice:
quickly on sampled trajectories that the oracle evaluates one by one plus properties that hold at any
size, and once on every step (the slow test of this file)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_14803_b200 as distrl
from paper_2410_14803_b200 import synth

from helpers import assert_close, dev

pytestmark = pytest.mark.gpu


def _pick_trajectories(off, n_random, tile, seed):
    """Trajectory indices: random ones, the first and last few, and ones that straddle tile boundaries."""
    m = off.shape[0] - 1
    rng = np.random.default_rng(seed)
    picks = [rng.integers(0, m, n_random), np.arange(0, 40), np.arange(m - 40, m)]
    n = int(off[-1])
    cuts = rng.integers(1, n // tile, 400) * tile            # transitions sitting on tile boundaries
    picks.append(np.searchsorted(off, cuts, side="right") - 1)
    picks.append(np.searchsorted(off, cuts - 1, side="right") - 1)
    return np.unique(np.clip(np.concatenate(picks), 0, m - 1))


def test_token_level_full_size_sampled_trajectories():
    w = synth.make_workload(4)                               # 67,108,864 steps, ~1.1e9 tokens
    a = w.arrays
    n, off, sto = w.n, a["traj_offsets"], a["step_token_offsets"]
    t_off, t_r, t_V, t_sto = dev(off), dev(a["rewards"]), dev(a["values"]), dev(sto)
    t_tp = dev(a["tok_logp_target"], torch.bfloat16)
    t_tm = dev(a["tok_logp_behaviour"], torch.bfloat16)
    batch = distrl.make_batch(t_off, t_r, t_V, None, None, None, t_sto, t_tp, t_tm)
    vt, adv, dl, lpo, lmo = (torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(5))
    ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    distrl.distrl_retrace_targets(batch, w.gamma, w.lam, vt, adv, dl, lpo, lmo, workspace=ws)
    assert distrl.distrl_get_status(ws) == 0

    # properties that hold everywhere: at a trajectory's last step Delta = delta exactly; v_target = V + Delta
    last = t_off[1:] - 1
    assert torch.equal(adv[last], dl[last])
    assert torch.all(torch.isfinite(vt)) and torch.all(torch.isfinite(adv))
    assert float((vt - (t_V + adv)).abs().max()) <= 1e-6

    # sampled trajectories, evaluated by the oracle on their own
    js = _pick_trajectories(off, 3000, 1024, 4)
    idx = np.concatenate([np.arange(off[j], off[j + 1]) for j in js])
    sub_off = np.concatenate([[0], np.cumsum(off[js + 1] - off[js])]).astype(np.int64)
    tok_idx = np.concatenate([np.arange(sto[off[j]], sto[off[j + 1]]) for j in js])
    cnt = sto[idx + 1] - sto[idx]
    sub_sto = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int64)
    lp = oracle.token_logp(sub_sto, oracle.bf16_bits_to_f64(a["tok_logp_target"][tok_idx]))
    lm = oracle.token_logp(sub_sto, oracle.bf16_bits_to_f64(a["tok_logp_behaviour"][tok_idx]))
    o_vt, o_adv, o_dl = oracle.retrace(sub_off, a["rewards"][idx], a["values"][idx], lp, lm, w.gamma, w.lam)
    g = torch.from_numpy(idx).cuda()
    assert_close(lpo[g].cpu().numpy(), lp, "token logp_target")
    assert_close(lmo[g].cpu().numpy(), lm, "token logp_behaviour")
    assert_close(vt[g].cpu().numpy(), o_vt, "v_target")
    assert_close(adv[g].cpu().numpy(), o_adv, "advantage")
    assert_close(dl[g].cpu().numpy(), o_dl, "td_delta")

    # the rest of the path on this buffer: priorities from the device's own sums, sampler, one round
    cfg = distrl.make_prio_cfg(w.w_td, w.w_rho, w.w_ent, w.rho_clip, w.alpha, w.scale)
    ent = dev(a["entropy"])
    del t_tp, t_tm
    mass = torch.empty(n, dtype=torch.float32, device="cuda")
    q = torch.empty(n, dtype=torch.int32, device="cuda")
    distrl.distrl_compute_priorities(dl, lpo, lmo, ent, cfg, mass, q)
    o_mass = oracle.priority_mass(o_dl, lp, lm, a["entropy"][idx], w.w_td, w.w_rho, w.w_ent, w.rho_clip, w.alpha)
    assert_close(mass[g].cpu().numpy(), o_mass, "prio_mass")
    qh = q.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(qh[idx], oracle.quantise(mass[g].cpu().numpy(), w.scale))
    ws2 = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(n))
    distrl.distrl_workspace_init(ws2)
    s = distrl.distrl_build_sampler(q, ws2)
    C, total = oracle.prefix(qh)
    tot = torch.zeros(1, dtype=torch.int64, device="cuda")
    distrl.distrl_sampler_total(s, tot)
    assert int(tot.cpu().numpy().view(np.uint64)[0]) == total
    u = synth.uniforms(w, 0)
    d_idx = torch.empty(w.batch, dtype=torch.int64, device="cuda")
    d_w = torch.empty(w.batch, dtype=torch.float32, device="cuda")
    distrl.distrl_sample(s, dev(u.view(np.int64)), w.beta, True, d_idx, d_w)
    y = np.array([(int(x) * total) >> 64 for x in u], dtype=np.uint64)
    want = np.searchsorted(C, y, side="right").astype(np.int64)
    np.testing.assert_array_equal(d_idx.cpu().numpy(), want)
    np.testing.assert_array_equal(want[:3], oracle.sample_linear(qh, u[:3]))   # the definition itself
    assert_close(d_w.cpu().numpy(), oracle.is_weights(qh, want, w.beta, True), "is_weight")
    assert distrl.distrl_get_status(ws2) == 0
    s.close()


def test_token_level_full_size_every_step():
    # All 67,108,864 steps against the oracle (about 45 s on a B200 machine, most of it the oracle's own
    # token sums over 1.1e9 tokens).  The oracle runs over ranges of whole trajectories, so the widened
    # fp64 copies of the token arrays stay at a few hundred MB at a time.
    w = synth.make_workload(4)
    a = w.arrays
    n, off, sto = w.n, a["traj_offsets"], a["step_token_offsets"]
    t_off, t_r, t_V, t_sto = dev(off), dev(a["rewards"]), dev(a["values"]), dev(sto)
    t_tp = dev(a["tok_logp_target"], torch.bfloat16)
    t_tm = dev(a["tok_logp_behaviour"], torch.bfloat16)
    batch = distrl.make_batch(t_off, t_r, t_V, None, None, None, t_sto, t_tp, t_tm)
    out = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(5)]
    ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    distrl.distrl_retrace_targets(batch, w.gamma, w.lam, *out, workspace=ws)
    assert distrl.distrl_get_status(ws) == 0
    del t_tp, t_tm, batch
    vt, adv, dl, lpo, lmo = (o.cpu().numpy() for o in out)
    m = off.shape[0] - 1
    step = 1 << 18                                           # trajectories per range (about 4 M steps, 67 M tokens)
    for j0 in range(0, m, step):
        j1 = min(m, j0 + step)
        s0, s1 = int(off[j0]), int(off[j1])
        k0, k1 = int(sto[s0]), int(sto[s1])
        sub_sto = sto[s0:s1 + 1] - k0
        lp = oracle.token_logp(sub_sto, oracle.bf16_bits_to_f64(a["tok_logp_target"][k0:k1]))
        lm = oracle.token_logp(sub_sto, oracle.bf16_bits_to_f64(a["tok_logp_behaviour"][k0:k1]))
        o_vt, o_adv, o_dl = oracle.retrace(off[j0:j1 + 1] - s0, a["rewards"][s0:s1], a["values"][s0:s1], lp, lm,
                                           w.gamma, w.lam)
        where = "trajectories %d..%d: " % (j0, j1)
        assert_close(lpo[s0:s1], lp, where + "token logp_target")
        assert_close(lmo[s0:s1], lm, where + "token logp_behaviour")
        assert_close(vt[s0:s1], o_vt, where + "v_target")
        assert_close(adv[s0:s1], o_adv, where + "advantage")
        assert_close(dl[s0:s1], o_dl, where + "td_delta")


def test_fused_pass_full_size():
    # workload 3 at its real size through the one-pass entry point, as the benchmark's fused mode runs it:
    # every target, mass, fixed-point image and partial sum, then a draw and a refresh on the sampler it built
    from helpers import prio_cfg_of, read_tree, sample_by_prefix, tree_from_q
    w = synth.make_workload(3)
    a = w.arrays
    n = w.n
    cfg = prio_cfg_of(w)
    scale = synth.heavy_tail_scale(w)
    t = [dev(a["traj_offsets"]), dev(a["rewards"]), dev(a["values"]), dev(a["logp_target"]), dev(a["logp_behaviour"])]
    t_ent, t_sc = dev(a["entropy"]), dev(scale)
    vt, adv, dl, mass = (torch.full((n,), float("nan"), dtype=torch.float32, device="cuda") for _ in range(4))
    tq = torch.zeros(n, dtype=torch.int32, device="cuda")
    ws_r = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    ws_s = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(n))
    distrl.distrl_workspace_init(ws_r)
    distrl.distrl_workspace_init(ws_s)
    s = distrl.distrl_retrace_priorities_build(distrl.make_batch(*t), w.gamma, w.lam, t_ent, t_sc, cfg, vt, adv, dl, tq,
                                               mass, retrace_workspace=ws_r, sampler_workspace=ws_s)
    assert distrl.distrl_get_status(ws_r) == 0
    o_vt, o_adv, o_dl = oracle.retrace(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"],
                                       a["logp_behaviour"], w.gamma, w.lam)
    assert_close(vt.cpu().numpy(), o_vt, "v_target")
    assert_close(adv.cpu().numpy(), o_adv, "advantage")
    assert_close(dl.cpu().numpy(), o_dl, "td_delta")
    o_mass = oracle.priority_mass(o_dl * scale.astype(np.float64), a["logp_target"], a["logp_behaviour"], a["entropy"],
                                  w.w_td, w.w_rho, w.w_ent, w.rho_clip, w.alpha)
    assert_close(mass.cpu().numpy(), o_mass, "prio_mass")
    q = tq.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(q, oracle.quantise(mass.cpu().numpy(), w.scale))
    got, info = read_tree(s)
    for lvl_got, lvl_want in zip(got, tree_from_q(q, info)):
        np.testing.assert_array_equal(lvl_got, lvl_want)
    u = synth.uniforms(w, 0)
    idx = torch.empty(w.batch, dtype=torch.int64, device="cuda")
    wts = torch.empty(w.batch, dtype=torch.float32, device="cuda")
    distrl.distrl_sample(s, dev(u.view(np.int64)), w.beta, True, idx, wts)
    h_idx = idx.cpu().numpy()
    np.testing.assert_array_equal(h_idx, sample_by_prefix(q, u))
    assert_close(wts.cpu().numpy(), oracle.is_weights(q, h_idx, w.beta, True), "is_weight")
    gm = torch.empty(w.batch, dtype=torch.float32, device="cuda")
    distrl.distrl_update_priorities(s, idx, dev(synth.fresh_abs_delta(w, 0)), t[3], t[4], t_ent, cfg, gm)
    oracle.update_from_mass(q, h_idx, gm.cpu().numpy(), w.scale)
    np.testing.assert_array_equal(tq.cpu().numpy().view(np.uint32), q)
    got, info = read_tree(s)
    for lvl_got, lvl_want in zip(got, tree_from_q(q, info)):
        np.testing.assert_array_equal(lvl_got, lvl_want)
    assert distrl.distrl_get_status(ws_s) == 0
    s.close()


def test_bootstrap_values_full_size():
    # workload 3 at its real size with a bootstrap value per trajectory (the pipelined kernel's BOOT path)
    from helpers import check_retrace
    w = synth.make_workload(3)
    a = w.arrays
    boot = np.random.default_rng(12).normal(0, 1, w.m).astype(np.float32)
    check_retrace(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"], w.gamma, w.lam,
                  boot=boot)


def test_large_buffer_trajectory_priorities_and_actor_coefficients():
    # workload 3 at its real size (16,777,216 steps, 1.4 M trajectories), every output against the oracle
    from helpers import prio_cfg_of
    w = synth.make_workload(3)
    a = w.arrays
    n, m, off = w.n, w.m, a["traj_offsets"]
    rng = np.random.default_rng(11)
    delta = (rng.standard_normal(n) * synth.heavy_tail_scale(w)).astype(np.float32)
    adv = rng.standard_normal(n).astype(np.float32)
    t_lp, t_lm, t_ent = dev(a["logp_target"]), dev(a["logp_behaviour"]), dev(a["entropy"])
    mass = torch.empty(m, dtype=torch.float32, device="cuda")
    q = torch.empty(m, dtype=torch.int32, device="cuda")
    distrl.distrl_compute_priorities_traj(dev(off), dev(delta), t_lp, t_lm, t_ent, prio_cfg_of(w), mass, q)
    coef = torch.empty(n, dtype=torch.float32, device="cuda")
    distrl.distrl_actor_coefficients(t_lp, t_lm, dev(adv), coef)
    torch.cuda.synchronize()
    ref = oracle.priority_mass_traj(off, delta, a["logp_target"], a["logp_behaviour"], a["entropy"], w.w_td, w.w_rho,
                                    w.w_ent, w.rho_clip, w.alpha)
    assert_close(mass.cpu().numpy(), ref, "trajectory-level mass, full size")
    np.testing.assert_array_equal(q.cpu().numpy().view(np.uint32), oracle.quantise(mass.cpu().numpy(), w.scale))
    assert_close(coef.cpu().numpy(), oracle.actor_coefficients(a["logp_target"], a["logp_behaviour"], adv),
                 "actor coefficients, full size", tol=1e-5)


def test_large_buffer_monte_carlo_returns():
    # workload 3 at its real size: 8192 tiles, many more than the persistent grid holds at once; every return
    # and label against the oracle
    w = synth.make_workload(3)
    a = w.arrays
    n = w.n
    t_off, t_r = dev(a["traj_offsets"]), dev(a["rewards"])          # the batch holds pointers only
    batch = distrl.make_batch(t_off, t_r, None)
    G = torch.full((n,), float("nan"), dtype=torch.float32, device="cuda")
    lab = torch.full((n,), 7, dtype=torch.uint8, device="cuda")
    ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    runs = []
    for _ in range(3):
        distrl.distrl_mc_returns(batch, w.gamma, G, lab, workspace=ws)
        assert distrl.distrl_get_status(ws) == 0
        runs.append(G.cpu().numpy().copy())
    Gr, labr = oracle.mc_return(a["traj_offsets"], a["rewards"], w.gamma)
    assert_close(runs[0], Gr, "mc_return, full size")
    np.testing.assert_array_equal(lab.cpu().numpy(), (runs[0] > 0).astype(np.uint8))
    clear = np.abs(Gr) > 1e-5
    np.testing.assert_array_equal(lab.cpu().numpy()[clear], labr[clear])
    for r in runs[1:]:
        np.testing.assert_array_equal(r, runs[0])
