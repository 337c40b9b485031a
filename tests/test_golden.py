"""The stored small case (tests/golden/path_small.json, written by tests/golden/make_golden.py from
the oracle alone): the oracle still reproduces it, and the CUDA path matches it."""
import json
import os

import numpy as np
import pytest

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def _load():
    with open(os.path.join(HERE, "golden", "path_small.json")) as f:
        g = json.load(f)
    f32 = lambda k: np.array(g[k], dtype=np.float32)
    return g, np.array(g["traj_offsets"], dtype=np.int64), f32("rewards"), f32("values"), f32("logp_target"), \
        f32("logp_behaviour"), f32("entropy")


def test_oracle_reproduces_the_stored_case():
    g, off, r, V, lp, lm, ent = _load()
    vt, adv, dl = oracle.retrace(off, r, V, lp, lm, g["gamma"], g["lam"])
    np.testing.assert_allclose(vt, g["v_target"], rtol=0, atol=1e-13)
    np.testing.assert_allclose(adv, g["advantage"], rtol=0, atol=1e-13)
    np.testing.assert_allclose(dl, g["td_delta"], rtol=0, atol=1e-13)
    p = g["prio"]
    mass = oracle.priority_mass(dl, lp, lm, ent, p["w_td"], p["w_rho"], p["w_ent"], p["rho_clip"], p["alpha"])
    np.testing.assert_allclose(mass, g["prio_mass"], rtol=1e-13)
    q = oracle.quantise(mass.astype(np.float32), p["scale"])
    assert q.tolist() == g["prio_q_of_oracle_mass"]
    assert oracle.prefix(q)[1] == g["total"]
    u = np.array(g["u_fix"], dtype=np.uint64)
    assert oracle.sample_linear(q, u).tolist() == g["sampled_idx"]
    # the last step of every trajectory has Delta = delta (nothing follows it)
    last = off[1:] - 1
    np.testing.assert_array_equal(np.array(g["advantage"])[last], np.array(g["td_delta"])[last])


@pytest.mark.gpu
def test_cuda_path_matches_the_stored_case():
    import torch
    import paper_2410_14803_b200 as distrl
    from helpers import assert_close, dev
    g, off, r, V, lp, lm, ent = _load()
    n = r.shape[0]
    t = [dev(off), dev(r), dev(V), dev(lp), dev(lm)]
    vt, adv, dl, mass = (torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(4))
    q = torch.empty(n, dtype=torch.int32, device="cuda")
    ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    distrl.distrl_retrace_targets(distrl.make_batch(*t), g["gamma"], g["lam"], vt, adv, dl, workspace=ws)
    p = g["prio"]
    cfg = distrl.make_prio_cfg(p["w_td"], p["w_rho"], p["w_ent"], p["rho_clip"], p["alpha"], p["scale"])
    distrl.distrl_compute_priorities(dl, t[3], t[4], dev(ent), cfg, mass, q)
    assert distrl.distrl_get_status(ws) == 0
    assert_close(vt.cpu().numpy(), g["v_target"], "v_target")
    assert_close(adv.cpu().numpy(), g["advantage"], "advantage")
    assert_close(dl.cpu().numpy(), g["td_delta"], "td_delta")
    assert_close(mass.cpu().numpy(), g["prio_mass"], "prio_mass")
    qh = q.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(qh, oracle.quantise(mass.cpu().numpy(), p["scale"]))
    # sampling is exact given the masses: draw from the device's own masses and compare with the linear scan
    ws2 = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(n))
    distrl.distrl_workspace_init(ws2)
    s = distrl.distrl_build_sampler(q, ws2)
    u = np.array(g["u_fix"], dtype=np.uint64)
    idx = torch.empty(u.shape[0], dtype=torch.int64, device="cuda")
    w = torch.empty(u.shape[0], dtype=torch.float32, device="cuda")
    distrl.distrl_sample(s, dev(u.view(np.int64)), g["beta"], True, idx, w)
    np.testing.assert_array_equal(idx.cpu().numpy(), oracle.sample_linear(qh, u))
    assert_close(w.cpu().numpy(), oracle.is_weights(qh, idx.cpu().numpy(), g["beta"], True), "is_weight")
    if np.array_equal(qh, np.array(g["prio_q_of_oracle_mass"], dtype=np.uint32)):
        assert idx.cpu().numpy().tolist() == g["sampled_idx"]
    s.close()
