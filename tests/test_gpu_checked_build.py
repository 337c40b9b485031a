"""The range-checked build of the library (the stand-in for a memory checker): every index a kernel computes is
checked right before the access, a violation is recorded and the access skipped.  The small adversarial cases of
the parity suite run through it here; the record must stay empty and the results must be the oracle's.  The same
build cuts the fp32 scan into tiles of half the size (1024 steps instead of 2048), so comparing its results with
the ordinary build's also shows that the results do not depend on how the buffer is tiled."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_14803_b200 as distrl
from paper_2410_14803_b200 import binding, synth

from helpers import assert_close, check_retrace, dev, gpu_retrace, prio_cfg_of, random_batch, read_tree, sample_by_prefix, tree_from_q

pytestmark = pytest.mark.gpu


@pytest.fixture
def checked():
    with binding.checked_build() as cb:
        yield cb
    assert cb.violations == (0, 0, 0, 0), "index out of range: count %d, first at unit*100000+line %d, index %d, limit %d" % cb.violations


def test_the_checked_build_reports_itself_and_the_ordinary_one_does_not():
    rec = (binding.ctypes.c_int64 * 4)()
    assert binding._load().distrl_bounds_report(rec) == 0 and list(rec) == [0, 0, 0, 0]
    with binding.checked_build() as cb:
        assert cb.report() == (0, 0, 0, 0)


@pytest.mark.parametrize("kind", ["single", "ones", "tile_aligned", "tile_straddle", "with_empty", "long_mixed"])
@pytest.mark.parametrize("n", [1, 5, 1023, 1024, 1025, 2049, 20000, 70001])
def test_retrace_layouts_checked(checked, kind, n):
    off = synth.adversarial_offsets(kind, n, tile=1024)
    r, V, lp, lm = random_batch(11 + n, off)
    check_retrace(off, r, V, lp, lm, 0.99, 0.95)
    boot = np.random.default_rng(n).normal(0, 1, off.shape[0] - 1).astype(np.float32)
    check_retrace(off, r, V, lp, lm, 0.97, 0.9, boot=boot)
    check_retrace(off, r, V, lp, lm, 0.97, 0.9, boot=boot, misalign=True)        # the general kernel


@pytest.mark.parametrize("kind", ["long_mixed", "tile_straddle", "with_empty"])
def test_results_do_not_depend_on_the_tiling(kind):
    # 2048-step tiles (ordinary build) against 1024-step tiles (checked build) on the same inputs
    n = 300_007
    off = synth.adversarial_offsets(kind, n)
    r, V, lp, lm = random_batch(3, off)
    a = gpu_retrace(off, r, V, lp, lm, 0.99, 0.95)
    with binding.checked_build() as cb:
        b = gpu_retrace(off, r, V, lp, lm, 0.99, 0.95)
    assert cb.violations == (0, 0, 0, 0)
    assert a["status"] == 0 and b["status"] == 0
    for name in ("v_target", "advantage", "td_delta"):
        assert_close(b[name], a[name].astype(np.float64), name + " (two tilings)", tol=2e-6)
    np.testing.assert_array_equal(a["td_delta"], b["td_delta"])                    # no scan in it: bit-equal


@pytest.mark.parametrize("n", [1, 511, 513, 546, 1025, 4097, 60001])
@pytest.mark.parametrize("counts", ["workload", "all32", "zeros_and_ones"])
def test_token_level_checked(checked, n, counts):
    rng = np.random.default_rng(n)
    off = synth.adversarial_offsets("long_mixed" if n > 600 else "with_empty", n)
    cnt = {"workload": rng.integers(1, 33, n), "all32": np.full(n, 32), "zeros_and_ones": rng.integers(0, 2, n)}[counts]
    sto = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int64)
    ntok = int(sto[-1])
    tok_m = synth.f32_to_bf16_bits(rng.normal(-0.3, 0.3, max(ntok, 1)).astype(np.float32))[:ntok]
    tok_p = synth.f32_to_bf16_bits((synth.bf16_bits_to_f32(tok_m) + rng.normal(0, 0.05, ntok)).astype(np.float32))
    r, V, _, _ = random_batch(n, off)
    out = gpu_retrace(off, r, V, None, None, 0.99, 0.95, tokens=(sto, tok_p, tok_m), want_logp=True)
    assert out["status"] == 0
    lp = oracle.token_logp(sto, oracle.bf16_bits_to_f64(tok_p))
    lm = oracle.token_logp(sto, oracle.bf16_bits_to_f64(tok_m))
    vt, adv, dl = oracle.retrace(off, r, V, lp, lm, 0.99, 0.95)
    assert_close(out["logp_target"], lp, "token logp")
    assert_close(out["v_target"], vt, "v_target")
    assert_close(out["advantage"], adv, "advantage")


@pytest.mark.parametrize("index", [0, 1, 2])
def test_whole_path_checked(checked, index):
    # Retrace -> priorities -> build -> draw -> refresh, the fused pass, Monte-Carlo returns, the trajectory filter
    w = synth.make_workload(index)
    a = w.arrays
    n, k = w.n, w.batch
    cfg = prio_cfg_of(w)
    d = {nm: dev(a[nm]) for nm in ("traj_offsets", "rewards", "values", "logp_target", "logp_behaviour", "entropy")}
    batch = distrl.make_batch(d["traj_offsets"], d["rewards"], d["values"], d["logp_target"], d["logp_behaviour"])
    vt, adv, dl, mass, G = (torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(5))
    q = torch.empty(n, dtype=torch.int32, device="cuda")
    ws_r = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    ws_s = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(n))
    distrl.distrl_workspace_init(ws_r)
    distrl.distrl_workspace_init(ws_s)
    distrl.distrl_retrace_targets(batch, w.gamma, w.lam, vt, adv, dl, workspace=ws_r)
    distrl.distrl_compute_priorities(dl, d["logp_target"], d["logp_behaviour"], d["entropy"], cfg, mass, q)
    s = distrl.distrl_build_sampler(q, ws_s)
    u = synth.uniforms(w, 0)
    idx = torch.empty(k, dtype=torch.int64, device="cuda")
    wts = torch.empty(k, dtype=torch.float32, device="cuda")
    distrl.distrl_sample(s, dev(u.view(np.int64)), w.beta, True, idx, wts)
    qh = q.cpu().numpy().view(np.uint32).copy()
    np.testing.assert_array_equal(idx.cpu().numpy(), sample_by_prefix(qh, u))
    assert_close(wts.cpu().numpy(), oracle.is_weights(qh, idx.cpu().numpy(), w.beta, True), "is_weight")
    um = torch.empty(k, dtype=torch.float32, device="cuda")
    distrl.distrl_update_priorities(s, idx, dev(synth.fresh_abs_delta(w, 0)), d["logp_target"], d["logp_behaviour"],
                                    d["entropy"], cfg, um)
    oracle.update_from_mass(qh, idx.cpu().numpy(), um.cpu().numpy(), w.scale)
    np.testing.assert_array_equal(q.cpu().numpy().view(np.uint32), qh)
    got, info = read_tree(s)
    for x, y in zip(got, tree_from_q(qh, info)):
        np.testing.assert_array_equal(x, y)
    o_vt, o_adv, o_dl = oracle.retrace(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"],
                                       w.gamma, w.lam)
    assert_close(vt.cpu().numpy(), o_vt, "v_target")
    assert_close(adv.cpu().numpy(), o_adv, "advantage")
    distrl.distrl_mc_returns(batch, w.gamma, G, None, workspace=ws_r)
    assert_close(G.cpu().numpy(), oracle.mc_return(a["traj_offsets"], a["rewards"], w.gamma)[0], "mc_return")
    s.close()
    ws_s2 = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(n))
    distrl.distrl_workspace_init(ws_s2)
    q2 = torch.empty(n, dtype=torch.int32, device="cuda")
    s2 = distrl.distrl_retrace_priorities_build(batch, w.gamma, w.lam, d["entropy"], None, cfg, vt, adv, None, q2, mass,
                                                retrace_workspace=ws_r, sampler_workspace=ws_s2)
    q2h = q2.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(q2h, oracle.quantise(mass.cpu().numpy(), w.scale))
    got, info = read_tree(s2)
    for x, y in zip(got, tree_from_q(q2h, info)):
        np.testing.assert_array_equal(x, y)
    score = torch.rand(w.m, device="cuda")
    distrl.distrl_filter_trajectories(d["traj_offsets"], score, 0.5, q2)
    want = q2h.copy()
    oracle.filter_trajectories(a["traj_offsets"], score.cpu().numpy().astype(np.float64), 0.5, want)
    np.testing.assert_array_equal(q2.cpu().numpy().view(np.uint32), want)
    assert distrl.distrl_get_status(ws_r) == 0 and distrl.distrl_get_status(ws_s) == 0 and distrl.distrl_get_status(ws_s2) == 0
    s2.close()


def test_ring_checked(checked):
    from test_gpu_replay import _Pair, _rows
    rng = np.random.default_rng(77)
    pair = _Pair(3001, 3001)
    for call in range(30):
        lens = rng.integers(0, 60, size=int(rng.integers(1, 20))).tolist()
        total = int(sum(lens))
        pair.ingest(lens, _rows(rng, total), rng.integers(1, 2 ** 32, size=total, dtype=np.uint64))
    pair.check()
    pair.close()
