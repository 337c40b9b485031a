"""Shared helpers for the GPU parity tests: run the CUDA path through the C ABI,
run the oracle on the same host arrays, compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2410_14803_b200 as distrl
from paper_2410_14803_b200 import synth

TOL = 1e-4  # max |err| <= TOL * (1 + |ref|) on every fp32 output


def assert_close(got, ref, what, tol=TOL):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, what
    if got.size == 0:
        return
    err = np.abs(got - ref) / (1.0 + np.abs(ref))
    worst = int(np.argmax(err))
    assert np.all(np.isfinite(got)), "%s: non-finite output" % what
    assert err[worst] <= tol, "%s: worst rel err %.3e at %d (got %r, ref %r)" % (
        what, err[worst], worst, got[worst], ref[worst])


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.view(dtype)
    return t.cuda()


def dev_misaligned(a):
    """Same data on the device, starting 4 bytes past a 16-byte boundary."""
    buf = torch.empty(a.shape[0] + 1, dtype=torch.from_numpy(a[:0]).dtype, device="cuda")
    view = buf[1:]
    view.copy_(torch.from_numpy(np.ascontiguousarray(a)))
    assert view.data_ptr() % 16 != 0
    return view


def gpu_retrace(off, r, V, lp, lm, gamma, lam, boot=None, want_delta=True, misalign=False, tokens=None,
                want_logp=False):
    """Returns dict of numpy outputs and the device status word."""
    up = dev_misaligned if misalign else dev
    n = r.shape[0]
    t_off, t_r, t_V = dev(off), up(r), up(V)
    t_boot = dev(boot) if boot is not None else None
    if tokens is None:
        t_lp, t_lm = up(lp), up(lm)
        batch = distrl.make_batch(t_off, t_r, t_V, t_lp, t_lm, t_boot)
        keep = (t_lp, t_lm)
    else:
        sto, tok_p, tok_m = tokens
        t_sto, t_tp, t_tm = dev(sto), dev(tok_p, torch.bfloat16), dev(tok_m, torch.bfloat16)
        batch = distrl.make_batch(t_off, t_r, t_V, None, None, t_boot, t_sto, t_tp, t_tm)
        keep = (t_sto, t_tp, t_tm)
    mk = (lambda: torch.empty(n + 1, dtype=torch.float32, device="cuda")[1:]) if misalign else \
         (lambda: torch.empty(n, dtype=torch.float32, device="cuda"))
    vt, adv = mk().fill_(float("nan")), mk().fill_(float("nan"))
    dl = mk().fill_(float("nan")) if want_delta else None
    lpo = mk().fill_(float("nan")) if want_logp else None
    lmo = mk().fill_(float("nan")) if want_logp else None
    ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    distrl.distrl_retrace_targets(batch, gamma, lam, vt, adv, dl, lpo, lmo, workspace=ws)
    status = distrl.distrl_get_status(ws)
    del keep
    out = dict(v_target=vt.cpu().numpy(), advantage=adv.cpu().numpy(), status=status)
    if want_delta:
        out["td_delta"] = dl.cpu().numpy()
    if want_logp:
        out["logp_target"] = lpo.cpu().numpy()
        out["logp_behaviour"] = lmo.cpu().numpy()
    return out


def check_retrace(off, r, V, lp, lm, gamma, lam, boot=None, **kw):
    out = gpu_retrace(off, r, V, lp, lm, gamma, lam, boot=boot, **kw)
    assert out["status"] == 0, out["status"]
    vt, adv, dl = oracle.retrace(off, r, V, lp, lm, gamma, lam, bootstrap=boot)
    assert_close(out["v_target"], vt, "v_target")
    assert_close(out["advantage"], adv, "advantage")
    if "td_delta" in out:
        assert_close(out["td_delta"], dl, "td_delta")
    return out


def random_batch(seed, off):
    rng = np.random.default_rng(seed)
    n = int(off[-1])
    r = rng.normal(0, 1, n).astype(np.float32)
    V = rng.random(n, dtype=np.float32)
    lm = rng.normal(-5, 2, n).astype(np.float32)
    lp = (lm + rng.normal(0, 0.7, n)).astype(np.float32)
    return r, V, lp, lm


def prio_cfg_of(w, alpha=None):
    return distrl.make_prio_cfg(w.w_td, w.w_rho, w.w_ent, w.rho_clip, w.alpha if alpha is None else alpha, w.scale)


def tree_from_q(q, levels_info):
    """Expected tree levels from the masses, by plain integer sums: list of uint64 arrays."""
    out = []
    cur = np.asarray(q, dtype=np.uint64)
    group = 128
    for (cnt,) in levels_info:
        pad = (-cur.shape[0]) % group
        if pad:
            cur = np.concatenate([cur, np.zeros(pad, dtype=np.uint64)])
        cur = cur.reshape(-1, group).sum(axis=1, dtype=np.uint64)
        assert cur.shape[0] == cnt
        out.append(cur)
        group = 32
    return out


def read_tree(sampler):
    levels, _, _ = distrl.distrl_sampler_level(sampler, 1)
    got, info = [], []
    raw = sampler.workspace
    for l in range(1, levels + 1):
        _, o, cnt = distrl.distrl_sampler_level(sampler, l)
        got.append(raw[o:o + 8 * cnt].view(torch.int64).cpu().numpy().view(np.uint64))
        info.append((cnt,))
    return got, info


def thresholds(u, total):
    """y = floor(u * total / 2^64), exactly, with Python integers."""
    return np.array([(int(x) * int(total)) >> 64 for x in u], dtype=np.uint64)


def sample_by_prefix(q, u):
    """Test-side fast equivalent of the oracle's linear scan (checked against it on subsets)."""
    C, total = oracle.prefix(q)
    y = thresholds(u, total)
    return np.searchsorted(C, y, side="right").astype(np.int64)
