"""Writes tests/golden/path_small.json: one small fixed case of the whole path, evaluated by the
fp64 oracle only (this script imports nothing but numpy and oracle/).  The stored values are a
regression anchor for the oracle and a second, file-based parity case for the CUDA path; they are
not values printed by the paper (it prints none for this path: Sections 5.2-5.3 give formulas only).

    python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))
import oracle  # noqa: E402


def main():
    rng = np.random.Generator(np.random.PCG64(20241014))
    lens = [3, 1, 7, 2, 12, 5, 1, 9]
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    n = int(off[-1])
    r = np.zeros(n, dtype=np.float32)
    r[off[1:] - 1] = (rng.random(len(lens)) < 0.5).astype(np.float32)
    r -= np.float32(0.01)
    V = rng.random(n, dtype=np.float32)
    lm = rng.normal(-5, 2, n).astype(np.float32)
    lp = (lm + rng.normal(0, 0.8, n)).astype(np.float32)
    ent = (rng.random(n, dtype=np.float32) * 3).astype(np.float32)
    gamma, lam = 0.97, 0.9
    w = dict(w_td=1.0, w_rho=0.5, w_ent=0.1, rho_clip=2.0, alpha=0.5, scale=float(2 ** 20))
    vt, adv, dl = oracle.retrace(off, r, V, lp, lm, gamma, lam)
    mass = oracle.priority_mass(dl, lp, lm, ent, w["w_td"], w["w_rho"], w["w_ent"], w["rho_clip"], w["alpha"])
    q = oracle.quantise(mass.astype(np.float32), w["scale"])
    C, total = oracle.prefix(q)
    u = rng.integers(0, 1 << 64, size=16, dtype=np.uint64)
    idx = oracle.sample_linear(q, u)
    isw = oracle.is_weights(q, idx, 0.4, True)
    out = dict(
        citation="DistRL / A-RIDE (arXiv 2410.14803): Retrace correction of Section 5.2, priority of Section 5.3, "
                 "sampling probability of App. A; evaluated by oracle/ in fp64",
        gamma=gamma, lam=lam, beta=0.4, prio=w,
        traj_offsets=off.tolist(), rewards=[float(x) for x in r], values=[float(x) for x in V],
        logp_target=[float(x) for x in lp], logp_behaviour=[float(x) for x in lm], entropy=[float(x) for x in ent],
        v_target=vt.tolist(), advantage=adv.tolist(), td_delta=dl.tolist(), prio_mass=mass.tolist(),
        prio_q_of_oracle_mass=[int(x) for x in q], total=int(total), u_fix=[int(x) for x in u],
        sampled_idx=[int(x) for x in idx], is_weight=isw.tolist())
    with open(os.path.join(HERE, "path_small.json"), "w") as f:
        json.dump(out, f, indent=1)
    print("wrote", os.path.join(HERE, "path_small.json"))


if __name__ == "__main__":
    main()
