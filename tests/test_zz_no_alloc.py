"""The workspace-free Retrace entry point against the ordinary one.

distrl_retrace_targets_static serves callers that cannot allocate device memory
at the point of the call (a framework that already owns the whole GPU, a loop
that must not hit cudaMalloc): its scan bookkeeping lives in a fixed array
inside the library.  Here it is called through the C ABI twice in a row, on
different inputs, and each result is compared with what the ordinary entry
point (caller-allocated workspace) returns for the same input.  The second call
finds the array as the first one left it, which is the case that matters.
This file sorts last on purpose, so a run that stops at the first failure has
already been through every other test.
"""
import numpy as np
import pytest
import torch

import paper_2410_14803_b200 as distrl
from paper_2410_14803_b200 import binding, synth

from helpers import TOL, assert_close, dev, random_batch

pytestmark = pytest.mark.gpu


def _both(off, r, V, lp, lm, gamma, lam):
    n = r.shape[0]
    t = [dev(off), dev(r), dev(V), dev(lp), dev(lm)]
    batch = distrl.make_batch(*t)
    new = lambda: torch.full((n,), float("nan"), dtype=torch.float32, device="cuda")
    ref = [new(), new(), new()]
    ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    distrl.distrl_retrace_targets(batch, gamma, lam, *ref, workspace=ws)
    assert distrl.distrl_get_status(ws) == 0
    got = [new(), new(), new()]
    status = torch.full((1,), -77, dtype=torch.int32, device="cuda")
    distrl.distrl_retrace_targets_static(batch, gamma, lam, *got, status_out=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for g, x, name in zip(got, ref, ("v_target", "advantage", "td_delta")):
        assert_close(g.cpu().numpy(), x.cpu().numpy().astype(np.float64), name, tol=TOL)


def test_static_entry_point_matches_the_workspace_one_twice_in_a_row():
    # call 1: short trajectories over ~20 tiles
    w = synth.make_workload(1)
    a = w.arrays
    _both(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"], w.gamma, w.lam)
    # call 2, right after: another size, with trajectories that cross many tile boundaries, so every
    # flag and carry the first call left in the fixed array would show up as a wrong value
    off = synth.adversarial_offsets("long_mixed", 150001)
    r, V, lp, lm = random_batch(99, off)
    _both(off, r, V, lp, lm, 0.99, 0.95)


def test_static_entry_point_reports_bad_offsets_and_recovers():
    off = np.array([0, 10, 7, 20], dtype=np.int64)
    r, V, lp, lm = random_batch(1, np.array([0, 20]))
    t = [dev(off), dev(r), dev(V), dev(lp), dev(lm)]
    out = [torch.empty(20, dtype=torch.float32, device="cuda") for _ in range(2)]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    distrl.distrl_retrace_targets_static(distrl.make_batch(*t), 0.9, 0.9, *out, status_out=status)
    assert int(status.item()) == binding.ERR_OFFSETS
    good = np.array([0, 10, 20], dtype=np.int64)
    _both(good, r, V, lp, lm, 0.9, 0.9)


def test_static_entry_point_rejects_sizes_beyond_its_array():
    n = binding.STATIC_MAX_N + 1
    z = torch.zeros(n, dtype=torch.float32, device="cuda")
    off = torch.tensor([0, n], dtype=torch.int64, device="cuda")
    batch = distrl.make_batch(off, z, z, z, z)
    out = torch.empty(n, dtype=torch.float32, device="cuda")
    with pytest.raises(distrl.DistrlError) as e:
        distrl.distrl_retrace_targets_static(batch, 0.9, 0.9, out, out.clone())
    assert e.value.code == binding.ERR_SIZE
