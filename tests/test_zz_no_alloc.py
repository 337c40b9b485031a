"""The workspace-free Retrace entry point against the ordinary one and against the oracle.

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

import oracle
import paper_2410_14803_b200 as distrl
from paper_2410_14803_b200 import binding, synth

from helpers import TOL, assert_close, dev, random_batch

pytestmark = pytest.mark.gpu


def _both(off, r, V, lp, lm, gamma, lam, boot=None, tokens=None, with_oracle=True):
    """The static entry point and the ordinary one on the same batch; both against each other and the oracle."""
    n = r.shape[0]
    t_boot = dev(boot) if boot is not None else None
    if tokens is None:
        t = [dev(off), dev(r), dev(V), dev(lp), dev(lm)]
        batch = distrl.make_batch(*t, t_boot)
    else:
        sto, tok_p, tok_m = tokens
        t = [dev(off), dev(r), dev(V), dev(sto), dev(tok_p, torch.bfloat16), dev(tok_m, torch.bfloat16)]
        batch = distrl.make_batch(t[0], t[1], t[2], None, None, t_boot, t[3], t[4], t[5])
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
    if with_oracle:
        if tokens is not None:
            lp = oracle.token_logp(tokens[0], oracle.bf16_bits_to_f64(tokens[1]))
            lm = oracle.token_logp(tokens[0], oracle.bf16_bits_to_f64(tokens[2]))
        for g, x, name in zip(got, oracle.retrace(off, r, V, lp, lm, gamma, lam, bootstrap=boot),
                              ("v_target", "advantage", "td_delta")):
            assert_close(g.cpu().numpy(), x, name + " vs oracle", tol=TOL)
    return batch, t, t_boot


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


def test_static_entry_point_at_its_size_limit_then_a_small_call():
    # N == DISTRL_STATIC_MAX_N exactly fills the fixed array (tile flags, first-end table, end mask with its slack);
    # each large call is followed by a small one, which finds the array as the large one left it
    n = binding.STATIC_MAX_N
    w = synth.make_workload(3, n_override=n)
    a = w.arrays
    assert w.n == n
    _both(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"], w.gamma, w.lam)
    off = synth.adversarial_offsets("tile_straddle", 5000)
    _both(off, *random_batch(5, off), 0.9, 0.8)
    # with a bootstrap value per trajectory: near the limit the fixed array has no room for what the pipelined
    # kernel keeps of them, so the call goes through the general kernel; at a small size it does not
    boot = np.random.default_rng(6).normal(0, 1, w.m).astype(np.float32)
    _both(a["traj_offsets"], a["rewards"], a["values"], a["logp_target"], a["logp_behaviour"], w.gamma, w.lam, boot=boot)
    off = synth.adversarial_offsets("long_mixed", 30000)
    _both(off, *random_batch(7, off), 0.97, 0.9, boot=np.random.default_rng(8).normal(0, 1, off.shape[0] - 1).astype(np.float32))
    # token-level mode at the limit (every array 16-byte aligned: the pipelined token kernel), then a small one
    wt = synth.make_workload(4, n_override=n)
    at = wt.arrays
    tok = (at["step_token_offsets"], at["tok_logp_target"], at["tok_logp_behaviour"])
    _both(at["traj_offsets"], at["rewards"], at["values"], None, None, wt.gamma, wt.lam, tokens=tok)
    ws_ = synth.make_workload(4, n_override=3000)
    as_ = ws_.arrays
    _both(as_["traj_offsets"], as_["rewards"], as_["values"], None, None, ws_.gamma, ws_.lam,
          tokens=(as_["step_token_offsets"], as_["tok_logp_target"], as_["tok_logp_behaviour"]))


def test_static_entry_point_takes_no_device_memory_and_leaves_other_calls_alone():
    # After the first call on the device, further calls must not change the amount of free device memory
    # (nothing is allocated, by this library or through it).  Meanwhile an ordinary call with its own
    # workspace runs on a second stream: the two do not share anything, so both results must be right.
    off = synth.adversarial_offsets("long_mixed", 400_000)
    r, V, lp, lm = random_batch(21, off)
    n = r.shape[0]
    t = [dev(off), dev(r), dev(V), dev(lp), dev(lm)]
    batch = distrl.make_batch(*t)
    out_s = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(3)]
    out_w = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(3)]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    distrl.distrl_workspace_init(ws)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    distrl.distrl_retrace_targets_static(batch, 0.99, 0.95, *out_s, status_out=status, stream=s1)   # warm-up call
    distrl.distrl_retrace_targets(batch, 0.99, 0.95, *out_w, workspace=ws, stream=s2)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(10):
        distrl.distrl_retrace_targets_static(batch, 0.99, 0.95, *out_s, status_out=status, stream=s1)
        distrl.distrl_retrace_targets(batch, 0.99, 0.95, *out_w, workspace=ws, stream=s2)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert int(status.item()) == 0 and distrl.distrl_get_status(ws, stream=s2) == 0
    ref = oracle.retrace(off, r, V, lp, lm, 0.99, 0.95)
    for got, name in ((out_s, "static"), (out_w, "workspace")):
        for g, x, what in zip(got, ref, ("v_target", "advantage", "td_delta")):
            assert_close(g.cpu().numpy(), x, "%s %s" % (name, what), tol=TOL)


def test_static_entry_point_checks_its_arguments_before_touching_the_array():
    # a refused call must leave the shared array alone: run a good call, then refused ones, then read the
    # status of the good call's successor
    off = np.array([0, 10, 20], dtype=np.int64)
    r, V, lp, lm = random_batch(2, off)
    t = [dev(off), dev(r), dev(V), dev(lp), dev(lm)]
    out = [torch.empty(20, dtype=torch.float32, device="cuda") for _ in range(2)]
    lib = binding._load()
    b = distrl.make_batch(*t)
    import ctypes
    assert lib.distrl_retrace_targets_static(ctypes.byref(b), 1.5, 0.9, out[0].data_ptr(), out[1].data_ptr(), None, None,
                                             None, None, None) == binding.ERR_PARAM
    assert lib.distrl_retrace_targets_static(ctypes.byref(b), 0.9, 0.9, None, out[1].data_ptr(), None, None, None, None,
                                             None) == binding.ERR_NULL
    assert lib.distrl_retrace_targets_static(None, 0.9, 0.9, None, None, None, None, None, None, None) == binding.ERR_NULL
    _both(off, r, V, lp, lm, 0.9, 0.9)
