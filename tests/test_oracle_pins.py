"""Pins for the fp64 oracle: every routine is checked against something that is
not itself -- closed forms, textbook reductions written independently here in
numpy / pure Python, hand-expanded small cases and brute-force enumeration.
Chosen so that a dropped term, a wrong sign or index, or a transposed operand
in the oracle fails at least one of them."""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle


def _rand_batch(rng, m, tmax, equal_policies=False):
    lens = rng.integers(1, tmax + 1, size=m)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    n = int(off[-1])
    r = rng.normal(0, 1, n)
    V = rng.uniform(0, 1, n)
    lm = rng.normal(-5, 2, n)
    lp = lm.copy() if equal_policies else lm + rng.normal(0, 0.7, n)
    return off, r, V, lp, lm


def _segments(off):
    return [(int(off[j]), int(off[j + 1])) for j in range(len(off) - 1)]


# ----------------------------------------------------------------- Retrace ---

def test_lambda_zero_is_one_step_td():
    # lambda = 0 => c = 0 => Delta_t = delta_t and the target is r + gamma V(s').
    rng = np.random.default_rng(1)
    off, r, V, lp, lm = _rand_batch(rng, 40, 12)
    g = 0.93
    vt, adv, dl = oracle.retrace(off, r, V, lp, lm, g, 0.0)
    vnext = np.zeros_like(V)
    for a, b in _segments(off):
        vnext[a:b - 1] = V[a + 1:b]
    np.testing.assert_allclose(dl, r + g * vnext - V, rtol=0, atol=1e-14)
    np.testing.assert_allclose(adv, dl, rtol=0, atol=0)
    np.testing.assert_allclose(vt, r + g * vnext, rtol=0, atol=1e-14)


def test_on_policy_lambda_one_is_discounted_mc_return():
    # pi = mu, lambda = 1, V(s_{H+1}) = 0: the target telescopes to
    # G_t = sum_k gamma^(k-t) r_k (Section 5.1's Monte-Carlo return).
    rng = np.random.default_rng(2)
    off, r, V, lp, lm = _rand_batch(rng, 30, 15, equal_policies=True)
    g = 0.9
    vt, adv, _ = oracle.retrace(off, r, V, lp, lm, g, 1.0)
    G = np.zeros_like(r)
    for a, b in _segments(off):
        for t in range(a, b):
            G[t] = sum(g ** (k - t) * r[k] for k in range(t, b))
    np.testing.assert_allclose(vt, G, rtol=0, atol=1e-12)
    np.testing.assert_allclose(adv, G - V, rtol=0, atol=1e-12)


def test_on_policy_is_gae():
    # pi = mu: Delta_t = sum_k (gamma lambda)^(k-t) delta_k (textbook GAE).
    rng = np.random.default_rng(3)
    off, r, V, lp, lm = _rand_batch(rng, 25, 20, equal_policies=True)
    g, lam = 0.97, 0.8
    _, adv, dl = oracle.retrace(off, r, V, lp, lm, g, lam)
    for a, b in _segments(off):
        for t in range(a, b):
            want = sum((g * lam) ** (k - t) * dl[k] for k in range(t, b))
            assert abs(adv[t] - want) < 1e-12


def test_vanishing_ratio_cuts_the_trace():
    # pi/mu = e^-80 everywhere: c ~ 0 and only the one-step error survives.
    rng = np.random.default_rng(4)
    off, r, V, lp, lm = _rand_batch(rng, 20, 10)
    lp = lm - 80.0
    _, adv, dl = oracle.retrace(off, r, V, lp, lm, 0.99, 0.95)
    np.testing.assert_allclose(adv, dl, rtol=0, atol=1e-30)


def test_constant_inputs_geometric_series():
    # V = 0, r = 1, pi = mu: delta = 1 and Delta_t = (1 - (gamma lambda)^n)/(1 - gamma lambda),
    # n = number of steps from t to the end of its trajectory.
    lens = [1, 2, 5, 9, 64]
    off = np.concatenate([[0], np.cumsum(lens)])
    n = int(off[-1])
    g, lam = 0.95, 0.9
    z = np.zeros(n)
    _, adv, dl = oracle.retrace(off, np.ones(n), z, z, z, g, lam)
    assert np.all(dl == 1.0)
    x = g * lam
    for a, b in _segments(off):
        for t in range(a, b):
            assert abs(adv[t] - (1 - x ** (b - t)) / (1 - x)) < 1e-12


def test_three_step_hand_expansion_uses_next_steps_trace():
    # One trajectory of three steps, written out term by term.  The trace that
    # multiplies delta_k carries c_{t+1}..c_k: the first step's own ratio never
    # appears, ratios above one are truncated, below one are kept.
    r = np.array([0.5, -1.0, 2.0])
    V = np.array([0.3, 0.7, 0.2])
    lp = np.array([-1.0, -2.0, -1.0])
    lm = np.array([-3.0, -1.5, -2.0])      # rho = e^2, e^-0.5, e^1
    g, lam, boot = 0.9, 0.8, 0.4
    d0 = r[0] + g * V[1] - V[0]
    d1 = r[1] + g * V[2] - V[1]
    d2 = r[2] + g * boot - V[2]
    c1 = lam * min(1.0, math.exp(-0.5))
    c2 = lam * min(1.0, math.exp(1.0))
    D2 = d2
    D1 = d1 + g * c2 * d2
    D0 = d0 + g * c1 * d1 + g * g * c1 * c2 * d2
    vt, adv, dl = oracle.retrace([0, 3], r, V, lp, lm, g, lam, bootstrap=[boot])
    np.testing.assert_allclose(dl, [d0, d1, d2], atol=1e-15)
    np.testing.assert_allclose(adv, [D0, D1, D2], atol=1e-15)
    np.testing.assert_allclose(vt, V + np.array([D0, D1, D2]), atol=1e-15)
    # changing the first step's ratio changes nothing
    lp2 = lp.copy(); lp2[0] = -7.0
    _, adv2, _ = oracle.retrace([0, 3], r, V, lp2, lm, g, lam, bootstrap=[boot])
    np.testing.assert_array_equal(adv, adv2)


def test_double_sum_equals_recursion():
    rng = np.random.default_rng(5)
    off, r, V, lp, lm = _rand_batch(rng, 12, 64)
    boot = rng.uniform(0, 1, len(off) - 1)
    for g, lam in [(0.99, 0.95), (1.0, 1.0), (0.5, 0.3)]:
        _, adv, _ = oracle.retrace(off, r, V, lp, lm, g, lam, bootstrap=boot)
        ds = oracle.retrace_double_sum(off, r, V, lp, lm, g, lam, bootstrap=boot)
        np.testing.assert_allclose(adv, ds, rtol=1e-12, atol=1e-12)


def test_trajectories_are_independent():
    # Permuting trajectories permutes outputs; splitting the batch changes nothing;
    # zero-length trajectories contribute nothing.
    rng = np.random.default_rng(6)
    off, r, V, lp, lm = _rand_batch(rng, 17, 9)
    g, lam = 0.95, 0.95
    base = oracle.retrace(off, r, V, lp, lm, g, lam)
    segs = _segments(off)
    perm = rng.permutation(len(segs))
    order = np.concatenate([np.arange(*segs[j]) for j in perm])
    off_p = np.concatenate([[0], np.cumsum([segs[j][1] - segs[j][0] for j in perm])])
    out_p = oracle.retrace(off_p, r[order], V[order], lp[order], lm[order], g, lam)
    for x, y in zip(base, out_p):
        np.testing.assert_array_equal(x[order], y)
    cut = 8
    a = oracle.retrace(off[:cut + 1], r[:off[cut]], V[:off[cut]], lp[:off[cut]], lm[:off[cut]], g, lam)
    b = oracle.retrace(off[cut:] - off[cut], r[off[cut]:], V[off[cut]:], lp[off[cut]:], lm[off[cut]:], g, lam)
    for x, ya, yb in zip(base, a, b):
        np.testing.assert_array_equal(x, np.concatenate([ya, yb]))
    off_z = np.sort(np.concatenate([off, off[[0, 3, 3, 9, -1]]]))
    z = oracle.retrace(off_z, r, V, lp, lm, g, lam)
    for x, y in zip(base, z):
        np.testing.assert_array_equal(x, y)


def test_bootstrap_enters_only_the_last_step():
    r = np.array([1.0, 1.0]); V = np.array([0.0, 0.0]); z = np.zeros(2)
    _, _, d0 = oracle.retrace([0, 2], r, V, z, z, 0.5, 0.0)
    _, _, d1 = oracle.retrace([0, 2], r, V, z, z, 0.5, 0.0, bootstrap=[4.0])
    np.testing.assert_array_equal(d0, [1.0, 1.0])
    np.testing.assert_array_equal(d1, [1.0, 3.0])


def test_mc_return_closed_form_and_label():
    g = 0.9
    off = [0, 4, 5, 11]
    r = np.ones(11)
    G, lab = oracle.mc_return(off, r, g)
    for a, b in _segments(off):
        for t in range(a, b):
            assert abs(G[t] - (1 - g ** (b - t)) / (1 - g)) < 1e-13
    assert lab.tolist() == [1] * 11
    G, lab = oracle.mc_return([0, 3], np.array([0.0, -0.01, 0.0]), g)
    np.testing.assert_allclose(G, [-0.009, -0.01, 0.0], atol=1e-15)
    assert lab.tolist() == [0, 0, 0]
    G, lab = oracle.mc_return([0, 3], np.array([-0.01, -0.01, 1.0]), 1.0)
    np.testing.assert_allclose(G, [0.98, 0.99, 1.0], atol=1e-15)
    assert lab.tolist() == [1, 1, 1]


# ----------------------------------------------------------- token log-prob ---

def test_token_logp():
    tok = np.array([-0.5, -0.25, -1.0, -2.0, -0.125, -4.0])
    sto = [0, 1, 3, 3, 6]
    np.testing.assert_array_equal(oracle.token_logp(sto, tok), [-0.5, -1.25, 0.0, -6.125])
    # single-token steps: the step's log-prob is the token
    np.testing.assert_array_equal(oracle.token_logp(np.arange(7), tok), tok)
    # bf16 widening is exact: 0x3F80 = 1.0, 0xBE80 = -0.25, 0x3DCD ~ 0.100098
    np.testing.assert_array_equal(oracle.bf16_bits_to_f64(np.array([0x3F80, 0xBE80, 0x3DCD], dtype=np.uint16)),
                                  [1.0, -0.25, 0.10009765625])


# ---------------------------------------------------------------- priority ---

def test_priority_hand_values():
    d = np.array([-2.0, 0.5, 0.0, 3.0])
    lp = np.array([-1.0, -1.0, -2.0, 0.0])
    lm = np.array([-1.0, -3.0, -1.0, -0.5])       # rho = 1, e^2 (clipped at 2), e^-1, e^0.5
    ent = np.array([0.3, 1.0, 2.0, 0.0])
    w1, w2, w3, clip = 1.0, 0.5, 0.1, 2.0
    p = np.array([2.0 + 0.5 * 1.0 + 0.03,
                  0.5 + 0.5 * 2.0 + 0.1,
                  0.0 + 0.5 * math.exp(-1.0) + 0.2,
                  3.0 + 0.5 * math.exp(0.5) + 0.0])
    np.testing.assert_allclose(oracle.priority_mass(d, lp, lm, ent, w1, w2, w3, clip, 1.0), p, rtol=1e-15)
    np.testing.assert_allclose(oracle.priority_mass(d, lp, lm, ent, w1, w2, w3, clip, 0.5), np.sqrt(p), rtol=1e-15)
    # only the TD term: |delta|
    np.testing.assert_array_equal(oracle.priority_mass(d, lp, lm, ent, 1.0, 0.0, 0.0, clip, 1.0), np.abs(d))
    # clip inactive when large
    big = oracle.priority_mass(d, lp, lm, ent, 0.0, 1.0, 0.0, 100.0, 1.0)
    np.testing.assert_allclose(big, np.exp(lp - lm), rtol=1e-15)
    # no entropy array: the paper's surrogate H_t = -log pi(a_t|s_t)
    np.testing.assert_allclose(oracle.priority_mass(d, lp, lm, None, 0.0, 0.0, 1.0, clip, 1.0), -lp, rtol=1e-15)


def test_trajectory_priority_is_the_mean_of_components():
    d = np.array([1.0, -3.0, 2.0, 4.0])
    lp = np.zeros(4); lm = np.array([0.0, math.log(2.0), 0.0, -5.0])   # rho = 1, .5, 1, e^5 -> clip 2
    ent = np.array([0.2, 0.4, 1.0, 3.0])
    out = oracle.priority_mass_traj([0, 2, 2, 4], d, lp, lm, ent, 1.0, 0.5, 0.1, 2.0, 1.0)
    want0 = 2.0 + 0.5 * 0.75 + 0.1 * 0.3
    want2 = 3.0 + 0.5 * 1.5 + 0.1 * 2.0
    np.testing.assert_allclose(out, [want0, 0.0, want2], rtol=1e-15)
    # single-step trajectories: identical to the per-transition priority
    a = oracle.priority_mass_traj(np.arange(5), d, lp, lm, ent, 1.0, 0.5, 0.1, 2.0, 0.5)
    b = oracle.priority_mass(d, lp, lm, ent, 1.0, 0.5, 0.1, 2.0, 0.5)
    np.testing.assert_array_equal(a, b)


def test_quantiser_table():
    S = 2.0 ** 20
    m = np.array([0.0, -1.0, np.nan, 2.0 ** -21, 1.5 / S, 2.5 / S, 3.5 / S, 1.0, 4095.999, 4096.0,
                  1e30, np.inf, 2.0 ** -30], dtype=np.float32)
    q = oracle.quantise(m, S)
    want = [1, 1, 1, 1, 2, 2, 4, 1 << 20, int(np.rint(np.float64(np.float32(4095.999)) * S)),
            2 ** 32 - 1, 2 ** 32 - 1, 2 ** 32 - 1, 1]
    assert q.tolist() == want
    assert q.dtype == np.uint32


def test_prefix_total_and_monotone():
    rng = np.random.default_rng(7)
    q = rng.integers(1, 2 ** 32, size=1000, dtype=np.uint64).astype(np.uint32)
    C, total = oracle.prefix(q)
    assert total == sum(int(x) for x in q) and total > 2 ** 32
    assert int(C[-1]) == total
    assert np.all(np.diff(C.astype(object)) > 0)
    run = 0
    for i in range(1000):
        run += int(q[i])
        assert int(C[i]) == run


# ---------------------------------------------------------------- sampling ---

def _u_for_y(y, total):
    """Smallest 0.64 fixed-point u whose threshold floor(u total / 2^64) is y."""
    return -((-y * (1 << 64)) // total)


def test_sampling_brute_force_frequencies():
    # Enumerate every threshold y in [0, total): index i must be hit exactly q_i times.
    q = np.array([3, 1, 7, 1, 1, 12, 5], dtype=np.uint32)
    total = int(q.sum())
    us = np.array([_u_for_y(y, total) for y in range(total)], dtype=np.uint64)
    for y, u in zip(range(total), us):
        assert (int(u) * total) >> 64 == y
    idx = oracle.sample_linear(q, us)
    counts = np.bincount(idx, minlength=len(q))
    assert counts.tolist() == q.tolist()
    assert np.all(np.diff(idx) >= 0)                       # monotone in u
    # interval form: y -> i  iff  C_{i-1} <= y < C_i
    C = np.cumsum(q)
    for y, i in zip(range(total), idx):
        assert (C[i - 1] if i else 0) <= y < C[i]


def test_sampling_extremes_and_large_total():
    rng = np.random.default_rng(8)
    q = rng.integers(2 ** 31, 2 ** 32, size=64, dtype=np.uint64).astype(np.uint32)
    idx = oracle.sample_linear(q, np.array([0, 2 ** 64 - 1, 2 ** 63], dtype=np.uint64))
    assert idx[0] == 0 and idx[1] == 63
    C = np.cumsum(q.astype(object))
    y = (2 ** 63 * int(C[-1])) >> 64
    assert (C[idx[2] - 1] if idx[2] else 0) <= y < C[idx[2]]


def test_is_weights_closed_forms():
    q = np.full(50, 1234, dtype=np.uint32)
    idx = np.array([0, 7, 49, 7])
    np.testing.assert_allclose(oracle.is_weights(q, idx, 0.4, True), 1.0, rtol=1e-15)
    np.testing.assert_allclose(oracle.is_weights(q, idx, 0.4, False), 1.0, rtol=1e-15)
    rng = np.random.default_rng(9)
    q = rng.integers(1, 10 ** 6, size=200).astype(np.uint32)
    idx = rng.integers(0, 200, size=32)
    np.testing.assert_allclose(oracle.is_weights(q, idx, 0.0, False), 1.0, rtol=0)
    beta = 0.6
    raw = oracle.is_weights(q, idx, beta, False)
    P = q[idx].astype(np.float64) / float(q.sum(dtype=np.uint64))
    np.testing.assert_allclose(raw * (200 * P) ** beta, 1.0, rtol=1e-13)
    nrm = oracle.is_weights(q, idx, beta, True)
    assert nrm.max() == 1.0
    assert np.argmax(nrm) == np.argmin(q[idx])            # the rarest sample weighs most
    np.testing.assert_allclose(nrm, (q[idx] / q[idx].min()) ** -beta, rtol=1e-13)
    # exact small case: N=2, q=(1,3), beta=1: weights (N P)^-1 = (2, 2/3)
    np.testing.assert_allclose(oracle.is_weights(np.array([1, 3], dtype=np.uint32), [0, 1], 1.0, False),
                               [2.0, 2.0 / 3.0], rtol=1e-15)


def test_update_sequential_last_wins_and_equals_rebuild():
    S = 2.0 ** 20
    n = 16
    q = np.full(n, 5, dtype=np.uint32)
    lp = np.zeros(n); lm = np.zeros(n); ent = np.zeros(n)
    idx = np.array([3, 9, 3, 15])
    nd = np.array([1.0, 4.0, 9.0, 0.0])
    mass = oracle.update(q, idx, nd, lp, lm, ent, 1.0, 0.0, 0.0, 2.0, 0.5, S)
    np.testing.assert_allclose(mass, [1.0, 2.0, 3.0, 0.0])
    want = np.full(n, 5, dtype=np.uint32)
    want[3] = 3 << 20; want[9] = 2 << 20; want[15] = 1
    np.testing.assert_array_equal(q, want)
    # the integer half alone, fed the same masses, lands in the same state
    q2 = np.full(n, 5, dtype=np.uint32)
    oracle.update_from_mass(q2, idx, mass.astype(np.float32), S)
    np.testing.assert_array_equal(q2, want)
    # total moved by exactly the winners' differences
    _, tot = oracle.prefix(q)
    assert tot == 5 * n + (3 << 20) - 5 + (2 << 20) - 5 + 1 - 5


def test_update_priority_terms_by_hand():
    # Every term of the Section 5.3 priority inside the refresh, worked by hand with alpha = 1:
    #   p = w1 |delta_new| + w2 min(rho, clip) + w3 H,   w = (1, 0.5, 0.25), clip = 2
    # index 1: rho = 1/2 (below the clip), H = 0.8  -> 3 + 0.25 + 0.2 = 3.45
    # index 2: rho = 8   (clipped to 2),   H = 0.4  -> 1 + 1.0  + 0.1 = 2.1
    # index 0: rho = 1,                    H = 2.0  -> 0 + 0.5  + 0.5 = 1.0   (delta sign is ignored below)
    S = 2.0 ** 20
    lp = np.array([0.0, math.log(0.25), math.log(0.5), -1.0])
    lm = np.array([0.0, math.log(0.5), math.log(0.0625), -1.0])
    ent = np.array([2.0, 0.8, 0.4, 9.0])
    q = np.full(4, 7, dtype=np.uint32)
    mass = oracle.update(q, [1, 2, 0], [3.0, -1.0, 0.0], lp, lm, ent, 1.0, 0.5, 0.25, 2.0, 1.0, S)
    np.testing.assert_allclose(mass, [3.45, 2.1, 1.0], rtol=1e-15)
    want = [1 << 20, int(np.rint(np.float64(np.float32(3.45)) * S)), int(np.rint(np.float64(np.float32(2.1)) * S)), 7]
    assert q.tolist() == want
    # alpha = 0.5 takes the square root of the same sums
    q = np.full(4, 7, dtype=np.uint32)
    mass = oracle.update(q, [1, 2, 0], [3.0, -1.0, 0.0], lp, lm, ent, 1.0, 0.5, 0.25, 2.0, 0.5, S)
    np.testing.assert_allclose(mass, np.sqrt([3.45, 2.1, 1.0]), rtol=1e-15)
    # no entropy array: H = -log pi(a|s) of the refreshed index.  Only that term: w = (0, 0, 1)
    q = np.full(4, 7, dtype=np.uint32)
    mass = oracle.update(q, [3, 1], [5.0, 5.0], lp, lm, None, 0.0, 0.0, 1.0, 2.0, 1.0, S)
    np.testing.assert_allclose(mass, [1.0, math.log(4.0)], rtol=1e-15)
    # only the ratio term, clip far away: the plain ratio pi / mu, not its inverse
    q = np.full(4, 7, dtype=np.uint32)
    mass = oracle.update(q, [1, 2], [5.0, 5.0], lp, lm, ent, 0.0, 1.0, 0.0, 100.0, 1.0, S)
    np.testing.assert_allclose(mass, [0.5, 8.0], rtol=1e-15)


def test_update_is_the_priority_of_the_fresh_delta_quantised():
    # The refresh of index i with a fresh |delta| must leave exactly what the (separately pinned) priority and
    # quantiser give for a buffer whose delta at i is the fresh one: update(q, idx, d_new) == Q(priority_mass(...))[idx].
    rng = np.random.default_rng(21)
    n, k, S = 300, 40, 2.0 ** 20
    lm = rng.normal(-5, 2, n)
    lp = lm + rng.normal(0, 1.0, n)           # ratios on both sides of the clip of 2
    ent = rng.uniform(0, 3, n)
    idx = rng.permutation(n)[:k]               # distinct, so the order does not matter here
    d_new = np.abs(rng.normal(0, 1, k))
    assert (np.exp(lp - lm)[idx] > 2.0).any() and (np.exp(lp - lm)[idx] < 2.0).any()
    for entropy in (ent, None):
        for alpha in (0.5, 1.0):
            full = np.zeros(n)
            full[idx] = d_new
            ref_mass = oracle.priority_mass(full, lp, lm, entropy, 1.0, 0.5, 0.1, 2.0, alpha)
            q = np.full(n, 3, dtype=np.uint32)
            mass = oracle.update(q, idx, d_new, lp, lm, entropy, 1.0, 0.5, 0.1, 2.0, alpha, S)
            np.testing.assert_array_equal(mass, ref_mass[idx])
            want = np.full(n, 3, dtype=np.uint32)
            want[idx] = oracle.quantise(ref_mass[idx].astype(np.float32), S)
            np.testing.assert_array_equal(q, want)


def test_trajectory_priority_without_entropy_uses_minus_log_pi():
    # H_t = -log pi(a_t|s_t) averaged over the trajectory (Section 5.3), only that term switched on
    lp = np.array([-1.0, -3.0, -0.5, -2.5, -4.0])
    lm = lp.copy()
    d = np.zeros(5)
    out = oracle.priority_mass_traj([0, 2, 5], d, lp, lm, None, 0.0, 0.0, 1.0, 2.0, 1.0)
    np.testing.assert_allclose(out, [2.0, 7.0 / 3.0], rtol=1e-15)
    # and together with the other terms: w = (1, 0.5, 0.1), rho = 1 everywhere, |delta| mean 1.5 and 2
    d = np.array([1.0, -2.0, 3.0, -1.0, 2.0])
    out = oracle.priority_mass_traj([0, 2, 5], d, lp, lm, None, 1.0, 0.5, 0.1, 2.0, 1.0)
    np.testing.assert_allclose(out, [1.5 + 0.5 + 0.2, 2.0 + 0.5 + 0.7 / 3.0], rtol=1e-15)


def test_sampling_frequency_tracks_mass_after_update():
    # After an update the linear scan must see the new masses: enumerate again.
    q = np.array([2, 2, 2, 2], dtype=np.uint32)
    oracle.update_from_mass(q, [1], np.array([6.0], dtype=np.float32), 1.0)
    total = int(q.sum())
    us = np.array([_u_for_y(y, total) for y in range(total)], dtype=np.uint64)
    assert np.bincount(oracle.sample_linear(q, us), minlength=4).tolist() == [2, 6, 2, 2]


def test_exact_rational_check_of_small_retrace():
    # pi = mu (c = lambda) with dyadic inputs: compare against exact rational arithmetic.
    g, lam = Fraction(3, 4), Fraction(1, 2)
    r = [Fraction(1), Fraction(0), Fraction(-2), Fraction(5, 2)]
    V = [Fraction(1, 2), Fraction(1, 4), Fraction(3, 4), Fraction(1, 8)]
    off = [0, 3, 4]
    want = []
    for a, b in [(0, 3), (3, 4)]:
        for t in range(a, b):
            s = Fraction(0)
            for k in range(t, b):
                vn = V[k + 1] if k + 1 < b else Fraction(0)
                s += (g * lam) ** (k - t) * (r[k] + g * vn - V[k])
            want.append(s)
    z = np.zeros(4)
    _, adv, _ = oracle.retrace(off, [float(x) for x in r], [float(x) for x in V], z, z, float(g), float(lam))
    assert [Fraction(x) for x in adv] == want


def test_circular_overwrite_wraps_and_later_writes_win():
    q = np.arange(1, 8, dtype=np.uint32)                      # capacity 7
    nxt = oracle.replay_overwrite(q, 5, np.array([70, 71, 72, 73], dtype=np.uint32))
    assert q.tolist() == [72, 73, 3, 4, 5, 70, 71] and nxt == 2
    q = np.arange(1, 4, dtype=np.uint32)                      # more writes than slots: the last three survive
    nxt = oracle.replay_overwrite(q, 1, np.arange(10, 18, dtype=np.uint32))
    assert q.tolist() == [15, 16, 17] and nxt == 0            # slots visited 1,2,0,1,2,0,1,2


# ------------------------------------------------ actor-loss coefficients ---
def test_actor_coefficient_hand_case_and_on_policy():
    # pi = 0.5, mu = 0.25 -> rho = 2; A = 3; w = 0.5  ->  0.5 * 2 * 3 = 3
    c = oracle.actor_coefficients([math.log(0.5)], [math.log(0.25)], [3.0], idx=[0], is_weight=[0.5])
    assert c[0] == pytest.approx(3.0, rel=1e-15)
    rng = np.random.default_rng(5)
    lm = rng.normal(-4, 2, 300)
    A = rng.normal(0, 1, 300)
    np.testing.assert_array_equal(oracle.actor_coefficients(lm, lm, A), A)   # on-policy: rho = 1


def test_actor_coefficient_is_the_derivative_of_the_importance_weighted_surrogate():
    # grad_theta [ w * (pi_theta / mu) * A ] = w * rho * A * grad_theta log pi_theta, so the coefficient
    # equals d/d(log pi) of S = w * A * exp(log pi - log mu): central differences, independent numpy.
    rng = np.random.default_rng(6)
    n, k = 500, 64
    lm = rng.normal(-5, 2, n)
    lp = lm + rng.normal(0, 0.7, n)
    A = rng.normal(0, 2, n)
    idx = rng.integers(0, n, k)
    w = rng.uniform(0.05, 1.0, k)
    h = 1e-6
    S = lambda x: w * A[idx] * np.exp(x - lm[idx])
    fd = (S(lp[idx] + h) - S(lp[idx] - h)) / (2 * h)
    np.testing.assert_allclose(oracle.actor_coefficients(lp, lm, A, idx, w), fd, rtol=1e-8, atol=1e-9)
    # swapping the two policies inverts the ratio
    a = oracle.actor_coefficients(lp, lm, np.ones(n))
    b = oracle.actor_coefficients(lm, lp, np.ones(n))
    np.testing.assert_allclose(a * b, np.ones(n), rtol=1e-14)
    with pytest.raises(IndexError):
        oracle.actor_coefficients(lp, lm, A, idx=[n])


def test_trajectory_ranges_tile_the_buffer():
    rng = np.random.default_rng(8)
    off = np.concatenate([[0], np.cumsum(rng.integers(0, 9, 40))]).astype(np.int64)
    b, e = oracle.trajectory_ranges(off, np.arange(40))
    assert b[0] == 0 and e[-1] == off[-1]
    np.testing.assert_array_equal(b[1:], e[:-1])                      # consecutive, no gaps
    np.testing.assert_array_equal(e - b, np.diff(off))                # lengths
    pick = rng.integers(0, 40, 17)
    pb, pe = oracle.trajectory_ranges(off, pick)
    for j, t in enumerate(pick):
        assert (pb[j], pe[j]) == (off[t], off[t + 1])
    with pytest.raises(IndexError):
        oracle.trajectory_ranges(off, [40])


# ------------------------------------------------------- trajectory filter ---
def test_filter_keeps_exactly_the_trajectories_at_or_above_the_threshold():
    rng = np.random.default_rng(12)
    lens = rng.integers(0, 7, 60)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    n = int(off[-1])
    q0 = rng.integers(1, 1000, n, dtype=np.uint64).astype(np.uint32)
    score = rng.uniform(0, 1, 60)
    score[3] = 0.5                 # exactly at the threshold: retained
    score[4] = np.nan              # not comparable: not retained
    q = q0.copy()
    kept = oracle.filter_trajectories(off, score, 0.5, q)
    assert kept == int(np.sum(score >= 0.5))
    for j in range(60):            # independent restatement, trajectory by trajectory
        seg = slice(int(off[j]), int(off[j + 1]))
        if score[j] >= 0.5:
            np.testing.assert_array_equal(q[seg], q0[seg])
        else:
            assert not q[seg].any()
    # threshold below every score keeps all and changes nothing; above every score leaves nothing
    q = q0.copy()
    assert oracle.filter_trajectories(off, np.nan_to_num(score, nan=0.2), -1.0, q) == 60
    np.testing.assert_array_equal(q, q0)
    q = q0.copy()
    assert oracle.filter_trajectories(off, score, 2.0, q) == 0 and not q.any()


def test_no_draw_returns_a_filtered_transition_and_the_rest_keep_their_proportions():
    off = np.array([0, 2, 2, 5, 6, 9], dtype=np.int64)            # five trajectories, one empty
    q = np.array([3, 1, 4, 1, 5, 9, 2, 6, 5], dtype=np.uint32)
    score = np.array([0.9, 0.9, 0.1, 0.7, 0.2])
    assert oracle.filter_trajectories(off, score, 0.5, q) == 3
    np.testing.assert_array_equal(q, [3, 1, 0, 0, 0, 9, 0, 0, 0])
    total = int(q.sum())
    # every threshold y in [0, total) by brute force: index i is hit exactly q_i times
    u = np.array([((y << 64) + total - 1) // total for y in range(total)], dtype=np.uint64)
    hits = np.bincount(oracle.sample_linear(q, u), minlength=9)
    np.testing.assert_array_equal(hits, q)


# ------------------------------------------- circular buffer of trajectories ---
def _ring_ingest(ring, lens, tag):
    """Ingest trajectories of the given lengths; row value = tag * 1000 + position in the call, mass = 1 + that."""
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    rows = tag * 1000.0 + np.arange(off[-1], dtype=np.float64)
    q = (1 + tag * 1000 + np.arange(off[-1])).astype(np.uint32)
    return ring.ingest(off, [rows, -rows], q), off, rows, q


def test_ring_hand_case_with_wrap_around():
    # capacity 10.  A (4 rows) and B (3 rows) fill slots 0..6.  C (4 rows) does not fit into slots 7..9:
    # they are retired, C goes to slots 0..3 and evicts A.
    ring = oracle.Ring(10, 2)
    ok, _, _, _ = _ring_ingest(ring, [4, 3], 1)
    assert ok and ring.head == 7
    assert ring.alive.tolist() == [1] * 7 + [0] * 3
    assert ring.start.tolist() == [1, 0, 0, 0, 1, 0, 0, 1, 0, 0]
    assert ring.q.tolist() == [1001, 1002, 1003, 1004, 1005, 1006, 1007, 0, 0, 0]
    ok, _, _, _ = _ring_ingest(ring, [4], 2)
    assert ok and ring.head == 4
    assert ring.alive.tolist() == [1] * 7 + [0] * 3
    assert ring.start.tolist() == [1, 0, 0, 0, 1, 0, 0, 1, 0, 0]
    assert ring.q.tolist() == [2001, 2002, 2003, 2004, 1005, 1006, 1007, 0, 0, 0]
    assert ring.fields[0].tolist() == [2000, 2001, 2002, 2003, 1004, 1005, 1006, 0, 0, 0]
    assert ring.fields[1].tolist() == [-2000, -2001, -2002, -2003, -1004, -1005, -1006, 0, 0, 0]
    off, alive = ring.segments()
    assert off.tolist() == [0, 4, 7, 10] and alive.tolist() == [1, 1, 0]


def test_ring_a_trajectory_cut_by_the_write_index_goes_as_a_whole():
    # A = slots 0..5, B = slots 6..9, head back at 0.  A 2-row trajectory overwrites slots 0..1: A lost
    # rows, so its slots 2..5 are dead (mass 0) although nothing was written there; B is untouched.
    ring = oracle.Ring(10, 2)
    assert _ring_ingest(ring, [6, 4], 1)[0] and ring.head == 0
    assert _ring_ingest(ring, [2], 2)[0] and ring.head == 2
    assert ring.alive.tolist() == [1, 1, 0, 0, 0, 0, 1, 1, 1, 1]
    assert ring.q.tolist() == [2001, 2002, 0, 0, 0, 0, 1007, 1008, 1009, 1010]
    assert ring.start.tolist() == [1, 0, 1, 0, 0, 0, 1, 0, 0, 0]
    assert ring.fields[0][2:6].tolist() == [1002, 1003, 1004, 1005]      # stale rows stay, but are dead
    off, alive = ring.segments()
    assert off.tolist() == [0, 2, 6, 10] and alive.tolist() == [1, 0, 1]
    # a trajectory landing in the middle of B's slots cuts B on both sides
    ring = oracle.Ring(10, 2)
    assert _ring_ingest(ring, [2, 8], 1)[0]
    ring.head = 4
    assert _ring_ingest(ring, [3], 2)[0] and ring.head == 7
    assert ring.alive.tolist() == [1, 1, 0, 0, 1, 1, 1, 0, 0, 0]
    assert ring.start.tolist() == [1, 0, 1, 0, 1, 0, 0, 1, 0, 0]
    assert ring.q.tolist() == [1001, 1002, 0, 0, 2001, 2002, 2003, 0, 0, 0]


def test_ring_capacity_exactly_filled_and_refusals():
    ring = oracle.Ring(8, 2)
    assert _ring_ingest(ring, [3, 0, 5], 1)[0]                       # an empty trajectory stores nothing
    assert ring.head == 0 and ring.alive.all()
    assert ring.start.tolist() == [1, 0, 0, 1, 0, 0, 0, 0]
    assert _ring_ingest(ring, [8], 2)[0] and ring.head == 0          # one trajectory as long as the buffer
    assert ring.alive.all() and ring.start.tolist() == [1] + [0] * 7
    assert ring.q.tolist() == list(range(2001, 2009))
    before = (ring.q.copy(), ring.alive.copy(), ring.start.copy(), ring.fields[0].copy(), ring.head)
    assert not _ring_ingest(ring, [9], 3)[0]                         # longer than the buffer
    assert not _ring_ingest(ring, [5, 5], 3)[0]                      # would overwrite its own first trajectory
    ring.head = 5
    assert not _ring_ingest(ring, [2, 4, 2], 3)[0]                   # 8 rows fit, but 2 + 1 retired + 4 + 2 > 8
    ring.head = 0
    assert not ring.ingest([0, 3, 2], [np.zeros(3), np.zeros(3)], np.ones(3))   # offsets decrease
    assert not ring.ingest([1, 3], [np.zeros(3), np.zeros(3)], np.ones(3))      # offsets do not start at 0
    for a, b in zip(before, (ring.q, ring.alive, ring.start, ring.fields[0], ring.head)):
        assert np.array_equal(a, b)                                  # a refused call changes nothing
    ring.head = 5
    assert _ring_ingest(ring, [2, 4], 3)[0] and ring.head == 4       # 2 + 1 retired + 4 = 7 <= 8
    assert ring.alive.tolist() == [1, 1, 1, 1, 0, 1, 1, 0]
    assert ring.start.tolist() == [1, 0, 0, 0, 1, 1, 0, 1]


class _ListRing:
    """The same buffer kept as a list of stored trajectories (an independent formulation: no flags)."""

    def __init__(self, n):
        self.n, self.head, self.trajs = n, 0, []       # trajs: (first slot, length, tag, first row of the call)

    def _drop_overlapping(self, a, b):
        self.trajs = [t for t in self.trajs if t[0] + t[1] <= a or t[0] >= b]

    def ingest(self, lens, tag):
        row = 0
        for T in lens:
            if T == 0:
                continue
            if self.head + T > self.n:
                self._drop_overlapping(self.head, self.n)
                self.head = 0
            self._drop_overlapping(self.head, self.head + T)
            self.trajs.append((self.head, T, tag, row))
            self.head = (self.head + T) % self.n
            row += T


def test_ring_against_a_list_of_trajectories_and_brute_force_draws():
    rng = np.random.default_rng(31)
    n = 97
    ring, model = oracle.Ring(n, 2), _ListRing(n)
    for call in range(1, 60):
        lens = rng.integers(0, 14, size=int(rng.integers(1, 6))).tolist()
        if call % 9 == 0:
            lens = [int(rng.integers(40, 60))]                         # now and then a long one
        ok, off, rows, q = _ring_ingest(ring, lens, call)
        assert ok
        model.ingest(lens, call)
        assert ring.head == model.head
        want_alive = np.zeros(n, dtype=np.uint8)
        want_q = np.zeros(n, dtype=np.uint32)
        for (s, T, tag, row) in model.trajs:
            want_alive[s:s + T] = 1
            want_q[s:s + T] = 1 + tag * 1000 + row + np.arange(T)
            np.testing.assert_array_equal(ring.fields[0][s:s + T], tag * 1000.0 + row + np.arange(T))
            np.testing.assert_array_equal(ring.fields[1][s:s + T], -(tag * 1000.0 + row + np.arange(T)))
        np.testing.assert_array_equal(ring.alive, want_alive)
        np.testing.assert_array_equal(ring.q, want_q)                  # dead slots carry no mass
        seg_off, seg_alive = ring.segments()
        assert seg_off[0] == 0 and seg_off[-1] == n and np.all(np.diff(seg_off) > 0)
        live = sorted((s, s + T) for (s, T, _, _) in model.trajs)
        assert live == [(int(seg_off[j]), int(seg_off[j + 1])) for j in range(len(seg_alive)) if seg_alive[j]]
        for j in range(len(seg_alive)):                                # segments are all alive or all dead
            assert ring.alive[seg_off[j]:seg_off[j + 1]].min() == ring.alive[seg_off[j]:seg_off[j + 1]].max()
    # every threshold by brute force: slot i is drawn exactly q_i times, an evicted slot never
    total = int(ring.q.sum(dtype=np.uint64))
    u = np.array([((y << 64) + total - 1) // total for y in range(0, total, 7)], dtype=np.uint64)
    drawn = oracle.sample_linear(ring.q, u)
    assert ring.alive[drawn].all()
    C = np.cumsum(ring.q.astype(np.uint64))
    np.testing.assert_array_equal(drawn, np.searchsorted(C, np.arange(0, total, 7, dtype=np.uint64), side="right"))


def test_ring_retrace_over_the_segments_equals_retrace_per_live_trajectory():
    # the CSR view of a wrapped buffer goes through Retrace like any other batch: a live trajectory's
    # targets do not depend on what lies around it (dead stretches included)
    rng = np.random.default_rng(32)
    n = 211
    ring = oracle.Ring(n, 4)                                           # r, V, log pi, log mu
    stored = {}
    for call in range(25):
        lens = rng.integers(1, 30, size=3)
        off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
        T = int(off[-1])
        new = [rng.normal(0, 1, T), rng.random(T), rng.normal(-3, 1, T), rng.normal(-3, 1, T)]
        assert ring.ingest(off, new, rng.integers(1, 99, T))
    seg_off, seg_alive = ring.segments()
    assert seg_alive.any() and not seg_alive.all()                     # wrapped: some stretches are dead
    vt, adv, dl = oracle.retrace(seg_off, *ring.fields, 0.97, 0.9)
    for j in np.flatnonzero(seg_alive):
        a, b = int(seg_off[j]), int(seg_off[j + 1])
        one = oracle.retrace([0, b - a], *[f[a:b] for f in ring.fields], 0.97, 0.9)
        np.testing.assert_array_equal(vt[a:b], one[0])
        np.testing.assert_array_equal(adv[a:b], one[1])


# ------------------------------------------------------------ stratified draws ---
def test_stratified_uniforms_fall_into_their_strata():
    rng = np.random.default_rng(40)
    for k in (1, 2, 3, 7, 256, 1000):
        u = rng.integers(0, 2 ** 64, size=k, dtype=np.uint64)
        u[0], u[-1] = 0, 2 ** 64 - 1
        s = oracle.stratify(u)
        for j in range(k):
            want = ((j << 64) + int(u[j])) // k                        # Python integers: exact
            assert int(s[j]) == want
            assert (j << 64) // k <= int(s[j]) < -((-((j + 1) << 64)) // k)   # stratum j: [j/k, (j+1)/k)
    # k = 1 changes nothing; thresholds of a stratified batch increase with j
    u = rng.integers(0, 2 ** 64, size=1, dtype=np.uint64)
    assert oracle.stratify(u)[0] == u[0]
    s = oracle.stratify(rng.integers(0, 2 ** 64, size=64, dtype=np.uint64))
    assert np.all(np.diff(s.astype(object)) > 0)
    # on equal masses a stratified batch of k = n draws hits every index exactly once
    q = np.full(64, 5, dtype=np.uint32)
    assert sorted(oracle.sample_linear(q, s).tolist()) == list(range(64))
