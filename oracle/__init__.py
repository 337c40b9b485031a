"""fp64 CPU oracle for the A-RIDE learner hot path -- TEST INFRASTRUCTURE ONLY.

This package wraps ``distrl_oracle.c`` (plain C, single-threaded, fp64) with
numpy argument marshalling.  It defines what the CUDA library must compute and
is deliberately slow and literal.  It is independent of the CUDA path: it
imports nothing from the product package and the product package imports
nothing from here.  Only the tests, the smoke check and the benchmark's
CPU-baseline / reference legs may use it.

Every function takes numpy arrays; floating-point inputs of any width are
widened exactly to float64 before the C routine sees them.

Paper: DistRL / A-RIDE (arXiv 2410.14803): Section 5.2 (Retrace), Section 5.3
(DPER priority), App. A "Priority-Based Sampling" and "Temporal-Difference
Error Calculation".
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "distrl_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-shared",
             "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _f64(a):
    return None if a is None else np.ascontiguousarray(np.asarray(a), dtype=np.float64)


def _i64(a):
    return np.ascontiguousarray(np.asarray(a), dtype=np.int64)


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _d(x):
    return ctypes.c_double(float(x))


def _n(x):
    return ctypes.c_int64(int(x))


def bf16_bits_to_f64(bits):
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def token_logp(step_token_offsets, tok):
    """Per-step action log-prob = sum of the step's token log-probs."""
    sto = _i64(step_token_offsets)
    tok = _f64(tok)
    n = sto.shape[0] - 1
    out = np.empty(n, dtype=np.float64)
    _load().oracle_token_logp(_n(n), _p(sto), _p(tok), _p(out))
    return out


def retrace(traj_offsets, rewards, values, logp_pi, logp_mu, gamma, lam, bootstrap=None):
    """Retrace(lambda) targets (Section 5.2).  Returns (v_target, advantage, td_delta)."""
    off = _i64(traj_offsets)
    r, V, lp, lm, boot = _f64(rewards), _f64(values), _f64(logp_pi), _f64(logp_mu), _f64(bootstrap)
    n, m = r.shape[0], off.shape[0] - 1
    vt, adv, dl = (np.empty(n, dtype=np.float64) for _ in range(3))
    _load().oracle_retrace(_n(n), _n(m), _p(off), _p(r), _p(V), _p(boot), _p(lp), _p(lm),
                           _d(gamma), _d(lam), _p(vt), _p(adv), _p(dl))
    return vt, adv, dl


def retrace_double_sum(traj_offsets, rewards, values, logp_pi, logp_mu, gamma, lam, bootstrap=None):
    """The correction Delta_t as the printed O(T^2) double sum of Section 5.2."""
    off = _i64(traj_offsets)
    r, V, lp, lm, boot = _f64(rewards), _f64(values), _f64(logp_pi), _f64(logp_mu), _f64(bootstrap)
    n, m = r.shape[0], off.shape[0] - 1
    out = np.empty(n, dtype=np.float64)
    _load().oracle_retrace_double_sum(_n(n), _n(m), _p(off), _p(r), _p(V), _p(boot), _p(lp),
                                      _p(lm), _d(gamma), _d(lam), _p(out))
    return out


def mc_return(traj_offsets, rewards, gamma):
    """Monte-Carlo return G_t and label I[G_t > 0] (Section 5.1)."""
    off, r = _i64(traj_offsets), _f64(rewards)
    n, m = r.shape[0], off.shape[0] - 1
    G = np.empty(n, dtype=np.float64)
    lab = np.empty(n, dtype=np.uint8)
    _load().oracle_mc_return(_n(n), _n(m), _p(off), _p(r), _d(gamma), _p(G), _p(lab))
    return G, lab


def priority_mass(td_delta, logp_pi, logp_mu, entropy, w_td, w_rho, w_ent, rho_clip, alpha):
    """Per-transition DPER mass p^alpha (Section 5.3)."""
    d, lp, lm, ent = _f64(td_delta), _f64(logp_pi), _f64(logp_mu), _f64(entropy)
    n = d.shape[0]
    out = np.empty(n, dtype=np.float64)
    _load().oracle_priority_mass(_n(n), _p(d), _p(lp), _p(lm), _p(ent), _d(w_td), _d(w_rho),
                                 _d(w_ent), _d(rho_clip), _d(alpha), _p(out))
    return out


def priority_mass_traj(traj_offsets, td_delta, logp_pi, logp_mu, entropy, w_td, w_rho, w_ent,
                       rho_clip, alpha):
    """Trajectory-level DPER mass from trajectory means (Section 5.3, literal)."""
    off = _i64(traj_offsets)
    d, lp, lm, ent = _f64(td_delta), _f64(logp_pi), _f64(logp_mu), _f64(entropy)
    n, m = d.shape[0], off.shape[0] - 1
    out = np.empty(m, dtype=np.float64)
    _load().oracle_priority_mass_traj(_n(n), _n(m), _p(off), _p(d), _p(lp), _p(lm), _p(ent),
                                      _d(w_td), _d(w_rho), _d(w_ent), _d(rho_clip), _d(alpha),
                                      _p(out))
    return out


def quantise(mass_f32, scale):
    """Fixed-point quantiser Q of an fp32 mass array -> uint32 in [1, 2^32-1]."""
    m = np.ascontiguousarray(mass_f32, dtype=np.float32)
    out = np.empty(m.shape[0], dtype=np.uint32)
    _load().oracle_quantise(_n(m.shape[0]), _p(m), _d(scale), _p(out))
    return out


def prefix(q):
    """Inclusive cumulative masses (uint64) and the total."""
    q = np.ascontiguousarray(q, dtype=np.uint32)
    C = np.empty(q.shape[0], dtype=np.uint64)
    tot = ctypes.c_uint64(0)
    _load().oracle_prefix(_n(q.shape[0]), _p(q), _p(C), ctypes.byref(tot))
    return C, int(tot.value)


def sample_linear(q, u):
    """Proportional sampling by linear scan from 0.64 fixed-point uniforms u."""
    q = np.ascontiguousarray(q, dtype=np.uint32)
    u = np.ascontiguousarray(u, dtype=np.uint64)
    out = np.empty(u.shape[0], dtype=np.int64)
    _load().oracle_sample_linear(_n(q.shape[0]), _p(q), _n(u.shape[0]), _p(u), _p(out))
    return out


def is_weights(q, idx, beta, normalise=True):
    """Importance-sampling weights (N P(i))^-beta, optionally / batch max."""
    q = np.ascontiguousarray(q, dtype=np.uint32)
    idx = _i64(idx)
    out = np.empty(idx.shape[0], dtype=np.float64)
    _load().oracle_is_weights(_n(q.shape[0]), _p(q), _n(idx.shape[0]), _p(idx), _d(beta),
                              ctypes.c_int(1 if normalise else 0), _p(out))
    return out


def update(q, idx, new_abs_delta, logp_pi, logp_mu, entropy, w_td, w_rho, w_ent, rho_clip,
           alpha, scale):
    """Sequential priority refresh, in place on q; returns the fp64 masses used."""
    assert q.dtype == np.uint32 and q.flags.c_contiguous
    idx = _i64(idx)
    d, lp, lm, ent = _f64(new_abs_delta), _f64(logp_pi), _f64(logp_mu), _f64(entropy)
    mass = np.empty(idx.shape[0], dtype=np.float64)
    _load().oracle_update(_n(q.shape[0]), _p(q), _n(idx.shape[0]), _p(idx), _p(d), _p(lp),
                          _p(lm), _p(ent), _d(w_td), _d(w_rho), _d(w_ent), _d(rho_clip),
                          _d(alpha), _d(scale), _p(mass))
    return mass


def update_from_mass(q, idx, mass_f32, scale):
    """Integer half of the refresh: requantise given fp32 masses, batch order, in place."""
    assert q.dtype == np.uint32 and q.flags.c_contiguous
    idx = _i64(idx)
    m = np.ascontiguousarray(mass_f32, dtype=np.float32)
    _load().oracle_update_from_mass(_n(q.shape[0]), _p(q), _n(idx.shape[0]), _p(idx), _p(m),
                                    _d(scale))
    return q


def replay_overwrite(q, head, new_q):
    """Circular-buffer overwrite of masses (App. A), in place on q; returns the next write index."""
    assert q.dtype == np.uint32 and q.flags.c_contiguous
    nq = np.ascontiguousarray(new_q, dtype=np.uint32)
    lib = _load()
    lib.oracle_replay_overwrite.restype = ctypes.c_int64
    return int(lib.oracle_replay_overwrite(_n(q.shape[0]), _p(q), _n(head), _n(nq.shape[0]), _p(nq)))


def actor_coefficients(logp_pi, logp_mu, advantage, idx=None, is_weight=None):
    """w_j * rho_i * A_i for the sampled transitions (actor loss of Section 5.1 / App. A)."""
    lp, lm, adv = _f64(logp_pi), _f64(logp_mu), _f64(advantage)
    n = lp.shape[0]
    ix = None if idx is None else _i64(idx)
    k = n if ix is None else ix.shape[0]
    w = _f64(is_weight)
    out = np.empty(k, dtype=np.float64)
    rc = _load().oracle_actor_coefficients(_n(n), _n(k), _p(ix), _p(lp), _p(lm), _p(adv), _p(w), _p(out))
    if rc:
        raise IndexError("index outside [0, n)")
    return out


def trajectory_ranges(traj_offsets, idx):
    """[begin, end) of the flat buffer for each drawn trajectory index (Section 5.3)."""
    off, ix = _i64(traj_offsets), _i64(idx)
    k = ix.shape[0]
    b = np.empty(k, dtype=np.int64)
    e = np.empty(k, dtype=np.int64)
    rc = _load().oracle_trajectory_ranges(_n(off.shape[0] - 1), _p(off), _n(k), _p(ix), _p(b), _p(e))
    if rc:
        raise IndexError("trajectory index outside [0, m)")
    return b, e


def filter_trajectories(traj_offsets, traj_score, threshold, q):
    """Zero, in place, the masses of every transition of trajectories scored below the threshold
    (the V_traj filter of Section 5.1); returns how many trajectories are retained."""
    assert q.dtype == np.uint32 and q.flags.c_contiguous
    off, sc = _i64(traj_offsets), _f64(traj_score)
    lib = _load()
    lib.oracle_filter_trajectories.restype = ctypes.c_int64
    return int(lib.oracle_filter_trajectories(_n(q.shape[0]), _n(off.shape[0] - 1), _p(off), _p(sc),
                                              _d(threshold), _p(q)))


def stratify(u):
    """Stratified uniforms: draw j gets floor((j 2^64 + u_j) / k), i.e. a uniform from the j-th of k equal strata."""
    u = np.ascontiguousarray(u, dtype=np.uint64)
    out = np.empty_like(u)
    _load().oracle_stratify(_n(u.shape[0]), _p(u), _p(out))
    return out


class Ring:
    """Circular replay buffer of whole trajectories (App. A "Circular Replay Buffer", Section 5.3): the
    oracle's state.  ``fields`` are the per-transition fp64 arrays, ``q`` the masses, ``alive`` / ``start``
    one flag per slot, ``head`` the next write index."""

    def __init__(self, capacity: int, n_fields: int):
        self.n = int(capacity)
        self.fields = [np.zeros(self.n, dtype=np.float64) for _ in range(n_fields)]
        self.q = np.zeros(self.n, dtype=np.uint32)
        self.alive = np.zeros(self.n, dtype=np.uint8)
        self.start = np.zeros(self.n, dtype=np.uint8)
        self.start[0] = 1
        self.head = 0

    def ingest(self, new_offsets, new_fields, new_q) -> bool:
        """Append trajectories (CSR offsets over the new rows); False if the call is refused."""
        off = _i64(new_offsets)
        k = off.shape[0] - 1
        nf = [_f64(a) for a in new_fields]
        assert len(nf) == len(self.fields)
        nq = np.ascontiguousarray(new_q, dtype=np.uint32)
        PP = ctypes.c_void_p * len(nf)
        dst = PP(*[a.ctypes.data for a in self.fields])
        src = PP(*[a.ctypes.data for a in nf])
        head = ctypes.c_int64(self.head)
        rc = _load().oracle_ring_ingest(_n(self.n), ctypes.c_int(len(nf)), dst, _p(self.q), _p(self.alive),
                                        _p(self.start), ctypes.byref(head), _n(k), _p(off), src, _p(nq))
        self.head = int(head.value)
        return rc == 0

    def segments(self):
        """(offsets[M+1], alive[M]): the buffer as CSR segments, live trajectories and dead stretches."""
        off = np.empty(self.n + 1, dtype=np.int64)
        al = np.empty(self.n, dtype=np.uint8)
        lib = _load()
        lib.oracle_ring_segments.restype = ctypes.c_int64
        m = int(lib.oracle_ring_segments(_n(self.n), _p(self.start), _p(self.alive), _p(off), _p(al)))
        return off[:m + 1].copy(), al[:m].copy()
