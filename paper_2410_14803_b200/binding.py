"""Thin ctypes binding of the C ABI declared in include/distrl.h.

Argument marshalling only: every function here has the name of the entry point
it calls, takes torch CUDA tensors (device memory) and passes their pointers on.
No arithmetic of the method happens in Python, and there is no fallback: if the
CUDA library cannot be loaded or a call fails, a DistrlError is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

_lib = None


class DistrlError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = "%s failed: %d" % (where, code)
        try:
            lib = _load()
            msg = "%s failed: %s (%d)" % (where, lib.distrl_error_string(code).decode(), code)
            if code == ERR_CUDA:
                msg += " -- " + lib.distrl_last_cuda_error().decode()
        except Exception:  # pragma: no cover
            pass
        super().__init__(msg)


OK, ERR_NULL, ERR_SIZE, ERR_ALIGN, ERR_WORKSPACE, ERR_CUDA = 0, -1, -2, -3, -4, -5
ERR_TIMEOUT, ERR_PARAM, ERR_OFFSETS, ERR_INDEX = -6, -7, -8, -9


class distrl_batch(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("reserved", ctypes.c_uint32),
        ("n_transitions", ctypes.c_int64), ("n_trajectories", ctypes.c_int64),
        ("traj_offsets", ctypes.c_void_p), ("rewards", ctypes.c_void_p), ("values", ctypes.c_void_p),
        ("bootstrap_values", ctypes.c_void_p), ("logp_target", ctypes.c_void_p),
        ("logp_behaviour", ctypes.c_void_p), ("step_token_offsets", ctypes.c_void_p),
        ("tok_logp_target_bf16", ctypes.c_void_p), ("tok_logp_behaviour_bf16", ctypes.c_void_p),
    ]


class distrl_prio_cfg(ctypes.Structure):
    _fields_ = [("w_td", ctypes.c_float), ("w_rho", ctypes.c_float), ("w_ent", ctypes.c_float),
                ("rho_clip", ctypes.c_float), ("alpha", ctypes.c_float), ("scale", ctypes.c_float)]


def library_path() -> str:
    return _build.LIB_PATH


def _load():
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if not os.path.exists(path):
        path = _build.build()
    _lib = _open(path)
    return _lib


_checked_lib = None


class checked_build:
    """Context manager: inside it every call of this module goes to the range-checked build of the library
    (compiled on first use).  On exit the ordinary library is back and `violations` holds what the checks
    recorded: (count, source line of the first, its index, its limit)."""

    def __enter__(self):
        global _lib, _checked_lib
        if _checked_lib is None:
            _checked_lib = _open(_build.build(checked=True))
        self._saved = _load()
        _lib = _checked_lib
        self.report()          # start from a clean record
        return self

    def report(self):
        rec = (ctypes.c_int64 * 4)()
        rc = _checked_lib.distrl_bounds_report(rec)
        if rc != 1:
            raise DistrlError(rc, "distrl_bounds_report (not a checked build?)")
        return tuple(int(x) for x in rec)

    def __exit__(self, *exc):
        global _lib
        self.violations = self.report()
        _lib = self._saved
        return False


def _open(path):
    lib = ctypes.CDLL(path)
    vp, i64, sz, f32, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t, ctypes.c_float, ctypes.c_int
    sig = {
        "distrl_retrace_workspace_bytes": (sz, [i64]),
        "distrl_workspace_init": (ci, [vp, sz, vp]),
        "distrl_retrace_targets": (ci, [ctypes.POINTER(distrl_batch), f32, f32, vp, vp, vp, vp, vp, vp, sz, vp]),
        "distrl_retrace_targets_static": (ci, [ctypes.POINTER(distrl_batch), f32, f32, vp, vp, vp, vp, vp, vp, vp]),
        "distrl_mc_returns": (ci, [ctypes.POINTER(distrl_batch), f32, vp, vp, vp, sz, vp]),
        "distrl_compute_priorities": (ci, [i64, vp, vp, vp, vp, ctypes.POINTER(distrl_prio_cfg), vp, vp, vp]),
        "distrl_compute_priorities_traj": (ci, [i64, i64, vp, vp, vp, vp, vp, ctypes.POINTER(distrl_prio_cfg),
                                                vp, vp, vp]),
        "distrl_sampler_workspace_bytes": (sz, [i64]),
        "distrl_build_sampler": (ci, [vp, i64, vp, sz, vp, ctypes.POINTER(vp)]),
        "distrl_sample": (ci, [vp, vp, i64, f32, ci, vp, vp, vp]),
        "distrl_stratify_uniforms": (ci, [vp, i64, vp, vp]),
        "distrl_route_draws": (ci, [vp, i64, vp, ci, ci, vp, vp, vp, vp, vp]),
        "distrl_finish_shard_draws": (ci, [i64, vp, vp, vp, vp, ci, ci, i64, i64, i64, f32, vp, vp, vp]),
        "distrl_normalise_weights": (ci, [vp, i64, vp]),
        "distrl_update_priorities": (ci, [vp, vp, i64, vp, vp, vp, vp, ctypes.POINTER(distrl_prio_cfg), vp, vp]),
        "distrl_retrace_priorities_build": (ci, [ctypes.POINTER(distrl_batch), f32, f32, vp, vp,
                                                 ctypes.POINTER(distrl_prio_cfg), vp, vp, vp, vp, vp, vp, sz, vp, sz, vp,
                                                 ctypes.POINTER(vp)]),
        "distrl_replay_overwrite": (ci, [vp, i64, i64, vp, vp]),
        "distrl_replay_workspace_bytes": (sz, [i64]),
        "distrl_replay_create": (ci, [i64, ci, vp, vp, vp, vp, i64, vp, sz, vp, ctypes.POINTER(vp)]),
        "distrl_replay_ingest": (ci, [vp, vp, i64, vp, vp, vp, vp, vp, vp]),
        "distrl_replay_head": (i64, [vp]),
        "distrl_replay_destroy": (ci, [vp]),
        "distrl_actor_coefficients": (ci, [i64, vp, i64, vp, vp, vp, vp, vp, vp, vp]),
        "distrl_trajectory_ranges": (ci, [i64, vp, vp, i64, vp, vp, vp, vp]),
        "distrl_filter_trajectories": (ci, [i64, i64, vp, vp, f32, vp, vp, vp]),
        "distrl_sampler_total": (ci, [vp, vp, vp]),
        "distrl_sampler_level": (ci, [vp, ci, ctypes.POINTER(sz), ctypes.POINTER(i64)]),
        "distrl_destroy_sampler": (ci, [vp]),
        "distrl_get_status": (ci, [vp, vp]),
        "distrl_selftest_bounded_wait": (ci, [vp, sz, vp]),
        "distrl_set_cooperative_launch": (ci, [ci]),
        "distrl_bounds_report": (ci, [vp]),
        "distrl_error_string": (ctypes.c_char_p, [ci]),
        "distrl_last_cuda_error": (ctypes.c_char_p, []),
        "distrl_version": (ctypes.c_char_p, []),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


def _ptr(t: Optional[torch.Tensor], dtype=None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError("expected dtype %s, got %s" % (dtype, t.dtype))
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream or None
    return int(stream) or None


def _check(rc: int, where: str):
    if rc != OK:
        raise DistrlError(rc, where)


def make_prio_cfg(w_td=1.0, w_rho=0.5, w_ent=0.1, rho_clip=2.0, alpha=0.5, scale=float(2 ** 20)) -> distrl_prio_cfg:
    return distrl_prio_cfg(w_td, w_rho, w_ent, rho_clip, alpha, scale)


def make_batch(traj_offsets, rewards, values, logp_target=None, logp_behaviour=None, bootstrap_values=None,
               step_token_offsets=None, tok_logp_target=None, tok_logp_behaviour=None) -> distrl_batch:
    """Fill a distrl_batch from CUDA tensors.  The struct holds device pointers only; the returned
    object also keeps references to the tensors, so they live as long as it does."""
    b = distrl_batch()
    b._tensors = (traj_offsets, rewards, values, logp_target, logp_behaviour, bootstrap_values,
                  step_token_offsets, tok_logp_target, tok_logp_behaviour)
    b.struct_size = ctypes.sizeof(distrl_batch)
    b.n_transitions = rewards.numel()
    b.n_trajectories = traj_offsets.numel() - 1
    b.traj_offsets = _ptr(traj_offsets, torch.int64)
    b.rewards = _ptr(rewards, torch.float32)
    b.values = _ptr(values, torch.float32) if values is not None else None
    b.bootstrap_values = _ptr(bootstrap_values, torch.float32)
    b.logp_target = _ptr(logp_target, torch.float32)
    b.logp_behaviour = _ptr(logp_behaviour, torch.float32)
    b.step_token_offsets = _ptr(step_token_offsets, torch.int64)
    b.tok_logp_target_bf16 = _ptr(tok_logp_target, torch.bfloat16)
    b.tok_logp_behaviour_bf16 = _ptr(tok_logp_behaviour, torch.bfloat16)
    return b


def distrl_set_cooperative_launch(allowed: bool) -> bool:
    """Library option: allow (default) or forbid the cooperative launch of a normalising draw; returns the old setting."""
    return bool(_load().distrl_set_cooperative_launch(1 if allowed else 0))


def distrl_version() -> str:
    return _load().distrl_version().decode()


def distrl_retrace_workspace_bytes(n: int) -> int:
    return int(_load().distrl_retrace_workspace_bytes(n))


def distrl_sampler_workspace_bytes(n: int) -> int:
    return int(_load().distrl_sampler_workspace_bytes(n))


def distrl_workspace_init(workspace: torch.Tensor, stream=None):
    _check(_load().distrl_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(),
                                         _stream(stream)), "distrl_workspace_init")


def distrl_selftest_bounded_wait(workspace: torch.Tensor, stream=None):
    _check(_load().distrl_selftest_bounded_wait(_ptr(workspace), workspace.numel() * workspace.element_size(),
                                                _stream(stream)), "distrl_selftest_bounded_wait")


def distrl_get_status(workspace: torch.Tensor, stream=None) -> int:
    return int(_load().distrl_get_status(_ptr(workspace), _stream(stream)))


def distrl_retrace_targets(batch: distrl_batch, gamma: float, lam: float, v_target, advantage, td_delta=None,
                           logp_target_out=None, logp_behaviour_out=None, *, workspace, stream=None):
    _check(_load().distrl_retrace_targets(
        ctypes.byref(batch), gamma, lam, _ptr(v_target, torch.float32), _ptr(advantage, torch.float32),
        _ptr(td_delta, torch.float32), _ptr(logp_target_out, torch.float32),
        _ptr(logp_behaviour_out, torch.float32), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _stream(stream)), "distrl_retrace_targets")


STATIC_MAX_N = 1 << 22


def distrl_retrace_targets_static(batch: distrl_batch, gamma: float, lam: float, v_target, advantage, td_delta=None,
                                  logp_target_out=None, logp_behaviour_out=None, status_out=None, stream=None):
    """distrl_retrace_targets for callers that cannot allocate a workspace (N <= STATIC_MAX_N).

    The tile bookkeeping sits in a fixed array inside the library, shared by every call on the
    device: keep such calls on one stream.  `status_out` is an optional int32 CUDA tensor (1 element)
    that receives the device status word of this call."""
    _check(_load().distrl_retrace_targets_static(
        ctypes.byref(batch), gamma, lam, _ptr(v_target, torch.float32), _ptr(advantage, torch.float32),
        _ptr(td_delta, torch.float32), _ptr(logp_target_out, torch.float32),
        _ptr(logp_behaviour_out, torch.float32), _ptr(status_out, torch.int32), _stream(stream)),
        "distrl_retrace_targets_static")


def distrl_mc_returns(batch: distrl_batch, gamma: float, mc_return=None, label=None, *, workspace, stream=None):
    _check(_load().distrl_mc_returns(
        ctypes.byref(batch), gamma, _ptr(mc_return, torch.float32), _ptr(label, torch.uint8), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _stream(stream)), "distrl_mc_returns")


def distrl_compute_priorities(td_delta, logp_target, logp_behaviour, entropy, cfg: distrl_prio_cfg, prio_mass,
                              prio_q, stream=None):
    _check(_load().distrl_compute_priorities(
        td_delta.numel(), _ptr(td_delta, torch.float32), _ptr(logp_target, torch.float32),
        _ptr(logp_behaviour, torch.float32), _ptr(entropy, torch.float32), ctypes.byref(cfg),
        _ptr(prio_mass, torch.float32), _ptr(prio_q), _stream(stream)), "distrl_compute_priorities")


def distrl_compute_priorities_traj(traj_offsets, td_delta, logp_target, logp_behaviour, entropy,
                                   cfg: distrl_prio_cfg, prio_mass, prio_q, stream=None):
    _check(_load().distrl_compute_priorities_traj(
        td_delta.numel(), traj_offsets.numel() - 1, _ptr(traj_offsets, torch.int64),
        _ptr(td_delta, torch.float32), _ptr(logp_target, torch.float32), _ptr(logp_behaviour, torch.float32),
        _ptr(entropy, torch.float32), ctypes.byref(cfg), _ptr(prio_mass, torch.float32), _ptr(prio_q),
        _stream(stream)), "distrl_compute_priorities_traj")


class Sampler:
    """Owns the host handle returned by distrl_build_sampler (frees it on close)."""

    def __init__(self, handle: int, prio_q: torch.Tensor, workspace: torch.Tensor):
        self.handle = handle
        self.prio_q = prio_q          # kept alive: the library reads and updates it
        self.workspace = workspace    # kept alive: holds the tree

    def close(self):
        if self.handle:
            _load().distrl_destroy_sampler(self.handle)
            self.handle = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass


def distrl_build_sampler(prio_q: torch.Tensor, workspace: torch.Tensor, stream=None) -> Sampler:
    if prio_q.element_size() != 4:
        raise ValueError("prio_q must hold 32-bit masses")
    out = ctypes.c_void_p()
    _check(_load().distrl_build_sampler(_ptr(prio_q), prio_q.numel(), _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), _stream(stream),
                                        ctypes.byref(out)), "distrl_build_sampler")
    return Sampler(out.value, prio_q, workspace)


def distrl_sample(s: Sampler, u_fix, beta: float, normalise: bool, idx_out, is_weight_out=None, stream=None):
    if u_fix.element_size() != 8:
        raise ValueError("u_fix must hold 64-bit fixed-point uniforms")
    _check(_load().distrl_sample(s.handle, _ptr(u_fix), u_fix.numel(), beta, 1 if normalise else 0,
                                 _ptr(idx_out, torch.int64), _ptr(is_weight_out, torch.float32),
                                 _stream(stream)), "distrl_sample")


def distrl_stratify_uniforms(u_fix: torch.Tensor, u_out: torch.Tensor, stream=None):
    """u_out[j] = floor((j 2^64 + u_fix[j]) / k): uniforms for stratified draws (u_out may be u_fix)."""
    if u_fix.element_size() != 8 or u_out.element_size() != 8 or u_out.numel() != u_fix.numel():
        raise ValueError("two arrays of 64-bit fixed-point uniforms of the same length")
    _check(_load().distrl_stratify_uniforms(_ptr(u_fix), u_fix.numel(), _ptr(u_out), _stream(stream)),
           "distrl_stratify_uniforms")


def distrl_route_draws(u_fix: torch.Tensor, shard_totals: torch.Tensor, my_shard: int, u_local_out: torch.Tensor,
                       mine_out: torch.Tensor, owner_out: Optional[torch.Tensor] = None,
                       status: Optional[torch.Tensor] = None, stream=None):
    """Global draws over several shards: the local uniform of every draw this shard owns (0 elsewhere) and
    which draws those are.  shard_totals: device array of the shards' total masses (64-bit), in shard order."""
    k = u_fix.numel()
    if u_fix.element_size() != 8 or shard_totals.element_size() != 8 or u_local_out.element_size() != 8:
        raise ValueError("uniforms and totals are 64-bit integers")
    if u_local_out.numel() != k or mine_out.numel() != k or mine_out.element_size() != 1:
        raise ValueError("one local uniform and one byte per draw")
    if owner_out is not None and (owner_out.numel() != k or owner_out.element_size() != 4):
        raise ValueError("owner_out holds one 32-bit integer per draw")
    _check(_load().distrl_route_draws(_ptr(u_fix), k, _ptr(shard_totals), shard_totals.numel(), int(my_shard),
                                      _ptr(u_local_out), _ptr(mine_out), _ptr(owner_out, torch.int32),
                                      _ptr(status, torch.int32), _stream(stream)), "distrl_route_draws")


def distrl_finish_shard_draws(mine, idx_local, w_local, shard_totals, my_shard: int, n_local: int, n_global: int,
                              index_base: int, beta: float, idx_global_out, w_global_out=None, stream=None):
    """Global indices and un-normalised global weights of the draws this shard owns; -1 and 0 elsewhere."""
    k = idx_local.numel()
    if mine.numel() != k or idx_global_out.numel() != k or (w_global_out is not None and w_global_out.numel() != k):
        raise ValueError("one entry per draw")
    _check(_load().distrl_finish_shard_draws(k, _ptr(mine, torch.uint8), _ptr(idx_local, torch.int64),
                                             _ptr(w_local, torch.float32), _ptr(shard_totals), shard_totals.numel(),
                                             int(my_shard), int(n_local), int(n_global), int(index_base), float(beta),
                                             _ptr(idx_global_out, torch.int64), _ptr(w_global_out, torch.float32),
                                             _stream(stream)), "distrl_finish_shard_draws")


def distrl_normalise_weights(is_weight: torch.Tensor, stream=None):
    """is_weight /= max(is_weight), in place."""
    _check(_load().distrl_normalise_weights(_ptr(is_weight, torch.float32), is_weight.numel(), _stream(stream)),
           "distrl_normalise_weights")


def distrl_update_priorities(s: Sampler, idx, new_abs_delta, logp_target, logp_behaviour, entropy,
                             cfg: distrl_prio_cfg, mass_out=None, stream=None):
    _check(_load().distrl_update_priorities(
        s.handle, _ptr(idx, torch.int64), idx.numel(), _ptr(new_abs_delta, torch.float32),
        _ptr(logp_target, torch.float32), _ptr(logp_behaviour, torch.float32), _ptr(entropy, torch.float32),
        ctypes.byref(cfg), _ptr(mass_out, torch.float32), _stream(stream)), "distrl_update_priorities")


def distrl_retrace_priorities_build(batch: distrl_batch, gamma: float, lam: float, entropy, delta_scale,
                                    cfg: distrl_prio_cfg, v_target, advantage, td_delta, prio_q, prio_mass, *,
                                    retrace_workspace, sampler_workspace, stream=None) -> Sampler:
    """Retrace targets, priorities and the sampler's tree in one pass; returns the sampler."""
    out = ctypes.c_void_p()
    _check(_load().distrl_retrace_priorities_build(
        ctypes.byref(batch), gamma, lam, _ptr(entropy, torch.float32), _ptr(delta_scale, torch.float32),
        ctypes.byref(cfg), _ptr(v_target, torch.float32), _ptr(advantage, torch.float32),
        _ptr(td_delta, torch.float32), _ptr(prio_q), _ptr(prio_mass, torch.float32), _ptr(retrace_workspace),
        retrace_workspace.numel() * retrace_workspace.element_size(), _ptr(sampler_workspace),
        sampler_workspace.numel() * sampler_workspace.element_size(), _stream(stream), ctypes.byref(out)),
        "distrl_retrace_priorities_build")
    return Sampler(out.value, prio_q, sampler_workspace)


def distrl_replay_overwrite(s: Sampler, head: int, new_q: torch.Tensor, stream=None):
    """Overwrite the masses of slots head, head+1, ... (mod n) with new_q and repair the tree."""
    if new_q.element_size() != 4:
        raise ValueError("new_q must hold 32-bit masses")
    _check(_load().distrl_replay_overwrite(s.handle, head, new_q.numel(), _ptr(new_q), _stream(stream)),
           "distrl_replay_overwrite")


def distrl_actor_coefficients(logp_target: torch.Tensor, logp_behaviour: torch.Tensor, advantage: torch.Tensor,
                              coef: torch.Tensor, idx: Optional[torch.Tensor] = None,
                              is_weight: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None,
                              stream=None):
    """coef[j] = is_weight[j] * rho_i * A_i for i = idx[j] (idx None: the whole buffer in order)."""
    n = logp_target.numel()
    k = n if idx is None else idx.numel()
    for t in (logp_behaviour, advantage):
        if t.numel() != n:
            raise ValueError("per-transition arrays must have one length")
    if coef.numel() != k or (is_weight is not None and is_weight.numel() != k):
        raise ValueError("coef and is_weight must have one entry per batch position")
    _check(_load().distrl_actor_coefficients(n, _ptr(idx, torch.int64), k, _ptr(logp_target, torch.float32),
                                             _ptr(logp_behaviour, torch.float32), _ptr(advantage, torch.float32),
                                             _ptr(is_weight, torch.float32), _ptr(coef, torch.float32),
                                             _ptr(status, torch.int32), _stream(stream)),
           "distrl_actor_coefficients")


def distrl_trajectory_ranges(traj_offsets: torch.Tensor, idx: torch.Tensor, begin: torch.Tensor, end: torch.Tensor,
                             status: Optional[torch.Tensor] = None, stream=None):
    """[begin, end) of the flat buffer for each drawn trajectory index."""
    k = idx.numel()
    if begin.numel() != k or end.numel() != k:
        raise ValueError("begin and end must have one entry per drawn index")
    _check(_load().distrl_trajectory_ranges(traj_offsets.numel() - 1, _ptr(traj_offsets, torch.int64),
                                            _ptr(idx, torch.int64), k, _ptr(begin, torch.int64),
                                            _ptr(end, torch.int64), _ptr(status, torch.int32), _stream(stream)),
           "distrl_trajectory_ranges")


def distrl_filter_trajectories(traj_offsets: torch.Tensor, traj_score: torch.Tensor, threshold: float,
                               prio_q: torch.Tensor, kept_out: Optional[torch.Tensor] = None, stream=None):
    """Zero the masses of every transition of trajectories scored below the threshold."""
    m = traj_offsets.numel() - 1
    if traj_score.numel() != m:
        raise ValueError("one score per trajectory")
    if prio_q.element_size() != 4:
        raise ValueError("prio_q must hold 32-bit masses")
    _check(_load().distrl_filter_trajectories(prio_q.numel(), m, _ptr(traj_offsets, torch.int64),
                                              _ptr(traj_score, torch.float32), threshold, _ptr(prio_q),
                                              _ptr(kept_out, torch.int64), _stream(stream)),
           "distrl_filter_trajectories")


class Replay:
    """Owns the host handle of a circular buffer of trajectories and keeps its tensors alive."""

    def __init__(self, handle, fields, prio_q, traj_offsets, traj_alive, workspace):
        self.handle = handle
        self.fields, self.prio_q = fields, prio_q
        self.traj_offsets, self.traj_alive, self.workspace = traj_offsets, traj_alive, workspace

    @property
    def head(self) -> int:
        return int(_load().distrl_replay_head(self.handle))

    def close(self):
        if self.handle:
            _load().distrl_replay_destroy(self.handle)
            self.handle = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass


def distrl_replay_workspace_bytes(capacity: int) -> int:
    return int(_load().distrl_replay_workspace_bytes(capacity))


def _ptr_array(tensors, dtype):
    arr = (ctypes.c_void_p * max(len(tensors), 1))()
    for i, t in enumerate(tensors):
        arr[i] = _ptr(t, dtype)
    return arr


def distrl_replay_create(fields, prio_q: torch.Tensor, traj_offsets: torch.Tensor, traj_alive: torch.Tensor,
                         workspace: torch.Tensor, stream=None) -> Replay:
    """fields: list of fp32 CUDA tensors of `capacity` elements each (the buffer's SoA arrays)."""
    if prio_q.element_size() != 4:
        raise ValueError("prio_q must hold 32-bit masses")
    capacity = prio_q.numel()
    for f in fields:
        if f.numel() != capacity:
            raise ValueError("every field needs `capacity` elements")
    if traj_offsets.numel() != traj_alive.numel() + 1:
        raise ValueError("traj_offsets needs one more entry than traj_alive")
    out = ctypes.c_void_p()
    _check(_load().distrl_replay_create(capacity, len(fields), _ptr_array(fields, torch.float32), _ptr(prio_q),
                                        _ptr(traj_offsets, torch.int64), _ptr(traj_alive, torch.float32),
                                        traj_alive.numel(), _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), _stream(stream),
                                        ctypes.byref(out)), "distrl_replay_create")
    return Replay(out.value, list(fields), prio_q, traj_offsets, traj_alive, workspace)


def distrl_replay_ingest(rb: Replay, sampler: Optional[Sampler], new_offsets_host, new_offsets: torch.Tensor, new_fields,
                         new_q: torch.Tensor, n_segments_out: Optional[torch.Tensor] = None, stream=None):
    """new_offsets_host: host int64 array (numpy) [k+1]; new_offsets: the same on the device."""
    import numpy as np
    host = np.ascontiguousarray(new_offsets_host, dtype=np.int64)
    if new_offsets.numel() != host.shape[0]:
        raise ValueError("host and device offsets differ in length")
    if len(new_fields) != len(rb.fields):
        raise ValueError("one array of new rows per field")
    _check(_load().distrl_replay_ingest(rb.handle, sampler.handle if sampler is not None else None, host.shape[0] - 1,
                                        host.ctypes.data_as(ctypes.c_void_p), _ptr(new_offsets, torch.int64),
                                        _ptr_array(new_fields, torch.float32), _ptr(new_q),
                                        _ptr(n_segments_out, torch.int64), _stream(stream)), "distrl_replay_ingest")


def distrl_sampler_total(s: Sampler, total_out: torch.Tensor, stream=None):
    _check(_load().distrl_sampler_total(s.handle, _ptr(total_out), _stream(stream)), "distrl_sampler_total")


def distrl_sampler_level(s: Sampler, level: int):
    """(levels, byte offset of `level` in the workspace, entry count)."""
    off, cnt = ctypes.c_size_t(0), ctypes.c_int64(0)
    levels = _load().distrl_sampler_level(s.handle, level, ctypes.byref(off), ctypes.byref(cnt))
    return int(levels), int(off.value), int(cnt.value)


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A zero-filled, 256-byte aligned device buffer (torch allocations are 512-byte aligned)."""
    ws = torch.zeros(max(int(nbytes), 256), dtype=torch.uint8, device=device)
    assert ws.data_ptr() % 256 == 0
    return ws
