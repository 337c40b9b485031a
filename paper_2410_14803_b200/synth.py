"""Seeded synthetic trajectory buffers shaped like mobile-control rollouts.

Input generation only: this module holds none of the method's arithmetic and is
the one piece of code that both the CUDA tests/benchmarks and the CPU oracle's
callers share.  Everything is produced on the host with numpy's PCG64 so that a
(config, seed) pair always yields the same bytes.

The five workloads follow the benchmark configurations: short horizons, a sparse
terminal success reward, small per-step penalties, behaviour log-probs far from
zero and a target policy that has drifted a little from the behaviour policy.
The second parameter of every N(., .) / LogNormal(., .) below is a standard
deviation.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

BASE_SEED = 241014800


@dataclass
class Workload:
    name: str
    index: int
    gamma: float
    lam: float
    batch: int                 # k: draws per sampling round
    beta: float                # importance-sampling exponent
    rounds: int                # sample -> update rounds
    heavy_tail: bool           # |delta| scaled by LogNormal(0, 2) before the priority stage
    arrays: Dict[str, np.ndarray] = field(default_factory=dict)
    # priority constants shared by every workload
    w_td: float = 1.0
    w_rho: float = 0.5
    w_ent: float = 0.1
    rho_clip: float = 2.0
    alpha: float = 0.5
    scale: float = float(2 ** 20)

    @property
    def n(self) -> int:
        return int(self.arrays["rewards"].shape[0])

    @property
    def m(self) -> int:
        return int(self.arrays["traj_offsets"].shape[0] - 1)

    @property
    def token_level(self) -> bool:
        return "step_token_offsets" in self.arrays


_SPECS = {
    0: dict(name="tiny", m=64, tmax=10, n=None, gamma=0.95, lam=0.95, batch=32, beta=0.4, rounds=1),
    1: dict(name="small", m=4096, tmax=20, n=None, gamma=0.95, lam=0.95, batch=256, beta=0.4, rounds=1),
    2: dict(name="medium", m=None, tmax=30, n=1 << 20, gamma=0.99, lam=0.9, batch=1024, beta=0.4, rounds=1),
    3: dict(name="large", m=None, tmax=64, n=1 << 24, gamma=0.99, lam=0.95, batch=4096, beta=0.4, rounds=100),
    4: dict(name="token", m=None, tmax=30, n=1 << 26, gamma=0.99, lam=0.95, batch=8192, beta=0.6, rounds=1),
}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (ties to even) and return the 16-bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _lengths_to_total(rng, n, draw):
    """Draw lengths until they sum to >= n, truncate the last so they sum to n exactly."""
    mean_guess = max(1.0, float(np.mean(draw(rng, 4096))))
    lens = draw(rng, int(n / mean_guess * 1.05) + 1024)
    cs = np.cumsum(lens)
    while cs[-1] < n:
        more = draw(rng, max(1024, lens.shape[0] // 10))
        lens = np.concatenate([lens, more])
        cs = np.cumsum(lens)
    last = int(np.searchsorted(cs, n, side="left"))
    lens = lens[:last + 1].copy()
    lens[last] -= int(cs[last] - n)
    return lens


def make_workload(index: int, n_override: Optional[int] = None, m_override: Optional[int] = None,
                  shard: int = 0) -> Workload:
    """Build workload `index` (0..4); the overrides shrink it for tests while keeping its recipe.
    `shard` > 0 gives an independent buffer of the same recipe (one per GPU in multi-GPU runs)."""
    spec = dict(_SPECS[index])
    rng = np.random.Generator(np.random.PCG64(BASE_SEED + index + 100000 * shard))
    n_fixed = n_override if (n_override is not None and spec["n"] is not None) else spec["n"]
    tmax = spec["tmax"]
    if index == 3:
        def draw(r, c):
            return np.minimum(r.geometric(1.0 / 12.0, size=c), 64).astype(np.int64)
    else:
        def draw(r, c):
            return r.integers(1, tmax + 1, size=c, dtype=np.int64)
    if n_fixed is None:
        lens = draw(rng, m_override or spec["m"])
    else:
        lens = _lengths_to_total(rng, n_fixed, draw)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    n = int(off[-1])
    last = off[1:] - 1                                  # flat index of each trajectory's last step

    step_pen, p_succ = (0.0, 0.3) if index < 2 else (-0.01, 0.2)
    rewards = np.full(n, step_pen, dtype=np.float32)
    succ = rng.random(last.shape[0]) < p_succ
    rewards[last[succ]] += np.float32(1.0)
    values = rng.random(n, dtype=np.float32)            # V(s) ~ U(0,1); V after the last step = 0
    entropy = (rng.random(n, dtype=np.float32) * np.float32(3.0)).astype(np.float32)

    w = Workload(name=spec["name"], index=index, gamma=spec["gamma"], lam=spec["lam"], batch=spec["batch"],
                 beta=spec["beta"], rounds=spec["rounds"], heavy_tail=(index == 3))
    w.arrays.update(traj_offsets=off, rewards=rewards, values=values, entropy=entropy)

    if index != 4:
        ratio_sigma = 1.0 if index == 2 else 0.5
        lm = rng.normal(-5.0, 2.0, n).astype(np.float32)
        lp = (lm + rng.normal(0.0, ratio_sigma, n).astype(np.float32)).astype(np.float32)
        w.arrays.update(logp_behaviour=lm, logp_target=lp)
    else:
        counts = rng.integers(1, 33, size=n, dtype=np.int64)
        sto = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
        n_tok = int(sto[-1])
        tok_m = np.empty(n_tok, dtype=np.uint16)
        tok_p = np.empty(n_tok, dtype=np.uint16)
        chunk = 1 << 24
        for a in range(0, n_tok, chunk):
            b = min(n_tok, a + chunk)
            mu = rng.standard_normal(b - a, dtype=np.float32) * np.float32(0.3) - np.float32(0.3)
            bits = f32_to_bf16_bits(mu)
            tok_m[a:b] = bits
            pi = bf16_bits_to_f32(bits) + rng.standard_normal(b - a, dtype=np.float32) * np.float32(0.05)
            tok_p[a:b] = f32_to_bf16_bits(pi)
        w.arrays.update(step_token_offsets=sto, tok_logp_behaviour=tok_m, tok_logp_target=tok_p)
    return w


def heavy_tail_scale(w: Workload) -> np.ndarray:
    """LogNormal(0, 2) factors that stand in for a heavy-tailed critic error (workload 3)."""
    rng = np.random.Generator(np.random.PCG64(BASE_SEED + 100 + w.index))
    return rng.lognormal(0.0, 2.0, w.n).astype(np.float32)


def uniforms(w: Workload, round_index: int, k: Optional[int] = None) -> np.ndarray:
    """Raw 64-bit uniforms (0.64 fixed point) for one sampling round."""
    rng = np.random.Generator(np.random.PCG64(977 + 1000 * w.index + round_index))
    return rng.integers(0, 1 << 64, size=k or w.batch, dtype=np.uint64)


def fresh_abs_delta(w: Workload, round_index: int, k: Optional[int] = None) -> np.ndarray:
    """|delta| values for the priority refresh of one round: |N(0,1)| (x LogNormal(0,2) if heavy-tailed)."""
    rng = np.random.Generator(np.random.PCG64(5000 + 1000 * w.index + round_index))
    k = k or w.batch
    d = np.abs(rng.standard_normal(k)).astype(np.float32)
    if w.heavy_tail:
        d = (d * rng.lognormal(0.0, 2.0, k).astype(np.float32)).astype(np.float32)
    return d


def adversarial_offsets(kind: str, n: int, tile: int = 2048) -> np.ndarray:
    """Trajectory layouts that stress the scan: see the tests for what each one exercises."""
    if kind == "single":            # one trajectory spanning every tile
        return np.array([0, n], dtype=np.int64)
    if kind == "ones":              # every trajectory has one step
        return np.arange(n + 1, dtype=np.int64)
    if kind == "tile_aligned":      # boundaries exactly on tile boundaries
        return np.unique(np.concatenate([np.arange(0, n, tile), [n]])).astype(np.int64)
    if kind == "tile_straddle":     # every boundary one past a tile boundary
        return np.unique(np.concatenate([[0], np.arange(1, n, tile), [n]])).astype(np.int64)
    if kind == "with_empty":        # repeated offsets = empty trajectories
        rng = np.random.Generator(np.random.PCG64(BASE_SEED + 7))
        cuts = np.sort(rng.integers(0, n + 1, size=max(2, n // 5)))
        return np.sort(np.concatenate([[0, 0], cuts, cuts[::3], [n, n]])).astype(np.int64)
    if kind == "long_mixed":        # a few very long trajectories between short ones
        rng = np.random.Generator(np.random.PCG64(BASE_SEED + 8))
        lens = []
        total = 0
        while total < n:
            t = int(rng.integers(1, 20)) if rng.random() < 0.9 else int(rng.integers(tile, 5 * tile))
            t = min(t, n - total)
            lens.append(t)
            total += t
        return np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    raise ValueError(kind)
