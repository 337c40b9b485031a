#!/usr/bin/env python
"""Benchmark of the A-RIDE learner hot path on B200.

One step = one pass of the whole path over one synthetic trajectory buffer:
Retrace(lambda) targets -> DPER priorities -> sampler build -> R rounds of
(sample k indices + IS weights -> refresh their priorities).  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload large]

N > 1 (torchrun): every rank owns an independent shard of the replay buffer of the
same size (trajectories are independent; no data-path collective), weak scaling.
`--impl reference` times the fp64 CPU oracle on a bounded sample of the workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOAD_INDEX = {"tiny": 0, "small": 1, "medium": 2, "large": 3, "token": 4}
METRIC = "transitions/s"


def _peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# --------------------------------------------------------------------------- oracle legs

def _oracle_sample(w, budget_transitions=2_000_000, draws=48):
    """Time the oracle, as it stands, on a bounded sample of workload `w` and scale to a whole step.

    Streaming stages (Retrace, priority, quantise, prefix) run on the first `budget_transitions`
    transitions (cut at a trajectory boundary); the linear-scan sampler and the refresh are timed on
    `draws` draws over the full buffer.  Returns (estimated seconds per whole step, description)."""
    import oracle
    a = w.arrays
    off = a["traj_offsets"]
    j = int(np.searchsorted(off, min(budget_transitions, w.n), side="right")) - 1
    j = max(j, 1)
    ns = int(off[j])
    sl = slice(0, ns)
    if w.token_level:
        sto = a["step_token_offsets"][:ns + 1]
        nt = int(sto[-1])
        t0 = time.perf_counter()
        lp = oracle.token_logp(sto, oracle.bf16_bits_to_f64(a["tok_logp_target"][:nt]))
        lm = oracle.token_logp(sto, oracle.bf16_bits_to_f64(a["tok_logp_behaviour"][:nt]))
    else:
        t0 = time.perf_counter()
        lp, lm = a["logp_target"][sl], a["logp_behaviour"][sl]
    vt, adv, dl = oracle.retrace(off[:j + 1], a["rewards"][sl], a["values"][sl], lp, lm, w.gamma, w.lam)
    mass = oracle.priority_mass(dl, lp, lm, a["entropy"][sl], w.w_td, w.w_rho, w.w_ent, w.rho_clip, w.alpha)
    q_s = oracle.quantise(mass.astype(np.float32), w.scale)
    oracle.prefix(q_s)
    t_stream = time.perf_counter() - t0
    # sampler legs on the full buffer (masses of the sample tiled: only their size matters for timing)
    from paper_2410_14803_b200 import synth
    q = np.resize(q_s, w.n)
    u = synth.uniforms(w, 0, draws)
    t0 = time.perf_counter()
    idx = oracle.sample_linear(q, u)
    oracle.is_weights(q, idx, w.beta, True)
    t_draw = (time.perf_counter() - t0) / draws
    t0 = time.perf_counter()
    oracle.update(q_s.copy(), np.minimum(idx, ns - 1), synth.fresh_abs_delta(w, 0, draws), lp, lm,
                  a["entropy"][sl], w.w_td, w.w_rho, w.w_ent, w.rho_clip, w.alpha, w.scale)
    t_upd = (time.perf_counter() - t0) / draws
    est = t_stream * (w.n / ns) + w.rounds * w.batch * (t_draw + t_upd)
    desc = ("oracle (1 thread, fp64): Retrace+priority+quantise+prefix timed on the first %d transitions "
            "(%.2f s) and scaled by N/%d; linear-scan sampling + IS weights + refresh timed on %d draws over "
            "all N=%d masses (%.2f ms/draw) and scaled to %d rounds x %d draws"
            % (ns, t_stream, ns, draws, w.n, 1e3 * (t_draw + t_upd), w.rounds, w.batch))
    return est, desc, dict(stream_s_per_transition=t_stream / ns, draw_s=t_draw + t_upd)


# ---- all-cores leg: the same oracle routines over contiguous ranges of whole trajectories, one process per core.
# Worker processes are started with "spawn" (a process forked after the first CUDA call hangs); each loads its
# range from a file once, untimed, and the timed call only computes.
_MC = {}


def _mc_load(job):
    path, j0, j1 = job
    import oracle
    z = np.load(path)
    off = z["off"]
    s0, s1 = int(off[j0]), int(off[j1])
    _MC["args"] = (off[j0:j1 + 1] - s0, z["r"][s0:s1], z["V"][s0:s1], z["lp"][s0:s1], z["lm"][s0:s1], z["ent"][s0:s1])
    _MC["oracle"] = oracle
    oracle.quantise(np.ones(4, dtype=np.float32), 1.0)      # loads the library
    return s1 - s0


def _mc_compute(cfg):
    gamma, lam, w_td, w_rho, w_ent, rho_clip, alpha, scale = cfg
    o = _MC["oracle"]
    off, r, V, lp, lm, ent = _MC["args"]
    vt, adv, dl = o.retrace(off, r, V, lp, lm, gamma, lam)
    mass = o.priority_mass(dl, lp, lm, ent, w_td, w_rho, w_ent, rho_clip, alpha)
    q = o.quantise(mass.astype(np.float32), scale)
    return int(q[:8].sum())


def _oracle_all_cores(w, per_core=1_000_000):
    """Retrace + priority + quantise (the stages without a dependency between trajectories) on all host cores.
    Returns (transitions per second, cores, description).  Fixed-N fp32 workloads only."""
    import multiprocessing as mp
    import tempfile
    try:
        cores = len(os.sched_getaffinity(0))
    except Exception:
        cores = os.cpu_count() or 1
    a = w.arrays
    off = a["traj_offsets"]
    ns_want = min(w.n, per_core * cores)
    j_end = max(cores, int(np.searchsorted(off, ns_want, side="right")) - 1)
    cuts = [int(np.searchsorted(off, int(off[j_end]) * c // cores, side="left")) for c in range(cores + 1)]
    cuts[0], cuts[-1] = 0, j_end
    ns = int(off[j_end])
    with tempfile.TemporaryDirectory() as d:
        path = os.path.join(d, "sample.npz")
        np.savez(path, off=off[:j_end + 1], r=a["rewards"][:ns], V=a["values"][:ns], lp=a["logp_target"][:ns],
                 lm=a["logp_behaviour"][:ns], ent=a["entropy"][:ns])
        ctx = mp.get_context("spawn")
        with ctx.Pool(cores) as pool:
            jobs = [(path, cuts[c], cuts[c + 1]) for c in range(cores)]
            pool.map(_mc_load, jobs, chunksize=1)
            cfg = (w.gamma, w.lam, w.w_td, w.w_rho, w.w_ent, w.rho_clip, w.alpha, w.scale)
            pool.map(_mc_compute, [cfg] * cores, chunksize=1)          # warm-up
            t0 = time.perf_counter()
            pool.map(_mc_compute, [cfg] * cores, chunksize=1)
            dt = time.perf_counter() - t0
    desc = ("multi-core baseline: oracle Retrace + priority + quantise (fp64, same routines) over %d contiguous "
            "ranges of whole trajectories, one process per core, first %d transitions in %.2f s; the sampler stages "
            "are not in this figure" % (cores, ns, dt))
    return ns / dt, cores, desc


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2410_14803_b200 import synth
    w = synth.make_workload(WORKLOAD_INDEX[args.workload])
    budget = 1_000_000 if args.steps > 3 else 2_000_000
    times = []
    desc = ""
    for i in range(args.warmup + args.steps):
        est, desc, _ = _oracle_sample(w, budget, draws=16)
        if i >= args.warmup:
            times.append(est)
    t = float(np.mean(times))
    value = w.n / t
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": METRIC, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": _config(w, args),
        "estimated": True,   # scaled from a bounded sample of the workload (see cpu_baseline.sample)
        "cpu_baseline": {"value": value, "unit": METRIC, "cores": 1, "kind": "oracle", "sample": desc, "estimated": True},
        "e2e": {"value": value, "unit": METRIC, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def _step_bytes(w, args):
    """Algorithmic bytes of the three streaming stages of one step: (Retrace call, priorities, sampler build)."""
    n, m = w.n, w.m
    if w.token_level:   # r, V, step offsets, both bf16 token arrays in; v_target, advantage, td_delta, logpi, logmu out; offsets
        retrace_bytes = (8 + 8 + 20) * n + 4 * int(w.arrays["step_token_offsets"][-1]) + 8 * (m + 1)
    else:               # r, V, logpi, logmu in; v_target, advantage, td_delta out; offsets
        retrace_bytes = 28 * n + 8 * (m + 1)
    prio_bytes = 20 * n                          # delta, logpi, logmu, entropy in; q out
    build_bytes = 4 * n + 8 * (n // 128)
    if getattr(args, "fused", False):   # r, V, logpi, logmu, entropy (+ scale) in; v_target, advantage, q out; offsets; tree levels 1-2
        retrace_bytes = (20 + (4 if w.heavy_tail else 0) + 12) * n + 8 * (m + 1) + 8 * (n // 128)
    return retrace_bytes, prio_bytes, build_bytes


def _config(w, args):
    l2 = "inputs larger than L2 (%.0f MB touched per step), two copies of the inputs alternate between steps" % (
        sum(_step_bytes(w, args)) / 1e6)
    return {"workload": "%s (configs[%d]): N=%d transitions, M=%d trajectories, batch k=%d, %d sample->update rounds"
                        % (w.name, w.index, w.n, w.m, w.batch, w.rounds),
            "gamma": w.gamma, "lambda": w.lam, "alpha": w.alpha, "beta": w.beta, "fixed_point_scale": w.scale,
            "parallelism": "independent replay shard per GPU (no data-path collective)" if args.gpus > 1 else "1 GPU",
            "l2": l2,
            "fused_pass": bool(getattr(args, "fused", False)), "rounds_launch": "eager" if getattr(args, "no_graph", False) else "caller-side CUDA graph of the rounds"}


# --------------------------------------------------------------------------- CUDA legs

class ClockSampler:
    def __init__(self, uuid):
        self.path = "/tmp/distrl_clocks_%d.csv" % os.getpid()
        self.f = open(self.path, "w")
        q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", uuid, "--query-gpu=" + q, "--format=csv,noheader,nounits",
                                       "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None
        self.t_mark = None

    def mark(self):
        """Samples taken from now on count as 'under load'."""
        import datetime
        self.t_mark = datetime.datetime.now()

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.p is None:
            return out
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.close()
        import datetime
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = []
        try:
            for ln in open(self.path):
                parts = [x.strip() for x in ln.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f")
                    rows.append((ts, float(parts[1]), float(parts[2]),
                                 [nm for nm, val in zip(names, parts[5:9]) if val.lower().startswith("active")]))
                except ValueError:
                    continue
            os.remove(self.path)
        except Exception:
            pass
        load = [r for r in rows if self.t_mark is None or r[0] >= self.t_mark] or rows
        if load:
            out = {"sm_mhz": float(np.median([r[1] for r in load])), "sm_max_mhz": float(max(r[2] for r in load)),
                   "reasons": sorted({nm for r in load for nm in r[3]}), "samples": len(load)}
        return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2410_14803_b200 as distrl
    from paper_2410_14803_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    w = synth.make_workload(WORKLOAD_INDEX[args.workload], n_override=args.n_override, shard=rank)  # one shard per rank
    a = w.arrays
    n, k, R = w.n, w.batch, w.rounds
    cfg = distrl.make_prio_cfg(w.w_td, w.w_rho, w.w_ent, w.rho_clip, w.alpha, w.scale)

    # ---- host (pinned) copies: the e2e leg starts from these every step
    tok = w.token_level
    names = ["traj_offsets", "rewards", "values", "entropy"] + \
            (["step_token_offsets", "tok_logp_target", "tok_logp_behaviour"] if tok else ["logp_target", "logp_behaviour"])
    as_t = lambda nm: torch.from_numpy(a[nm]).view(torch.bfloat16) if nm.startswith("tok_") else torch.from_numpy(a[nm])
    host = {nm: as_t(nm).pin_memory() for nm in names}
    u_all = np.stack([synth.uniforms(w, r) for r in range(R)]).view(np.int64)
    nd_all = np.stack([synth.fresh_abs_delta(w, r) for r in range(R)])
    host_u, host_nd = torch.from_numpy(u_all).pin_memory(), torch.from_numpy(nd_all).pin_memory()
    tail = torch.from_numpy(synth.heavy_tail_scale(w)).cuda() if w.heavy_tail else None

    f32 = lambda: torch.empty(n, dtype=torch.float32, device="cuda")
    vt, adv, dl = f32(), f32(), f32()
    q = torch.empty(n, dtype=torch.int32, device="cuda")
    idx = torch.empty((R, k), dtype=torch.int64, device="cuda")
    wts = torch.empty((R, k), dtype=torch.float32, device="cuda")
    ws_r = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(n))
    ws_s = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(n))
    distrl.distrl_workspace_init(ws_r)
    distrl.distrl_workspace_init(ws_s)

    class InputSet:
        """One device copy of a step's inputs (the e2e leg alternates between two, so that the upload of
        the next step's inputs overlaps the current step), with the batch descriptor over it."""

        def __init__(self):
            self.dv = {nm: host[nm].cuda() for nm in names}
            self.d_u, self.d_nd = host_u.cuda(), host_nd.cuda()
            dv = self.dv
            if tok:   # per-step log-probs are the token sums the Retrace pass writes out
                self.lp_buf, self.lm_buf = f32(), f32()
                self.batch = distrl.make_batch(dv["traj_offsets"], dv["rewards"], dv["values"], None, None, None,
                                               dv["step_token_offsets"], dv["tok_logp_target"], dv["tok_logp_behaviour"])
            else:
                self.lp_buf, self.lm_buf = dv["logp_target"], dv["logp_behaviour"]
                self.batch = distrl.make_batch(dv["traj_offsets"], dv["rewards"], dv["values"], self.lp_buf, self.lm_buf)
            self.lp_out, self.lm_out = (self.lp_buf, self.lm_buf) if tok else (None, None)
            self.graph = None

        def upload(self):
            for nm in names:
                self.dv[nm].copy_(host[nm], non_blocking=True)
            self.d_u.copy_(host_u, non_blocking=True)
            self.d_nd.copy_(host_nd, non_blocking=True)

    main_set = InputSet()
    sets = [main_set, InputSet()]   # two copies of the inputs: consecutive steps never read the same arrays

    # The heavy-tailed critic error of workload 3 is workload synthesis, not part of the method: the
    # scaled |delta| array that the priority stage reads is prepared once from the same td_delta the
    # Retrace stage writes every step (bit-identical each step), so no foreign kernel runs in the timed region.
    distrl.distrl_retrace_targets(main_set.batch, w.gamma, w.lam, vt, adv, dl, main_set.lp_out, main_set.lm_out,
                                  workspace=ws_r)
    prio_in = (dl * tail) if tail is not None else dl
    # real masses before the rounds are recorded below (their first, unrecorded run draws from q)
    distrl.distrl_compute_priorities(prio_in, main_set.lp_buf, main_set.lm_buf, main_set.dv["entropy"], cfg, None, q)
    torch.cuda.synchronize()

    ev = lambda: torch.cuda.Event(enable_timing=True)
    # a refresh of up to 8192 positions is one launch, a longer one a claim and an apply launch per 65536 positions
    per_round = 1 + (1 if (k <= 8192 and n < 2 ** 31) else 2 * ((k + 65535) // 65536))
    retrace_launches = 5 if tok else 2   # end mask + scan (token-level: + the dense instance and the general pair, which return at once)
    launches_per_step = retrace_launches + 1 + 2 + per_round * R   # Retrace, priorities, 2 build, (sample, refresh) x R
    if args.fused:
        launches_per_step = 3 + per_round * R       # end mask + fused scan + upper tree levels, then the rounds

    def rounds(s, ins):
        for r in range(R):
            distrl.distrl_sample(s, ins.d_u[r], w.beta, True, idx[r], wts[r])
            distrl.distrl_update_priorities(s, idx[r], ins.d_nd[r], ins.lp_buf, ins.lm_buf, ins.dv["entropy"], cfg, None)

    # The R sample->refresh rounds are launch-bound (3 short kernels each), so the caller records them once
    # into a CUDA graph and replays it every step.  The sampler handle only holds pointers into ws_s and q,
    # which never move, so the recorded launches stay valid when the tree is rebuilt each step.
    s_graph = None

    def record_rounds(ins):
        nonlocal s_graph
        if args.no_graph:
            return
        if s_graph is None:
            s_graph = distrl.distrl_build_sampler(q, ws_s)
        rounds(s_graph, ins)                  # first use outside capture (one-time function attributes)
        torch.cuda.synchronize()
        ins.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(ins.graph):
            rounds(s_graph, ins)
        torch.cuda.synchronize()

    for ins_ in sets:
        record_rounds(ins_)

    def step(marks=None, ins=main_set):
        if args.fused:   # Retrace + priorities + sampler build in one pass over the buffer
            if marks: marks[0].record()
            s = distrl.distrl_retrace_priorities_build(ins.batch, w.gamma, w.lam, ins.dv["entropy"], tail, cfg, vt, adv,
                                                       None, q, None, retrace_workspace=ws_r, sampler_workspace=ws_s)
            if marks:
                marks[1].record(); marks[2].record(); marks[3].record()
            if ins.graph is not None:
                ins.graph.replay()
            else:
                rounds(s, ins)
            if marks: marks[4].record()
            s.close()
            return
        if marks: marks[0].record()
        distrl.distrl_retrace_targets(ins.batch, w.gamma, w.lam, vt, adv, dl, ins.lp_out, ins.lm_out, workspace=ws_r)
        if marks: marks[1].record()
        distrl.distrl_compute_priorities(prio_in, ins.lp_buf, ins.lm_buf, ins.dv["entropy"], cfg, None, q)
        if marks: marks[2].record()
        s = distrl.distrl_build_sampler(q, ws_s)
        if marks: marks[3].record()
        if ins.graph is not None:
            ins.graph.replay()
        else:
            rounds(s, ins)
        if marks: marks[4].record()
        s.close()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    uuid = "GPU-" + str(torch.cuda.get_device_properties(local).uuid).replace("GPU-", "")
    clocks = ClockSampler(uuid)
    for i in range(max(args.warmup, 3)):
        step(ins=sets[i & 1])
    barrier()
    marks = [[ev() for _ in range(5)] for _ in range(args.steps)]
    t_begin, t_end = ev(), ev()
    barrier()
    clocks.mark()
    t_begin.record()
    for i in range(args.steps):
        step(marks[i], ins=sets[i & 1])
    t_end.record()
    barrier()
    clk = clocks.stop()
    total_ms = t_begin.elapsed_time(t_end)
    stage_all = np.array([[m[i].elapsed_time(m[i + 1]) for i in range(4)] for m in marks])
    stage_ms, stage_med, stage_min = stage_all.mean(axis=0), np.median(stage_all, axis=0), stage_all.min(axis=0)
    st_r = distrl.distrl_get_status(ws_r)
    st_s = distrl.distrl_get_status(ws_s)
    if st_r or st_s:
        raise SystemExit("device status after the timed region: retrace %d sampler %d" % (st_r, st_s))

    # ---- the first stage back to back: in the step above one call stands alone between two events, so its figure
    # includes the idle time before its first kernel starts (about 4 us, which matters for a call of 87 us).  Here
    # calls follow one another, captured into a CUDA graph (the two copies of the inputs taken in turn) and replayed:
    # the time per call is what the kernels themselves take.
    b2b_ms = None
    if not args.no_graph:
        per = 10 if not tok else 4
        def first_stage(i):
            ins = sets[i & 1]
            if args.fused:
                distrl.distrl_retrace_priorities_build(ins.batch, w.gamma, w.lam, ins.dv["entropy"], tail, cfg, vt, adv, None, q,
                                                       None, retrace_workspace=ws_r, sampler_workspace=ws_s).close()
            else:
                distrl.distrl_retrace_targets(ins.batch, w.gamma, w.lam, vt, adv, dl, ins.lp_out, ins.lm_out, workspace=ws_r)
        for i in range(2):
            first_stage(i)
        torch.cuda.synchronize()
        g_b2b = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_b2b):
            for i in range(per):
                first_stage(i)
        g_b2b.replay()
        b0, b1 = ev(), ev()
        barrier()
        b0.record()
        for _ in range(10):
            g_b2b.replay()
        b1.record()
        barrier()
        b2b_ms = b0.elapsed_time(b1) / (10 * per)
        if distrl.distrl_get_status(ws_r):
            raise SystemExit("device status after the back-to-back leg")

    # ---- e2e: same step through the same calls, inputs from pinned host memory, results back to the host,
    # every step.  Three streams: uploads alternate between two device copies of the inputs, so the upload
    # of step i+1 runs while step i computes and step i-1's results travel back (PCIe is full duplex);
    # each step still waits for its own inputs, and nothing of a step is skipped or reused.
    h_vt = torch.empty(n, dtype=torch.float32).pin_memory()
    h_adv = torch.empty(n, dtype=torch.float32).pin_memory()
    h_idx = torch.empty((R, k), dtype=torch.int64).pin_memory()
    h_w = torch.empty((R, k), dtype=torch.float32).pin_memory()
    h2d = sum(host[nm].numel() * host[nm].element_size() for nm in names) + host_u.numel() * 8 + host_nd.numel() * 4
    d2h = 2 * 4 * n + R * k * 12
    e2e_steps = max(4, min(args.steps, 8))
    e2e_ms = float("nan")
    if not args.no_e2e:
        main_stream = torch.cuda.current_stream()
        up_stream, down_stream = torch.cuda.Stream(), torch.cuda.Stream()
        plain = lambda: torch.cuda.Event()
        uploaded = [plain(), plain()]     # inputs of the step using set b have arrived
        computed = [plain(), plain()]     # the step using set b has finished (its inputs may be overwritten)
        downloaded = plain()              # the previous step's results have left vt / adv / idx / wts

        def e2e_run(count):
            for i in range(count):
                b = i & 1
                with torch.cuda.stream(up_stream):
                    if i >= 2:
                        up_stream.wait_event(computed[b])
                    sets[b].upload()
                    uploaded[b].record(up_stream)
                main_stream.wait_event(uploaded[b])
                if i >= 1:
                    main_stream.wait_event(downloaded)
                step(ins=sets[b])
                computed[b].record(main_stream)
                with torch.cuda.stream(down_stream):
                    down_stream.wait_event(computed[b])
                    h_vt.copy_(vt, non_blocking=True)
                    h_adv.copy_(adv, non_blocking=True)
                    h_idx.copy_(idx, non_blocking=True)
                    h_w.copy_(wts, non_blocking=True)
                    downloaded.record(down_stream)
            main_stream.wait_event(downloaded)

        e2e_run(2)
        barrier()
        e0, e1 = ev(), ev()
        e0.record()
        e2e_run(e2e_steps)
        e1.record()
        barrier()
        e2e_ms = e0.elapsed_time(e1) / e2e_steps

    # ---- the entry points beyond the main path, each timed alone on the same buffer (not part of `value`):
    # Monte-Carlo returns + labels, trajectory-level priorities, a circular overwrite of 2^20 slots, and the
    # actor-loss coefficients of the whole buffer and of one drawn batch
    next_rows = None
    if args.next_rows and not tok:
        def timed(fn, reps=20):
            for _ in range(3):
                fn()
            t0, t1 = ev(), ev()
            torch.cuda.synchronize()
            t0.record()
            for _ in range(reps):
                fn()
            t1.record()
            torch.cuda.synchronize()
            return t0.elapsed_time(t1) / reps * 1e-3
        def timed_graph(fn, per=20, reps=10):
            # short calls: `per` of them captured into a CUDA graph (fn gets the call's number, so that it can
            # alternate between two sets of arrays) and replayed, so that the host's launch rate does not
            # bound the figure
            for i in range(4):
                fn(i)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in range(per):
                    fn(i)
            return timed(g.replay, reps) / per
        ins = main_set
        g_ret, lab = f32(), torch.empty(n, dtype=torch.uint8, device="cuda")
        t_mc = timed_graph(lambda i: distrl.distrl_mc_returns(sets[i & 1].batch, w.gamma, g_ret, lab, workspace=ws_r))
        # Retrace with a bootstrap value per trajectory (the pipelined kernel's other instance)
        boot_v = torch.rand(w.m, dtype=torch.float32, device="cuda")
        boot_batches = [distrl.make_batch(x.dv["traj_offsets"], x.dv["rewards"], x.dv["values"], x.lp_buf, x.lm_buf, boot_v)
                        for x in sets]
        t_bt = timed_graph(lambda i: distrl.distrl_retrace_targets(boot_batches[i & 1], w.gamma, w.lam, vt, adv, dl,
                                                                   workspace=ws_r))
        # token-level Retrace on a dense buffer (32 tokens per step, 8 M steps, trajectories of 10 steps): the
        # instance of the pipelined token kernel with one step per lane
        nd, per = 8_000_000, 32
        d_sto = torch.arange(0, (nd + 1) * per, per, dtype=torch.int64, device="cuda")
        d_tm = torch.randn(nd * per, device="cuda").mul_(0.3).sub_(0.3).to(torch.bfloat16)
        d_tp = (d_tm.float() + torch.randn(nd * per, device="cuda") * 0.05).to(torch.bfloat16)
        d_off = torch.arange(0, nd + 1, 10, dtype=torch.int64, device="cuda")
        d_r, d_v = torch.randn(nd, device="cuda"), torch.rand(nd, device="cuda")
        d_batch = distrl.make_batch(d_off, d_r, d_v, None, None, None, d_sto, d_tp, d_tm)
        d_out = [torch.empty(nd, dtype=torch.float32, device="cuda") for _ in range(5)]
        ws_d = distrl.alloc_workspace(distrl.distrl_retrace_workspace_bytes(nd))
        distrl.distrl_workspace_init(ws_d)
        t_td = timed_graph(lambda i: distrl.distrl_retrace_targets(d_batch, w.gamma, w.lam, *d_out, workspace=ws_d), per=5)
        if distrl.distrl_get_status(ws_d):
            raise SystemExit("device status after the dense token-level call")
        td_bytes = 36 * nd + 4 * nd * per + 8 * (nd // 10 + 1)
        del d_tm, d_tp, d_out
        q_traj = torch.empty(w.m, dtype=torch.int32, device="cuda")
        t_tr = timed_graph(lambda i: distrl.distrl_compute_priorities_traj(
            sets[i & 1].dv["traj_offsets"], prio_in, sets[i & 1].lp_buf, sets[i & 1].lm_buf, sets[i & 1].dv["entropy"],
            cfg, None, q_traj))
        s_tmp = distrl.distrl_build_sampler(q, ws_s)
        k_over = min(1 << 20, n)
        new_q = torch.randint(1, 1 << 24, (k_over,), dtype=torch.int32, device="cuda")
        t_ov = timed_graph(lambda i: distrl.distrl_replay_overwrite(s_tmp, n - k_over // 2, new_q))
        s_tmp.close()
        coef_all, coef_k = f32(), torch.empty(k, dtype=torch.float32, device="cuda")
        t_ca = timed_graph(lambda i: distrl.distrl_actor_coefficients(sets[i & 1].lp_buf, sets[i & 1].lm_buf,
                                                                      (adv, vt)[i & 1], coef_all))   # vt: a second array of advantages' size
        # one drawn batch: 20 calls (one per round's batch) replayed from a CUDA graph, so that the
        # figure is the device's and not the Python caller's
        def coef_batches():
            for r in range(20):
                distrl.distrl_actor_coefficients(ins.lp_buf, ins.lm_buf, adv, coef_k, idx=idx[r % R],
                                                 is_weight=wts[r % R])
        coef_batches()
        torch.cuda.synchronize()
        g_ck = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_ck):
            coef_batches()
        t_ck = timed(g_ck.replay) / 20
        # two sets of offsets, scores and masses (168 MB together, more than L2), taken in turn
        q_f = [q.clone(), q.clone()]
        v_traj = [torch.rand(w.m, dtype=torch.float32, device="cuda") for _ in range(2)]   # stand in for V_traj's scores
        t_fl = timed_graph(lambda i: distrl.distrl_filter_trajectories(sets[i & 1].dv["traj_offsets"], v_traj[i & 1], 0.5,
                                                                       q_f[i & 1]))
        # the same on one set of arrays: masses, offsets and scores (84 MB) stay in L2, as the masses do when the
        # call follows the priorities call that wrote them
        t_fl_warm = timed_graph(lambda i: distrl.distrl_filter_trajectories(sets[0].dv["traj_offsets"], v_traj[0], 0.5, q_f[0]))
        # circular buffer of trajectories: one ingest of 512 new trajectories (their rows and masses already on the
        # device, their lengths known on the host) into a ring of N slots with its sampler kept exact
        ring_f = [f32() for _ in range(5)]
        ring_q = torch.empty(n, dtype=torch.int32, device="cuda")
        m_cap = w.m + 4096
        ring_off = torch.empty(m_cap + 1, dtype=torch.int64, device="cuda")
        ring_alive = torch.empty(m_cap, dtype=torch.float32, device="cuda")
        ws_ring = distrl.alloc_workspace(distrl.distrl_replay_workspace_bytes(n))
        rb = distrl.distrl_replay_create(ring_f, ring_q, ring_off, ring_alive, ws_ring)
        ws_rs = distrl.alloc_workspace(distrl.distrl_sampler_workspace_bytes(n))
        distrl.distrl_workspace_init(ws_rs)
        s_ring = distrl.distrl_build_sampler(ring_q, ws_rs)
        new_off = a["traj_offsets"][:513].copy()
        rows_new = int(new_off[-1])
        d_new_off = torch.from_numpy(new_off).cuda()
        new_fields = [ins.dv["rewards"][:rows_new], ins.dv["values"][:rows_new], ins.lp_buf[:rows_new],
                      ins.lm_buf[:rows_new], ins.dv["entropy"][:rows_new]]
        new_mass = q[:rows_new].clone()
        t_in = timed(lambda: distrl.distrl_replay_ingest(rb, s_ring, new_off, d_new_off, new_fields, new_mass))
        if distrl.distrl_get_status(ws_ring) or distrl.distrl_get_status(ws_rs):
            raise SystemExit("device status after the ring ingest")
        s_ring.close()
        rb.close()
        mc_bytes, tr_bytes = 9 * n + 8 * (w.m + 1), 16 * n + 8 * (w.m + 1) + 4 * w.m
        bt_bytes = 28 * n + 8 * (w.m + 1) + 4 * w.m      # the Retrace call's bytes and one bootstrap value per trajectory
        next_rows = {
            "mc_returns": {"ms": t_mc * 1e3, "gbs": mc_bytes / t_mc / 1e9, "frac": mc_bytes / t_mc / 1e9 / _peaks()[0]},
            "retrace_bootstrap": {"ms": t_bt * 1e3, "gbs": bt_bytes / t_bt / 1e9, "frac": bt_bytes / t_bt / 1e9 / _peaks()[0]},
            "retrace_tokens_dense": {"steps": nd, "tokens_per_step": per, "ms": t_td * 1e3, "gbs": td_bytes / t_td / 1e9,
                                     "frac": td_bytes / t_td / 1e9 / _peaks()[0]},
            "priorities_traj": {"ms": t_tr * 1e3, "gbs": tr_bytes / t_tr / 1e9, "frac": tr_bytes / t_tr / 1e9 / _peaks()[0]},
            "replay_overwrite": {"slots": k_over, "ms": t_ov * 1e3, "slots_per_s": k_over / t_ov},
            "actor_coefficients_buffer": {"ms": t_ca * 1e3, "gbs": 16 * n / t_ca / 1e9,
                                          "frac": 16 * n / t_ca / 1e9 / _peaks()[0]},
            "actor_coefficients_batch": {"k": k, "us": t_ck * 1e6},
            "filter_trajectories": {"ms": t_fl * 1e3, "dropped_fraction": 0.5, "transitions_per_s": n / t_fl,
                                    "gbs": (8 * (w.m + 1) + 4 * w.m + 2 * n) / t_fl / 1e9,   # offsets, scores, zeros over half the steps
                                    "frac": (8 * (w.m + 1) + 4 * w.m + 2 * n) / t_fl / 1e9 / _peaks()[0],
                                    "ms_l2_warm": t_fl_warm * 1e3,
                                    "gbs_l2_warm": (8 * (w.m + 1) + 4 * w.m + 2 * n) / t_fl_warm / 1e9},
            "replay_ingest": {"trajectories": 512, "rows": rows_new, "us": t_in * 1e6},
        }
        if distrl.distrl_get_status(ws_r) or distrl.distrl_get_status(ws_s):
            raise SystemExit("device status after the extra entry points")

    ms_per_step = total_ms / args.steps
    from paper_2410_14803_b200.shard import max_over_ranks
    ms_per_step, e2e_ms = max_over_ranks([ms_per_step, e2e_ms], device="cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    peak, peak_kind = _peaks()
    retrace_bytes, prio_bytes, build_bytes = _step_bytes(w, args)
    ach = retrace_bytes / (stage_ms[0] * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": world * n / (ms_per_step * 1e-3), "unit": METRIC, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": _config(w, args),
        "stages": {
            # with --fused the first stage is the one fused pass and the next two are empty
            "retrace_ms": float(stage_ms[0]), "priorities_ms": None if args.fused else float(stage_ms[1]),
            "build_sampler_ms": None if args.fused else float(stage_ms[2]),
            "rounds_ms": float(stage_ms[3]), "us_per_round": float(1e3 * stage_ms[3] / R),
            "retrace_priority_transitions_per_s": n / ((stage_ms[0] + stage_ms[1]) * 1e-3),
            "samples_per_s": R * k / (stage_ms[3] * 1e-3),
            "priorities_gbs": None if args.fused else prio_bytes / (stage_ms[1] * 1e-3) / 1e9,
            "build_sampler_gbs": None if args.fused else build_bytes / (stage_ms[2] * 1e-3) / 1e9,
            # the figures above are means over the timed steps; median and minimum of the same per-step timings
            "median_ms": {"retrace": float(stage_med[0]), "priorities": None if args.fused else float(stage_med[1]),
                          "build_sampler": None if args.fused else float(stage_med[2]), "rounds": float(stage_med[3])},
            "min_ms": {"retrace": float(stage_min[0]), "priorities": None if args.fused else float(stage_min[1]),
                       "build_sampler": None if args.fused else float(stage_min[2]), "rounds": float(stage_min[3])},
            "timed_steps": int(args.steps),
        },
        "roofline": {"bound": "hbm", "kernel": ("scan_mask_kernel + scan_pipe_kernel<fused> (distrl_retrace_priorities_build)" if args.fused else "scan_mask_kernel + %s (distrl_retrace_targets)" % ("scan_tok_pipe_kernel (+ three stand-ins for dense buffers that return at once)" if tok else "scan_pipe_kernel")), "achieved": ach, "peak": peak,
                     "unit": "GB/s", "frac": ach / peak, "peak_kind": "of " + peak_kind,
                     "frac_of_nominal_8000": ach / 8000.0, "traffic": _measured_traffic(w.name) if (args.n_override is None and not args.fused) else None,
                     "algorithmic_bytes": retrace_bytes,
                     # the same call when calls follow one another (graph-replayed; see the comment at that leg)
                     "back_to_back": None if b2b_ms is None else {
                         "ms_per_call": b2b_ms, "achieved": retrace_bytes / (b2b_ms * 1e-3) / 1e9,
                         "frac": retrace_bytes / (b2b_ms * 1e-3) / 1e9 / peak}},
        "e2e": {"value": world * n / (e2e_ms * 1e-3) if e2e_ms == e2e_ms else None, "unit": METRIC,
                "ms_per_step": e2e_ms if e2e_ms == e2e_ms else None,   # None: leg skipped with --no-e2e
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": launches_per_step * args.steps,
        "clocks": clk,
    }
    if next_rows is not None:
        line["next_rows"] = next_rows
    if not args.no_cpu_baseline and world == 1:
        est, desc, _ = _oracle_sample(w, 2_000_000, draws=48)
        line["cpu_baseline"] = {"value": w.n / est, "unit": METRIC, "cores": 1, "kind": "oracle", "sample": desc,
                                "estimated": True}
        if not tok:
            try:
                v_mc, cores, desc_mc = _oracle_all_cores(w)
                line["cpu_baseline"]["multi_core"] = {"value": v_mc, "unit": "transitions/s (Retrace + priority only)",
                                                      "cores": cores, "kind": "oracle", "sample": desc_mc}
            except Exception as e:   # the one-core figure stands on its own
                line["cpu_baseline"]["multi_core"] = {"value": None, "error": repr(e)[:200]}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def _measured_traffic(workload_name):
    """dram__bytes_read.sum + dram__bytes_write.sum per call of the Retrace entry point, from the profiler capture
    recorded in profiles/traffic.json (written by `python -m paper_2410_14803_b200.ncu_summary`).  The record names
    the kernel sources it was taken with; once they have changed the counters are stale and None is reported."""
    try:
        from paper_2410_14803_b200 import ncu_summary
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            rec = json.load(f).get(workload_name)
        if not rec or rec.get("source_sha256") != ncu_summary.kernel_sources_sha256(rec.get("sources")):
            return None
        return int(rec["bytes_per_call"])
    except Exception:
        return None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=sorted(WORKLOAD_INDEX), default="large")
    ap.add_argument("--n-override", type=int, default=None,
                    help="shrink a fixed-N workload to this many transitions (profiler captures; not a bench line)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--fused", action="store_true",
                    help="use distrl_retrace_priorities_build (one pass) instead of the three separate calls")
    ap.add_argument("--no-graph", action="store_true", help="launch the sampling rounds one call at a time")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--next-rows", action="store_true",
                    help="also time the entry points beyond the main path, each alone on the same buffer")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
