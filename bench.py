#!/usr/bin/env python
"""Benchmark of the BalanceRoute routing step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A "step" is one call of br_step: one launch of the whole routing path (ARRIVE, PREDICT, ROUTE,
RECORD, ADVANCE) over one batch of 4,096 independent BR-0 instances (G = 32, 256 waiting each:
the batched HBM-throughput configuration), advancing every instance by --steps-per-launch
decode steps (16, or with a short timed region the number with which its calls cover the
configuration once; `config.steps_per_launch` says which).  The timed
region of --steps calls is repeated --repeats times, each repeat on instance sets put back to
their starting snapshots; the median repeat is reported, minimum and
maximum beside it.  Several instance sets are stepped in rotation so that the data touched
between two visits of the same set exceeds the L2 cache; they start at evenly spaced points of
the configuration's trajectory, so that a short timed region still samples all of it.  Prints one JSON line whose last key,
`summary`, repeats every headline figure in compact form.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2605_06113_b200 import workload as wlm  # noqa: E402

UNIT = "instance-steps/s"
METRICS = {
    "c3": "routing instance-steps/sec (batched BR-0, 4096 instances, G=32, W=256)",
    "c4": "routing instance-steps/sec (batched BR-H H=8, 1024 instances, G=64, W=1024)",
    "h80": "routing instance-steps/sec (batched BR-H H=80 with perfect lookahead, 1024 instances, G=8, W=512)",
}
WORKLOADS = {
    "c3": "c3: BR-0 batched, 4096 instances/GPU, G=32, B=64, W=256, seeds 100..",
    "c4": "c4: BR-H H=8 batched, 1024 instances/GPU, G=64, B=64, W=1024, seeds 5000..",
    "h80": "h80: BR-H H=80 (the paper's deployed horizon), perfect-lookahead predictor, requests with lifetimes, "
           "1024 instances/GPU, G=8, B=64, W=512, seeds 9000..",
}
BATCH_INSTANCES = {"h80": 1024}          # workloads defined on one instance, benchmarked as a batch
ARRIVALS_PER_STEP = {"c3": 10.0, "c4": 20.0, "h80": 0.7, "c2": 8.0}
L2_BYTES = 126 * 1024 * 1024
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


# ----------------------------------------------------------------------------- helpers
def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def kernel_source_hash() -> str:
    """Hash of the CUDA sources; the DRAM-traffic figures under profiles/ are valid only for
    the kernel they were captured on."""
    import hashlib
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2605_06113_b200", "csrc")
    for f in ("br_device.cuh", "br_small.cuh", "br_step.cuh"):       # the files that define the step kernels
        h.update(open(os.path.join(d, f), "rb").read())
    return h.hexdigest()[:16]


def _recorded(field: str, workload: str, spl: int):
    """A per-launch counter from the ncu captures in profiles/traffic.json.  For a launch shape that
    was not captured itself the figure is interpolated linearly in the steps per launch between
    the two shapes that were (the first step of a launch reads the state from DRAM, every further
    step adds the same amount)."""
    p = os.path.join(ROOT, "profiles", "traffic.json")
    try:
        rec = json.load(open(p))
        if rec.get("kernel_source_hash") != kernel_source_hash():
            return None
        tab = rec.get(field, {})
        if f"{workload}_spl{spl}" in tab:
            return tab[f"{workload}_spl{spl}"]
        pts = sorted((int(k.rsplit("spl", 1)[1]), v) for k, v in tab.items() if k.startswith(workload + "_spl"))
        if len(pts) >= 2:
            (s0, v0), (s1, v1) = pts[0], pts[-1]
            return v0 + (v1 - v0) * (spl - s0) / (s1 - s0)
    except Exception:
        pass
    return None


def recorded_traffic(workload: str, spl: int = 1):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture recorded in
    profiles/traffic.json, or None if the kernel sources changed since that capture."""
    return _recorded("bytes_per_launch", workload, spl)


def recorded_instructions(workload: str, spl: int = 1):
    """Warp instructions per launch from the same ncu capture (None if the kernel changed)."""
    return _recorded("warp_instructions_per_launch", workload, spl)


def algorithmic_bytes(cfg, edits_per_step: float, rho: float) -> float:
    """Bytes one instance-step has to move once: running-request state in, queue in,
    assignments out, per-worker state in and out, slot edits; for BR-H the prediction state
    (4 bytes per slot read, 4 / Delta_T written) and the classifier rows of the refreshed
    requests.  The library stores the prediction state in 5 bytes per slot (fp32 c_hat plus a
    one-byte refresh stamp); the extra byte is layout cost and is not counted here."""
    A, G, W, H = cfg.G * cfg.B, cfg.G, cfg.W, cfg.H
    b = 4.0 * A + 8.0 * W + 4.0 * W + 20.0 * G + 28.0 * G + 24.0 + 8.0 * edits_per_step
    if H > 0 and cfg.pred_mode == 1:
        b += 4.0 * A + 8.0 * W           # perfect lookahead: the step each request ends at; output lengths of the queue
    elif H > 0:
        b += 4.0 * A + 4.0 * H * A * rho + 4.0 * A / cfg.delta_T
    return b


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "10"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self, t0=None, t1=None):
        """Summary of the samples taken between host times t0 and t1 (all samples if none fall inside)."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is not None:
            self.p.terminate()
            try:
                self.p.wait(timeout=5)
            except Exception:
                self.p.kill()
        try:
            self.f.flush()
            rows = [l.strip().split(", ") for l in open(self.f.name) if l.strip()]
            rows = [r for r in rows if len(r) >= 9]
            if t0 is not None:
                import datetime

                def ts(r):
                    return datetime.datetime.strptime(r[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                inside = [r for r in rows if t0 <= ts(r) <= t1]
                out["samples_total"] = len(rows)
                if inside:
                    rows = inside
            sm = [float(r[1]) for r in rows if len(r) >= 9]
            if sm:
                out["sm_mhz"] = float(np.median(sm))
                out["sm_max_mhz"] = float(rows[0][2])
                out["samples"] = len(sm)
                names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
                for j, n in enumerate(names):
                    if any(r[5 + j].strip().lower() == "active" for r in rows if len(r) >= 9):
                        out["reasons"].append(n)
            os.unlink(self.f.name)
        except Exception:
            pass
        return out


def shard_of(rank: int, world: int, instances_per_rank: int, sets: int = 1):
    """First instance and instance count owned by `rank`: ranks own disjoint, equally sized
    seed ranges (weak scaling); there is no exchange between ranks on the data path."""
    n = instances_per_rank * sets
    return rank * n, n


def max_over_ranks(ms: float, dist, device="cuda") -> float:
    """Timed region of the job = the slowest rank's."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def dist_setup(args):
    import torch
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        if args.impl == "reference":
            return world, rank, local, None
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
        return world, rank, local, dist
    return world, rank, local, None


def steps_per_launch_for(cfg, asked: int, calls: int = 0) -> int:
    """Decode steps per br_step call.  What was asked for, if anything; else 16, or, when the timed
    region has too few calls to walk one configuration length at 16 steps per call, the number
    (at most 32) with which `calls` calls cover the configuration's steps exactly once, the
    rotating sets taking one stretch of the trajectory each."""
    if asked > 0:
        return max(1, min(asked, cfg.steps))
    if calls > 0 and calls * 16 < cfg.steps:
        return max(1, min(32, -(-cfg.steps // calls)))
    return 16


# ----------------------------------------------------------------------------- CPU arm
def _oracle_worker(job):
    """Runs the CPU checker on instances [first, first + n) of a configuration for at most
    `budget_s` seconds or `max_steps` decode steps (a top-level function: pool workers are
    started with `spawn`)."""
    cfg_name, first, n, max_steps, budget_s = job
    import oracle
    cfg = wlm.get_config(cfg_name)
    wl = wlm.make_workload(cfg, n_instances=n, first_instance=first)
    orcs = [oracle.instance_from_workload(wl, i) for i in range(n)]
    probs = [wlm.term_probs_np(wl, k) for k in range(min(max_steps, 4))] if cfg.H > 0 and cfg.pred_mode == 0 else None
    done = 0
    t0 = time.perf_counter()
    for k in range(max_steps):
        for i, o in enumerate(orcs):
            o.step(None if probs is None else probs[k % len(probs)][i])
        done += n
        if time.perf_counter() - t0 > budget_s:
            break
    return done, time.perf_counter() - t0


def oracle_rate(cfg_name: str, budget_s: float, n_inst: int, max_steps: int):
    """Instance-steps/s of the CPU checker, single thread, on the first n_inst instances."""
    done, dt = _oracle_worker((cfg_name, 0, n_inst, max_steps, budget_s))
    return done / dt, done, dt


def oracle_rate_all_cores(cfg_name: str, budget_s: float, n_per_proc: int, max_steps: int):
    """Aggregate instance-steps/s of the checker with one process per host core, each on its own
    instances.  The pool is started with `spawn` (a fork after CUDA initialisation can hang)."""
    import multiprocessing as mp
    cores = len(os.sched_getaffinity(0))
    jobs = [(cfg_name, p * n_per_proc, n_per_proc, max_steps, budget_s) for p in range(cores)]
    with mp.get_context("spawn").Pool(cores) as pool:
        t0 = time.perf_counter()
        res = pool.map(_oracle_worker, jobs)
        wall = time.perf_counter() - t0
    done = sum(r[0] for r in res)
    rate = sum(r[0] / r[1] for r in res)
    return rate, done, wall, cores


def cpu_baselines(args):
    """The checker as it stands on the host cores: the headline workload on one thread and on all
    cores, and the other configurations on one thread, each on a bounded sample."""
    out = {}
    rate, done, dt = oracle_rate("c3", 12.0, 512, 500)
    out["c3"] = {"value": rate, "unit": UNIT, "cores": 1, "kind": "oracle",
                 "sample": f"{done} instance-steps of c3 (first 512 instances, steps 0..{done // 512 - 1}), "
                           f"{dt:.1f} s, single thread"}
    try:
        rate, done, wall, cores = oracle_rate_all_cores("c3", 6.0, 64, 500)
        out["c3_all_cores"] = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                               "sample": f"{done} instance-steps of c3, {cores} processes x 64 instances, "
                                         f"{wall:.1f} s wall including process start"}
    except Exception as ex:
        out["c3_all_cores"] = {"error": repr(ex)}
    for name, n, steps, budget in (("c4", 32, 100, 4.0), ("c1", 32, 2000, 3.0), ("c2", 32, 2000, 3.0)):
        rate, done, dt = oracle_rate(name, budget, n, steps)
        out[name] = {"value": rate, "unit": UNIT, "cores": 1, "kind": "oracle",
                     "ms_per_instance_step": 1e3 / rate,
                     "sample": f"{done} instance-steps of {name} ({n} instance(s)), {dt:.1f} s, single thread"}
    return out


def run_reference(args):
    """The CPU checker as it stands, timed on host cores (rank 0 only).  One step is the same
    unit as on the GPU arm (--steps-per-launch decode steps of the batch), carried out on a
    bounded sample of the batch: its first 32 instances."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    cfg = wlm.get_config("c3")
    n_inst = 32
    spl = steps_per_launch_for(cfg, args.steps_per_launch, args.steps)
    steps = args.steps
    wl = wlm.make_workload(cfg, n_instances=n_inst)
    orcs = [oracle.instance_from_workload(wl, i) for i in range(n_inst)]
    for _ in range(args.warmup * spl):
        for o in orcs:
            o.step()
    t0 = time.perf_counter()
    for _ in range(steps * spl):
        for o in orcs:
            o.step()
    dt = time.perf_counter() - t0
    val = n_inst * steps * spl / dt
    line = {
        "impl": "reference", "metric": METRICS["c3"], "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
        "data": "synthetic",
        "config": {"workload": WORKLOADS["c3"], "steps_per_launch": spl,
                   "sample": f"the first {n_inst} instances, {spl} decode steps of each per step"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"{n_inst} instances x {steps * spl} decode steps of c3, single thread"},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- GPU arm
class RotatingSets:
    """R independent instance sets of one configuration, stepped in rotation; one call of
    step() is one launch that advances one set by `spl` decode steps.  reset() puts every set
    back to its initial snapshot (device copies), so that repeats time the same work."""

    def __init__(self, cfg_name, n_inst, n_sets, device, seed_offset=0, threads=0, probs_ring=1, spl=1,
                 start_steps=None, **params):
        import torch
        from paper_2605_06113_b200.binding import Router
        self.torch = torch
        self.cfg = wlm.get_config(cfg_name)
        self.N, self.n_sets, self.spl = n_inst, n_sets, spl
        self.sets = []
        for r in range(n_sets):
            wl = wlm.make_workload(self.cfg, n_instances=n_inst, first_instance=seed_offset + r * n_inst)
            router = Router(wl, device=device, threads=threads, **params)
            st = router.device_state()
            st0 = {k: v.clone() for k, v in st.items()}
            out = router.outputs(n_inst, n_steps=spl)
            probs = []
            if self.cfg.H > 0 and self.cfg.pred_mode == 0:      # classifier rows (the perfect-lookahead predictor reads none)
                seeds_t = torch.from_numpy(wl.seeds.astype(np.int64)).to(device)
                tab_t = torch.from_numpy(wl.beta_tab).to(device)
                for j in range(max(1, probs_ring)):
                    probs.append(torch.stack([wlm.term_probs_torch(wl, j * spl + i, device, seeds_t=seeds_t, tab_t=tab_t)
                                              for i in range(spl)]).contiguous())
            calls = [router.prepare(st, out, pr, N=n_inst, first=0, n_steps=spl) for pr in (probs or [None])]
            self.sets.append(dict(wl=wl, router=router, st=st, st0=st0, out=out, probs=probs, calls=calls))
        self.router = self.sets[0]["router"]
        self.launch = 0
        # Sets may start at different points of the configuration's trajectory (untimed launches
        # bring them there); the snapshot that reset() restores is taken afterwards.
        self.start_steps = [0] * n_sets
        if start_steps is not None:
            for j, s in enumerate(self.sets):
                n = int(start_steps[j]) // spl
                for i in range(n):
                    s["calls"][i % len(s["calls"])]()
                self.start_steps[j] = n * spl
            torch.cuda.synchronize()
            for s in self.sets:
                s["st0"] = {k: v.clone() for k, v in s["st"].items()}

    def step(self):
        s = self.sets[self.launch % self.n_sets]
        s["calls"][(self.launch // self.n_sets) % len(s["calls"])]()
        self.launch += 1

    def reset(self):
        for s in self.sets:
            for k, v in s["st"].items():
                v.copy_(s["st0"][k])
        self.launch = 0

    def counters_mean(self):
        t = self.torch
        return t.stack([s["out"]["counters"].to(t.float64).mean(dim=(0, 1)) for s in self.sets]).mean(0).cpu().numpy()

    def bad_status(self):
        return sum(int((s["out"]["status"] & ~1).ne(0).sum().item()) for s in self.sets)

    def close(self):
        for s in self.sets:
            s["router"].close()
        self.sets = []


def time_region(torch, fn, steps, dist=None):
    """Device time of exactly `steps` calls of fn, bracketed by a barrier and a device
    synchronisation on both sides; the slowest rank's time."""
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
        torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    if dist is not None:
        ms = max_over_ranks(ms, dist)
        dist.barrier()
        torch.cuda.synchronize()
    return ms


def measure_batched(torch, wname, device, launches, warmup, spl, repeats=5, threads=0,
                    seed_offset=0, dist=None, sampler=None, probs_ring=2, n_inst=None):
    """Times `launches` br_step calls of the batched configuration `wname`, `spl` decode steps per
    call, `repeats` times.  Enough instance sets rotate that the data between two visits of a set
    exceeds L2 and that no instance runs past the configuration's length.  The work of a decode
    step changes along a configuration's trajectory (c3 starts with half-empty workers and a full
    queue, so its first ~80 steps admit several times more requests than the rest), so the sets
    start at evenly spaced points of the trajectory and the timed region is a stratified sample of
    it (the whole of it, step 0 included, when launches * spl reaches sets * configuration length:
    the default arguments do that for c3).  Before every repeat the sets return to their starting
    snapshots; `warmup` untimed calls precede the first repeat."""
    cfg = wlm.get_config(wname)
    N = cfg.N if n_inst is None else n_inst
    per_inst_state = 4 * cfg.G * cfg.B + 8 * cfg.W + 4 * cfg.W + 64 * cfg.G
    n_sets = max(2, int(np.ceil(1.6 * L2_BYTES / (N * per_inst_state))))
    n_sets = max(n_sets, int(np.ceil(launches * spl / cfg.steps)))
    prime = 0                                                 # the timed region starts at the sets' starting snapshots
    per_set = -(-(launches + prime) // n_sets)                # launches a set sees in one repeat
    span = per_set * spl
    room = max(0, cfg.steps - span)
    starts = [int(round(j * room / max(1, n_sets - 1))) // spl * spl for j in range(n_sets)]
    sets = RotatingSets(wname, N, n_sets, device, seed_offset=seed_offset, threads=threads,
                        probs_ring=probs_ring, spl=spl, start_steps=starts)
    starts = list(sets.start_steps)
    launches_before = sum(st // spl for st in starts) + warmup + prime      # before the first timed call
    for _ in range(warmup):
        sets.step()
    torch.cuda.synchronize()
    if sampler is not None:
        sampler.start()
        time.sleep(0.3)                      # let the sampler come up before the timed regions
    t0 = time.time()
    reps = []
    for _ in range(repeats):
        sets.reset()
        for _ in range(prime):
            sets.step()
        reps.append(time_region(torch, sets.step, launches, dist))
    t1 = time.time()
    clocks = sampler.stop(t0, t1) if sampler is not None else None
    cnt = sets.counters_mean()
    bad = sets.bad_status()
    tpi = sets.router.params.threads
    sets.close()
    del sets
    torch.cuda.empty_cache()
    ms = float(np.median(reps))
    # edits per instance-step: admissions + terminations (= admissions in steady state) + arrivals
    edits = float(2.0 * cnt[1] + ARRIVALS_PER_STEP[wname])
    # share of the classifier rows a step needs: every row when terminations are drawn from them
    rho = 0.0 if cfg.H == 0 else (1.0 if cfg.term_mode == 2 else 1.0 / cfg.delta_T)
    abytes = algorithmic_bytes(cfg, edits, rho) * N * spl
    us_per_launch = 1e3 * ms / launches
    return dict(ms=ms, ms_per_launch=ms / launches, us_per_launch=us_per_launch, n_sets=n_sets, N=N, spl=spl,
                launches_before_timed=launches_before,
                trajectory=f"sets start at decode steps {starts} of {cfg.steps} and advance {span} steps per repeat",
                repeats_ms=[float(x) for x in reps], abytes_per_launch=abytes,
                achieved=abytes / (us_per_launch * 1e-6) / 1e9, bad=bad, clocks=clocks, threads=tpi,
                launches=launches, value=N * spl * launches / (ms * 1e-3))


def kernel_name(wname):
    return {"c3": "br_small_kernel<2,4>", "c4": "br_step_kernel<true,8,2,1>", "h80": "br_step_kernel<true,80,1,0>",
            "c2": "br_step_kernel<true,4,1,0>"}[wname]


def roofline_of(m, wname, peak, peak_kind, clocks=None):
    """HBM roofline entry of one measurement.  `achieved` is the algorithmic bytes of a launch over
    its measured duration (a normalised throughput: the kernel may move fewer bytes than that --
    BR-0 advances loads without streaming the per-request state -- or more); `dram` is the DRAM
    traffic ncu counted for the same launch shape over the same duration, i.e. the share of the
    HBM bandwidth the kernel really uses; `issue` is what binds the step kernels."""
    spl = m["spl"]
    traffic = recorded_traffic(wname, spl)
    r = {"bound": "hbm", "achieved": m["achieved"], "peak": peak, "unit": "GB/s",
         "frac": m["achieved"] / peak, "frac_of_nominal_8TBs": m["achieved"] / NOMINAL_HBM_GBS,
         "peak_kind": peak_kind, "traffic": traffic,
         "achieved_kind": "algorithmic bytes per launch / measured launch time",
         "algorithmic_bytes_per_launch": m["abytes_per_launch"],
         "us_per_launch": m["us_per_launch"], "kernel": kernel_name(wname)}
    if traffic:
        dram = traffic / (m["us_per_launch"] * 1e-6) / 1e9
        r["dram"] = {"achieved": dram, "unit": "GB/s", "frac": dram / peak,
                     "traffic_over_algorithmic": traffic / m["abytes_per_launch"]}
    winst = recorded_instructions(wname, spl)
    if winst:
        # what binds the step: instruction issue.  Peak = 148 SMs x 4 schedulers x 1 warp
        # instruction per clock at the SM clock sampled during the run.
        clk = ((clocks or {}).get("sm_mhz") or 1965.0) * 1e6
        peak_issue = 148 * 4 * clk
        ach = winst / (m["us_per_launch"] * 1e-6)
        r["issue"] = {"bound": "alu", "achieved": ach / 1e9, "peak": peak_issue / 1e9,
                      "unit": "G warp-instructions/s", "frac": ach / peak_issue,
                      "warp_instructions_per_launch": winst}
    return r


def brief(m, roof):
    return {"us_per_launch": round(m["us_per_launch"], 2), "us_per_decode_step": round(m["us_per_launch"] / m["spl"], 2),
            "inst_steps_per_s": round(m["value"]), "frac": round(roof["frac"], 4),
            "dram_frac": round(roof["dram"]["frac"], 4) if "dram" in roof else None,
            "traffic_over_algorithmic": round(roof["dram"]["traffic_over_algorithmic"], 3) if "dram" in roof else None}


def run_ours(args):
    import torch
    world, rank, local, dist = dist_setup(args)
    device = f"cuda:{local}"
    torch.cuda.set_device(local)
    peak, peak_kind = measured_peaks()

    # ---------------- headline: batched, several decode steps per launch ----------------
    wname = args.workload
    cfg = wlm.get_config(wname)
    spl = steps_per_launch_for(cfg, args.steps_per_launch, args.steps)
    first, _ = shard_of(rank, world, cfg.N, 64)
    m = measure_batched(torch, wname, device, args.steps, args.warmup, spl, repeats=args.repeats,
                        threads=args.threads, seed_offset=first, dist=dist, sampler=ClockSampler(local),
                        n_inst=BATCH_INSTANCES.get(wname))
    N = m["N"]
    value = world * m["value"]
    clocks = m["clocks"]
    roofline = roofline_of(m, wname, peak, peak_kind, clocks)
    line = {
        "metric": METRICS[wname], "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": m["ms_per_launch"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        # arithmetic of the path: Eq. 1 scores, loads and keys in 32-bit integers (ranges proven at
        # br_create), 64-bit outputs; the BR-H workload scores Eq. 2 in fp64
        "dtype": "int32" if wname == "c3" else "f64", "data": "synthetic",
        "config": {"workload": WORKLOADS[wname],
                   "step": f"one br_step call = one launch advancing {N} instances by {spl} decode steps "
                           f"({N * spl} instance-steps)",
                   "instances_per_launch": N, "steps_per_launch": spl, "rotating_sets": m["n_sets"],
                   "repeats": args.repeats,
                   "timing": f"median of {args.repeats} repeats of the {args.steps}-call region (CUDA events; "
                             f"before each repeat the sets return to their starting snapshots)",
                   "trajectory": m["trajectory"], "launches_before_timed": m["launches_before_timed"],
                   "l2": f"{m['n_sets']} instance sets stepped in rotation: data touched between two visits of a "
                         f"set exceeds the 126 MB L2; no instance runs past the configuration's {cfg.steps} steps",
                   "threads_per_instance": m["threads"]},
        "ms_per_step_min": min(m["repeats_ms"]) / args.steps, "ms_per_step_max": max(m["repeats_ms"]) / args.steps,
        "roofline": roofline, "clocks": clocks, "gpu_launches": m["launches"],
        "bad_status_instances": m["bad"],
    }
    summary = {f"{wname}_{spl}_steps_per_launch": brief(m, roofline)}

    if rank == 0 and world == 1 and not args.quick and wname == "c3":
        # the same workload with one decode step per launch (the form the latency path replays)
        m1 = measure_batched(torch, wname, device, cfg.steps, 40, 1, repeats=5, threads=args.threads)   # one pass over the trajectory
        r1 = roofline_of(m1, wname, peak, peak_kind, clocks)
        line["single_step_launches"] = {"value": m1["value"], "unit": UNIT, "ms_per_step": m1["ms_per_launch"],
                                        "roofline": r1, "gpu_launches": m1["launches"], "repeats_ms": m1["repeats_ms"]}
        summary["c3_1_step_per_launch"] = brief(m1, r1)
        # two batches in one call (8,192 instances, one decode step): the second wave of thread blocks
        # fills the SMs that the first wave's short instances leave early
        m2 = measure_batched(torch, wname, device, cfg.steps, 20, 1, repeats=5, threads=args.threads, n_inst=2 * N)
        line["single_step_launches_8192_instances"] = {
            "value": m2["value"], "unit": UNIT, "ms_per_step": m2["ms_per_launch"], "instances_per_launch": 2 * N,
            "us_per_4096_instance_steps": m2["us_per_launch"] / 2, "repeats_ms": m2["repeats_ms"],
            "frac": m2["achieved"] / peak}
        summary["c3_1_step_per_launch_8192_instances"] = {
            "us_per_launch": round(m2["us_per_launch"], 2), "us_per_4096_instance_steps": round(m2["us_per_launch"] / 2, 2),
            "inst_steps_per_s": round(m2["value"]), "frac": round(m2["achieved"] / peak, 4)}
        # ---------------- end to end through the host-buffer entry point ----------------
        line["e2e"] = e2e_host(torch, device, args)
        summary["e2e_c3_host_buffers"] = {"inst_steps_per_s": round(line["e2e"]["value"]),
                                          "ms_per_step": round(line["e2e"]["ms_per_step"], 3)}
        # ---------------- extras: c4 batched BR-H, stand-alone entry points, latency path ----------------
        try:
            line["extra"] = extras(torch, device, args, peak, peak_kind, summary)
        except Exception as ex:  # keep the headline line even if an extra fails
            line["extra"] = {"error": repr(ex)}
        # ---------------- CPU baseline: the checker on host cores ----------------
        try:
            cb = cpu_baselines(args)
            line["cpu_baseline"] = cb["c3"]
            line["cpu_baseline_other"] = {k: v for k, v in cb.items() if k != "c3"}
            summary["cpu_oracle_inst_steps_per_s"] = {k: (round(v["value"]) if "value" in v else None, v.get("cores"))
                                                      for k, v in cb.items()}
        except Exception as ex:
            line["cpu_baseline"] = {"error": repr(ex)}
    elif rank == 0:
        line["e2e"] = None
    line["summary"] = summary                 # last key: the tail of the line holds every headline figure
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def e2e_host(torch, device, args):
    from paper_2605_06113_b200.binding import Router
    cfg = wlm.get_config("c3")
    wl = wlm.make_workload(cfg, n_instances=cfg.N, first_instance=1 << 20)
    r = Router(wl, device=device, threads=args.threads)
    st = {k: torch.from_numpy(np.ascontiguousarray(v).view(
        {np.dtype(np.uint64): np.int64, np.dtype(np.uint32): np.int32}.get(v.dtype, v.dtype))).pin_memory()
          for k, v in wl.state.items()}
    out = {k: v.pin_memory() for k, v in r.outputs(cfg.N, device="cpu").items()}
    steps = 30
    up = down = 0
    for _ in range(3):
        r.step_host(st, out)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        up, down = r.step_host(st, out)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    r.close()
    return {"value": cfg.N * steps / dt, "unit": UNIT, "h2d_bytes_per_step": up,
            "d2h_bytes_per_step": down, "steps": steps, "ms_per_step": 1e3 * dt / steps,
            "step": "one decode step of 4096 instances through br_step_host: pinned host snapshot up, "
                    "kernel, snapshot and results down"}


def extras(torch, device, args, peak, peak_kind, summary):
    ex = {}
    # c4: BR-H batched (H = 8), 4 decode steps per launch and one step per launch
    for spl in (4, 1):
        m = measure_batched(torch, "c4", device, 200 // spl, 20, spl, repeats=5)
        roof = roofline_of(m, "c4", peak, peak_kind)
        key = "c4_batched" if spl == 4 else "c4_single_step_launches"
        ex[key] = {"value": m["value"], "unit": UNIT, "ms_per_step": m["ms_per_launch"], "steps_per_launch": spl,
                   "repeats_ms": m["repeats_ms"], "roofline": roof}
        summary[f"c4_{spl}_step{'s' if spl > 1 else ''}_per_launch"] = brief(m, roof)
    # the deployed lookahead as a batch: 1,024 instances of the h80 workload (H = 80, G = 8, R_max = 4), 8 steps per launch
    try:
        mh = measure_batched(torch, "h80", device, 24, 4, 8, repeats=5, n_inst=1024)
        rh = roofline_of(mh, "h80", peak, peak_kind)
        ex["h80_batched"] = {"value": mh["value"], "unit": UNIT, "ms_per_step": mh["ms_per_launch"], "steps_per_launch": 8,
                             "instances_per_launch": 1024, "repeats_ms": mh["repeats_ms"], "roofline": rh}
        summary["h80_batched_1024_instances"] = brief(mh, rh)
    except Exception as e:
        ex["h80_batched"] = {"error": repr(e)}
    # the c2 shape as a batch (2,048 instances, H = 4, terminations drawn from the classifier rows, so every
    # row is read every step): the most HBM-like of the step workloads
    try:
        m2 = measure_batched(torch, "c2", device, 60, 6, 4, repeats=5, n_inst=2048)
        r2 = roofline_of(m2, "c2", peak, peak_kind)
        ex["c2_batched"] = {"value": m2["value"], "unit": UNIT, "ms_per_step": m2["ms_per_launch"], "steps_per_launch": 4,
                            "instances_per_launch": 2048, "repeats_ms": m2["repeats_ms"], "roofline": r2}
        summary["c2_batched_2048_instances"] = brief(m2, r2)
    except Exception as e:
        ex["c2_batched"] = {"error": repr(e)}
    # the stand-alone entry points: F-score matrix, pool-bypass dispatch, exact subset solver
    try:
        ex["entry_points"] = entry_points(torch, device, peak)
        summary["br_fscore_eq1_frac"] = round(ex["entry_points"]["br_fscore_eq1"]["roofline"]["frac"], 3)
    except Exception as e:
        ex["entry_points"] = {"error": repr(e)}
    # latency path: one instance, one graph-replayed step per decode step
    lat = [latency_path(torch, "c1", device, 2000), latency_path(torch, "c2", device, 2000),
           latency_path(torch, "c4", device, 1000), latency_path(torch, "h80", device, 1500)]
    # the paper's own figure for its Python dispatcher at the same H, G and R_max (Section 5.3
    # "Dispatch overhead", another machine and language): context, not a target
    lat[3]["paper_dispatcher_tick_p50_us"] = 1200.0
    ex["latency"] = lat
    summary["latency_device_p50_us"] = {f"{l['workload']}(G={l['G']},W={l['W']},H={l['H']})": round(l["device_p50_us"], 1)
                                        for l in lat}
    summary["latency_host_p50_us"] = {l["workload"]: round(l["host_p50_us"], 1) for l in lat}
    return ex


def latency_path(torch, cfg_name, device, steps, overrides=None):
    """Single instance, graph-replayed step: host-observed and device latency per step."""
    from paper_2605_06113_b200.binding import Router
    cfg = wlm.get_config(cfg_name, **(overrides or {}))
    wl = wlm.make_workload(cfg, n_instances=1)
    r = Router(wl, device=device)
    st = r.device_state()
    out = r.outputs(1)
    probs = None
    seeds_t = tab_t = None
    need_probs = cfg.H > 0 and cfg.pred_mode == 0          # the perfect-lookahead predictor reads no classifier rows
    if need_probs:
        seeds_t = torch.from_numpy(wl.seeds.astype(np.int64)).to(device)
        tab_t = torch.from_numpy(wl.beta_tab).to(device)
        probs = wlm.term_probs_torch(wl, 0, device, seeds_t=seeds_t, tab_t=tab_t).contiguous()
    r.graph_capture(st, out, probs)
    host_us, dev_us = [], []
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    for k in range(steps):
        if need_probs:
            wlm.term_probs_torch(wl, k, device, seeds_t=seeds_t, tab_t=tab_t, out=probs)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        e0.record()
        r.graph_step()
        e1.record()
        torch.cuda.synchronize()
        host_us.append(1e6 * (time.perf_counter() - t0))
        dev_us.append(1e3 * e0.elapsed_time(e1))
    # per-phase split of the step (the kernel's own cycle counters; the paper splits its dispatcher
    # the same way: preparation / Stage 1 / Stage 2), averaged over the next 200 steps
    out["phase_cycles"] = torch.zeros((1, 1, 8), dtype=torch.int32, device=device)
    acc = np.zeros(8)
    n_ph = 200
    for k in range(steps, steps + n_ph):
        if need_probs:
            wlm.term_probs_torch(wl, k, device, seeds_t=seeds_t, tab_t=tab_t, out=probs)
        r.step(st, out, probs)
        torch.cuda.synchronize()
        acc += out["phase_cycles"][0, 0].cpu().numpy()
    mhz = float(torch.cuda.get_device_properties(device).clock_rate) / 1e3 if hasattr(
        torch.cuda.get_device_properties(device), "clock_rate") else 1965.0
    names = ["arrive", "predict", "stage1", "stage2", "record_compact", "advance", "prologue", "kernel_total"]
    phases = {n: float(acc[i] / n_ph / mhz) for i, n in enumerate(names)}
    r.close()
    h = np.array(host_us[20:]); d = np.array(dev_us[20:])
    return {"workload": cfg_name, "G": cfg.G, "W": cfg.W, "H": cfg.H, "steps": steps,
            "host_p50_us": float(np.percentile(h, 50)), "host_p95_us": float(np.percentile(h, 95)),
            "host_p99_us": float(np.percentile(h, 99)), "device_p50_us": float(np.percentile(d, 50)),
            "device_p99_us": float(np.percentile(d, 99)),
            "phase_us_at_max_clock": phases,
            "phase_note": "phase split taken with the kernel's cycle counters on br_step_kernel (the "
                          "kernel that offers them); the latencies above are those of the kernel the "
                          "library picks for the shape"}


def _time_call(torch, fn, reps=20, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def entry_points(torch, device, peak):
    """Timings of br_fscore (HBM-bound: the matrix is written once), br_bypass_dispatch and
    br_best_subset on synthetic inputs of the c3 / c4 shapes."""
    from paper_2605_06113_b200.binding import Router
    res = {}
    gen = torch.Generator(device=device); gen.manual_seed(7)
    # F-score matrix: c4 shape, 1024 instances x 1024 requests x 64 workers in fp64 (512 MB out)
    cfg = wlm.get_config("c4")
    wl = wlm.make_workload(cfg, n_instances=1)
    r = Router(wl, device=device)
    N, n_req, G, H = 1024, 1024, cfg.G, cfg.H
    s = torch.randint(1, 60000, (N, n_req), dtype=torch.int32, device=device, generator=gen)
    Lh = torch.randint(100000, 400000, (N, G, H + 1), dtype=torch.int64, device=device, generator=gen)
    F = torch.empty((N, n_req, G), dtype=torch.float64, device=device)
    ms = _time_call(torch, lambda: r.fscore(s, Lh, F))
    byt = F.numel() * 8 + s.numel() * 4 + Lh.numel() * 8
    res["br_fscore"] = {"workload": "c4 shape (Eq. 2, H=8): 1024 instances x 1024 requests x 64 workers, fp64 matrix",
                        "ms": ms, "scores_per_s": F.numel() / (ms * 1e-3),
                        "roofline": {"bound": "hbm", "achieved": byt / (ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                                     "frac": byt / (ms * 1e-3) / 1e9 / peak, "traffic": None,
                                     "algorithmic_bytes_per_launch": byt, "kernel": "br_fscore_kernel"}}
    del F
    r.close()
    # pool-bypass dispatch and subset solver: c3 shape (Eq. 1)
    cfg = wlm.get_config("c3")
    wl = wlm.make_workload(cfg, n_instances=1)
    r = Router(wl, device=device)
    N, n_req, G = 4096, 256, cfg.G
    s = torch.randint(1, 40000, (N, n_req), dtype=torch.int32, device=device, generator=gen)
    L0 = torch.randint(0, 300000, (N, G), dtype=torch.int64, device=device, generator=gen)
    F = torch.empty((N, 1024, G), dtype=torch.float64, device=device)
    s4 = torch.randint(1, 40000, (N, 1024), dtype=torch.int32, device=device, generator=gen)
    ms = _time_call(torch, lambda: r.fscore(s4, L0.view(N, G, 1), F))
    byt = F.numel() * 8 + s4.numel() * 4 + L0.numel() * 8
    res["br_fscore_eq1"] = {"workload": "c3 shape (Eq. 1): 4096 instances x 1024 requests x 32 workers, fp64 matrix",
                            "ms": ms, "scores_per_s": F.numel() / (ms * 1e-3),
                            "roofline": {"bound": "hbm", "achieved": byt / (ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                                         "frac": byt / (ms * 1e-3) / 1e9 / peak, "traffic": None,
                                         "algorithmic_bytes_per_launch": byt, "kernel": "br_fscore_kernel<0>"}}
    del F, s4
    cap = torch.full((N, G), 1 << 30, dtype=torch.int32, device=device)
    L = L0.clone(); infl = torch.zeros((N, G), dtype=torch.int32, device=device)
    out = torch.empty((N, n_req), dtype=torch.int32, device=device)
    ms = _time_call(torch, lambda: r.bypass_dispatch(s, L, infl, cap, out))
    res["br_bypass_dispatch"] = {"workload": "c3 shape: 4096 instances, 256 requests each dispatched in order over 32 workers",
                                 "ms": ms, "requests_per_s": N * n_req / (ms * 1e-3)}
    R, P = 16, 4096
    win = torch.randint(1, 40000, (P, R), dtype=torch.int32, device=device, generator=gen)
    m = torch.randint(0, 200000, (P, 1), dtype=torch.int64, device=device, generator=gen)
    lim = torch.full((P,), R, dtype=torch.int32, device=device)
    mask = torch.empty((P,), dtype=torch.int32, device=device)
    ms = _time_call(torch, lambda: r.best_subset(win, m, lim, mask))
    res["br_best_subset"] = {"workload": "4096 problems, window of 16 requests (65,535 subsets each), Eq. 1",
                             "ms": ms, "problems_per_s": P / (ms * 1e-3), "subsets_per_s": P * ((1 << R) - 1) / (ms * 1e-3)}
    r.close()
    # empirical-survival estimator: 4M requests against a history of 1M output lengths (H = 8)
    cfg = wlm.get_config("c4")
    wl = wlm.make_workload(cfg, n_instances=1)
    r = Router(wl, device=device)
    hist = torch.sort(torch.randint(1, 4000, (1 << 20,), dtype=torch.int32, device=device, generator=gen)).values
    prefix = torch.cat([torch.zeros(1, dtype=torch.int64, device=device), torch.cumsum(hist.to(torch.int64), 0)])
    age = torch.randint(0, 4000, (1 << 22,), dtype=torch.int32, device=device, generator=gen)
    c = torch.empty(age.numel(), dtype=torch.float32, device=device)
    ms = _time_call(torch, lambda: r.survival_chat(hist, prefix, age, c))
    res["br_survival_chat"] = {"workload": "4,194,304 requests, history of 1,048,576 output lengths, H = 8",
                               "ms": ms, "requests_per_s": age.numel() / (ms * 1e-3)}
    r.close()
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=124,
                    help="br_step calls in the timed region (124 calls of 16 decode steps walk four instance sets "
                         "through the whole 500-step configuration)")
    ap.add_argument("--warmup", type=int, default=10, help="untimed br_step calls before the first repeat")
    ap.add_argument("--steps-per-launch", type=int, default=0,
                    help="decode steps advanced by one br_step call (batch.n_steps); 0 = 16, or with fewer than 32 "
                         "calls in the timed region the number with which they cover the configuration exactly once")
    ap.add_argument("--repeats", type=int, default=7, help="repeats of the timed region; the median is reported")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--threads", type=int, default=0, help="threads per instance (0 = library default)")
    ap.add_argument("--quick", action="store_true", help="headline measurement only")
    ap.add_argument("--workload", default="c3", choices=["c3", "c4", "h80"],
                    help="batched configuration timed as the headline (c4 is used for profiling the BR-H kernel)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    args.repeats = max(args.repeats, 1)
    if args.impl == "reference":
        args.steps = min(args.steps, 25)
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
