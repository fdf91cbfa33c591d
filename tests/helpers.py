"""Side-by-side runs of the CUDA library and the CPU checker on the same seeded inputs."""
import numpy as np

import oracle
from paper_2605_06113_b200 import workload as wlm
from paper_2605_06113_b200.binding import Router, state_to_numpy

EMPTY = oracle.EMPTY


def compare_state(cfg, st_np, o, i, k):
    """Boundary-format device state of instance i against the checker's state entering step k."""
    s = o.get_state()
    assert int(st_np["step"][i]) == s["step"] == k
    assert int(st_np["next_id"][i]) == s["next_id"]
    assert np.array_equal(st_np["act_base"][i], s["act_base"]), f"act_base inst {i} step {k}"
    occ = s["act_base"] != EMPTY
    assert np.array_equal(st_np["act_id"][i][occ], s["act_id"][occ])
    assert np.array_equal(st_np["nact"][i], occ.sum(1))
    cur = np.where(occ, s["act_base"].astype(np.int64) + k, 0)
    assert np.array_equal(st_np["load"][i], cur.sum(1))
    bits = np.zeros((cfg.G, cfg.B), dtype=bool)
    for b in range(cfg.B):
        bits[:, b] = (st_np["occ"][i][:, b // 64] >> np.uint64(b % 64)) & np.uint64(1) != 0
    assert np.array_equal(bits, occ)
    n = s["wq_n"]
    assert int(st_np["wq_n"][i]) == n
    assert np.array_equal(st_np["wq_s"][i][:n], s["wq_s"][:n])
    assert np.array_equal(st_np["wq_id"][i][:n], s["wq_id"][:n])
    if cfg.term_mode == 3:
        ae, qo = o.get_lifetimes() if hasattr(o, "get_lifetimes") else (s["act_end"], s["wq_o"])
        assert np.array_equal(st_np["act_end"][i][occ], ae[occ]), f"act_end inst {i} step {k}"
        assert np.array_equal(st_np["wq_o"][i][:n], qo[:n])
    if cfg.H > 0 and cfg.pred_mode == 0:
        chat, tau = oracle.explicit_pred_state(st_np["act_chat0"][i], st_np["act_kref"][i], k)
        assert np.array_equal(chat[occ], s["chat"][occ]), f"c_hat inst {i} step {k}"
        assert np.array_equal(tau[occ], s["tau"][occ])


def run_parity(cfg, n_inst, steps, threads=0, fscore=False, launch_steps=1, first_instance=0,
               check_every=1, device="cuda:0", graph=False):
    """Runs `steps` decode steps on both sides; compares assignments, loads, trace and counters
    at every step and the whole snapshot at the end.  Returns the per-step traces."""
    import torch
    wl = wlm.make_workload(cfg, n_instances=n_inst, first_instance=first_instance)
    r = Router(wl, device=device, threads=threads)
    st = r.device_state()
    out = r.outputs(n_inst, n_steps=launch_steps, fscore=fscore)
    orcs = [oracle.instance_from_workload(wl, i) for i in range(n_inst)]
    H = cfg.H
    traces = []
    probs_t = None
    if H > 0:
        probs_t = torch.empty((launch_steps, n_inst, cfg.G, cfg.B, H), dtype=torch.float32, device=device)
    captured = False
    k = 0
    while k < steps:
        probs_np = None
        if H > 0:
            probs_np = np.stack([wlm.term_probs_np(wl, k + j) for j in range(launch_steps)])
            probs_t.copy_(torch.from_numpy(probs_np))
        if graph:
            if not captured:
                r.graph_capture(st, out, probs_t, n_steps=launch_steps)
                captured = True
            r.graph_step()
        else:
            r.step(st, out, probs_t, n_steps=launch_steps)
        torch.cuda.synchronize()
        g = {kk: v.cpu().numpy() for kk, v in out.items()}
        for j in range(launch_steps):
            for i, o in enumerate(orcs):
                c0 = o.get_state()["counters"].copy()
                a, l, t, fs = o.step(None if H == 0 else probs_np[j, i], want_fscore=fscore)
                c1 = o.get_state()["counters"]
                where = f"inst {i} step {k + j}"
                assert np.array_equal(g["assign"][j, i], a), where
                assert np.array_equal(g["load"][j, i], l), where
                assert np.array_equal(g["trace"][j, i], t), where
                assert np.array_equal(g["counters"][j, i], (c1 - c0)[:4]), where
                assert (g["status"][j, i] & ~1) == 0, where
                assert bool(g["status"][j, i] & 1) == bool(c1[0] - c0[0]), where
                if fscore:
                    ref = fs
                    got = g["fscore"][j, i]
                    err = np.abs(got - ref) / np.maximum(1.0, np.abs(ref))
                    assert err.max() <= 1e-6, where          # stated tolerance; equality expected
                    assert np.array_equal(got, ref), where
                if i == 0:
                    traces.append(t.copy())
        k += launch_steps
        if (k // launch_steps) % check_every == 0 or k >= steps:
            st_np = state_to_numpy(st)
            for i, o in enumerate(orcs):
                compare_state(cfg, st_np, o, i, k)
    r.close()
    return np.array(traces)


# ---- whole batches: the checker fanned out over host processes -------------------------------
def oracle_chunk(job):
    """Runs the checker on instances [first, first + n) of a configuration for `steps` decode
    steps.  Returns the per-step outputs (assign as int16, load, trace, counters) and the final
    snapshot of every instance.  Top-level so that a `spawn` pool can import it."""
    name, overrides, first, n, steps = job
    cfg = wlm.get_config(name, **overrides)
    wl = wlm.make_workload(cfg, n_instances=n, first_instance=first)
    orcs = [oracle.instance_from_workload(wl, i) for i in range(n)]
    assign = np.empty((steps, n, cfg.W), dtype=np.int16)
    load = np.empty((steps, n, cfg.G), dtype=np.int64)
    trace = np.empty((steps, n, 3), dtype=np.int64)
    cnt = np.empty((steps, n, 4), dtype=np.int64)
    c_prev = [o.get_state()["counters"].copy() for o in orcs]
    for k in range(steps):
        probs = wlm.term_probs_np(wl, k) if cfg.H > 0 else None
        for i, o in enumerate(orcs):
            a, l, t, _ = o.step(None if probs is None else probs[i])
            assign[k, i] = a; load[k, i] = l; trace[k, i] = t
            c1 = o.get_state()["counters"].copy()
            cnt[k, i] = (c1 - c_prev[i])[:4]
            c_prev[i] = c1
    fin = [o.get_state() for o in orcs]
    return first, assign, load, trace, cnt, fin


def oracle_batch(name, n_total, steps, overrides=None, chunk=None):
    """The checker on instances 0..n_total-1, one process per host core (`spawn`: the parent has
    CUDA initialised).  Returns the concatenated per-step outputs, the final snapshots and the
    number of processes used."""
    import multiprocessing as mp
    import os
    cores = len(os.sched_getaffinity(0))
    chunk = chunk or max(1, -(-n_total // (cores * 2)))
    jobs = [(name, overrides or {}, f, min(chunk, n_total - f), steps) for f in range(0, n_total, chunk)]
    procs = min(cores, len(jobs))
    if procs <= 1:
        res = [oracle_chunk(j) for j in jobs]
    else:
        with mp.get_context("spawn").Pool(procs) as pool:
            res = pool.map(oracle_chunk, jobs)
    res.sort(key=lambda r: r[0])
    assign = np.concatenate([r[1] for r in res], axis=1)
    load = np.concatenate([r[2] for r in res], axis=1)
    trace = np.concatenate([r[3] for r in res], axis=1)
    cnt = np.concatenate([r[4] for r in res], axis=1)
    fin = [s for r in res for s in r[5]]
    return assign, load, trace, cnt, fin, procs


def compare_state_dict(cfg, st_np, s, i, k):
    """compare_state against a snapshot dictionary of the checker (as oracle_chunk returns it)."""
    class _Snap:
        def get_state(self_inner):
            return s
    compare_state(cfg, st_np, _Snap(), i, k)
