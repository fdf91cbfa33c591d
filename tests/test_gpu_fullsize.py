"""Full-size batches in the launch configuration the benchmark times (4,096 BR-0 instances,
1,024 BR-H instances): sampled instances are compared with the CPU checker step by step, and
properties that hold at any size are checked on every instance."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_06113_b200 import workload as wlm
from paper_2605_06113_b200.binding import Router, state_to_numpy
from helpers import compare_state

pytestmark = pytest.mark.gpu


def _run(name, steps, n_sample, seed):
    cfg = wlm.get_config(name)
    N = cfg.N
    wl = wlm.make_workload(cfg)
    r = Router(wl, device="cuda:0")
    st = r.device_state()
    out = r.outputs(N)
    rng = np.random.default_rng(seed)
    idx = sorted(set([0, 1, N - 1] + [int(x) for x in rng.integers(0, N, n_sample - 3)]))
    orcs = {i: oracle.instance_from_workload(wl, i) for i in idx}
    seeds_t = torch.from_numpy(wl.seeds.astype(np.int64)).cuda()
    tab_t = torch.from_numpy(wl.beta_tab).cuda()
    call = None
    probs_t = None
    nact_prev = st["nact"].clone()
    for k in range(steps):
        probs_np = None
        if cfg.H > 0:
            probs_new = wlm.term_probs_torch(wl, k, "cuda:0", seeds_t=seeds_t, tab_t=tab_t)
            if probs_t is None:
                probs_t = probs_new.contiguous()
            else:
                probs_t.copy_(probs_new)
            probs_np = wlm.term_probs_np(wl, k, instances=idx)
        if call is None:
            call = r.prepare(st, out, probs_t)
        call()
        torch.cuda.synchronize()
        a = out["assign"][0]; load = out["load"][0]; tr = out["trace"][0]; cnt = out["counters"][0]
        # ---- properties on every instance ----
        assert int((out["status"][0] & ~1).ne(0).sum()) == 0
        assert torch.equal(tr[:, 0], load.max(1).values) and torch.equal(tr[:, 1], load.min(1).values)
        assert torch.equal(tr[:, 2], load.sum(1))
        adm = (a >= 0).sum(1)
        assert torch.equal(adm.to(torch.int32), cnt[:, 1])                  # one slot per admission
        free = cfg.G * cfg.B - nact_prev.sum(1)
        assert bool((adm <= free).all())                                    # capacity
        srt = torch.sort(torch.where(a >= 0, a, torch.full_like(a, -1)), dim=1).values
        dup = (srt[:, 1:] == srt[:, :-1]) & (srt[:, 1:] >= 0)
        assert not bool(dup.any())                                          # disjoint assignments
        assert int(a.max()) < cfg.G * cfg.B
        nact_prev = st["nact"].clone()
        # ---- sampled instances against the checker ----
        ah = a[idx].cpu().numpy(); lh = load[idx].cpu().numpy(); th = tr[idx].cpu().numpy()
        for j, i in enumerate(idx):
            ao, lo, to, _ = orcs[i].step(None if probs_np is None else probs_np[j])
            assert np.array_equal(ah[j], ao), (name, i, k)
            assert np.array_equal(lh[j], lo), (name, i, k)
            assert np.array_equal(th[j], to), (name, i, k)
    fin = state_to_numpy(st)
    for i in idx:
        compare_state(cfg, fin, orcs[i], i, steps)
    r.close()


def test_c3_full_batch_sampled_instances():
    _run("c3", 150, 16, 5)


def test_c4_full_batch_sampled_instances():
    _run("c4", 40, 10, 6)


def test_c3_full_batch_sixteen_steps_per_launch():
    """The launch the benchmark times: 4,096 instances, sixteen decode steps per launch.  Sampled
    instances are compared with the checker at every step of every launch."""
    cfg = wlm.get_config("c3")
    N, S = cfg.N, 16
    wl = wlm.make_workload(cfg)
    r = Router(wl, device="cuda:0")
    st = r.device_state()
    out = r.outputs(N, n_steps=S)
    rng = np.random.default_rng(11)
    idx = sorted(set([0, N - 1] + [int(x) for x in rng.integers(0, N, 10)]))
    orcs = {i: oracle.instance_from_workload(wl, i) for i in idx}
    call = r.prepare(st, out, None, N=N, first=0, n_steps=S)
    for launch in range(20):
        call()
        torch.cuda.synchronize()
        assert int((out["status"] & ~1).ne(0).sum()) == 0
        tr = out["trace"]; load = out["load"]
        assert torch.equal(tr[:, :, 0], load.max(2).values) and torch.equal(tr[:, :, 2], load.sum(2))
        assert torch.equal(tr[:, :, 1], load.min(2).values)
        ah = out["assign"][:, idx].cpu().numpy(); lh = load[:, idx].cpu().numpy(); th = tr[:, idx].cpu().numpy()
        for j in range(S):
            for c, i in enumerate(idx):
                ao, lo, to, _ = orcs[i].step()
                assert np.array_equal(ah[j, c], ao), (i, launch, j)
                assert np.array_equal(lh[j, c], lo), (i, launch, j)
                assert np.array_equal(th[j, c], to), (i, launch, j)
    fin = state_to_numpy(st)
    for i in idx:
        compare_state(cfg, fin, orcs[i], i, 20 * S)
    r.close()


def test_c4_full_batch_four_steps_per_launch():
    """The BR-H launch the benchmark times: 1,024 instances, four decode steps per launch, the
    classifier output of the four steps passed as one block."""
    cfg = wlm.get_config("c4")
    N, S = cfg.N, 4
    wl = wlm.make_workload(cfg)
    r = Router(wl, device="cuda:0")
    st = r.device_state()
    out = r.outputs(N, n_steps=S)
    rng = np.random.default_rng(13)
    idx = sorted(set([0, N - 1] + [int(x) for x in rng.integers(0, N, 4)]))
    orcs = {i: oracle.instance_from_workload(wl, i) for i in idx}
    seeds_t = torch.from_numpy(wl.seeds.astype(np.int64)).cuda()
    tab_t = torch.from_numpy(wl.beta_tab).cuda()
    probs_t = torch.empty((S, N, cfg.G, cfg.B, cfg.H), dtype=torch.float32, device="cuda:0")
    call = r.prepare(st, out, probs_t, N=N, first=0, n_steps=S)
    for launch in range(6):
        for j in range(S):
            wlm.term_probs_torch(wl, launch * S + j, "cuda:0", seeds_t=seeds_t, tab_t=tab_t, out=probs_t[j])
        call()
        torch.cuda.synchronize()
        assert int((out["status"] & ~1).ne(0).sum()) == 0
        tr = out["trace"]; load = out["load"]
        assert torch.equal(tr[:, :, 0], load.max(2).values) and torch.equal(tr[:, :, 2], load.sum(2))
        assert torch.equal(tr[:, :, 1], load.min(2).values)
        ah = out["assign"][:, idx].cpu().numpy(); lh = load[:, idx].cpu().numpy(); th = tr[:, idx].cpu().numpy()
        for j in range(S):
            probs_np = wlm.term_probs_np(wl, launch * S + j, instances=idx)
            for c, i in enumerate(idx):
                ao, lo, to, _ = orcs[i].step(probs_np[c])
                assert np.array_equal(ah[j, c], ao), (i, launch, j)
                assert np.array_equal(lh[j, c], lo), (i, launch, j)
                assert np.array_equal(th[j, c], to), (i, launch, j)
    fin = state_to_numpy(st)
    for i in idx:
        compare_state(cfg, fin, orcs[i], i, 6 * S)
    r.close()
