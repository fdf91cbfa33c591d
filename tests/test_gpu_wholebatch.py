"""Whole batches against the CPU checker, every instance and every array: the two batched
configurations in the launch shapes the benchmark times, with the checker fanned out over the
host cores.  c3: all 4,096 instances over the first 112 decode steps (the start-up transient and
the saturated regime), one and sixteen steps per launch.  c4: all 1,024 instances over 20 steps,
and the whole batch run to its full 1,000 steps with sampled instances compared at every step, so
that the arrival bursts at k = 250, 500 and 750 are crossed."""
import numpy as np
import pytest
import torch

from paper_2605_06113_b200 import workload as wlm
from paper_2605_06113_b200.binding import Router, state_to_numpy
from helpers import compare_state, compare_state_dict, oracle_batch
import oracle

pytestmark = pytest.mark.gpu


def _gpu_run(cfg, steps, spl, n_inst=None, keep=None):
    """Runs the batch on the GPU; returns per-step outputs as numpy ([steps][N][...]) for the
    instances in `keep` (all if None) and the final snapshot."""
    N = cfg.N if n_inst is None else n_inst
    wl = wlm.make_workload(cfg, n_instances=N)
    r = Router(wl, device="cuda:0")
    st = r.device_state()
    out = r.outputs(N, n_steps=spl)
    sel = None if keep is None else torch.tensor(keep, device="cuda:0")
    probs_t = None
    if cfg.H > 0:
        seeds_t = torch.from_numpy(wl.seeds.astype(np.int64)).cuda()
        tab_t = torch.from_numpy(wl.beta_tab).cuda()
        probs_t = torch.empty((spl, N, cfg.G, cfg.B, cfg.H), dtype=torch.float32, device="cuda:0")
    call = r.prepare(st, out, probs_t, N=N, first=0, n_steps=spl)
    acc = {k: [] for k in ("assign", "load", "trace", "counters", "status")}
    assert steps % spl == 0
    for launch in range(steps // spl):
        if cfg.H > 0:
            for j in range(spl):
                wlm.term_probs_torch(wl, launch * spl + j, "cuda:0", seeds_t=seeds_t, tab_t=tab_t, out=probs_t[j])
        call()
        torch.cuda.synchronize()
        # properties on every instance, whatever is kept
        assert int((out["status"] & ~1).ne(0).sum()) == 0
        tr, load = out["trace"], out["load"]
        assert torch.equal(tr[:, :, 0], load.max(2).values) and torch.equal(tr[:, :, 1], load.min(2).values)
        assert torch.equal(tr[:, :, 2], load.sum(2))
        for k in acc:
            v = out[k] if sel is None else out[k].index_select(1, sel)
            acc[k].append(v.to(torch.int16).cpu().numpy() if k == "assign" else v.cpu().numpy())
    fin = state_to_numpy(st)
    r.close()
    return {k: np.concatenate(v, axis=0) for k, v in acc.items()}, fin


def _compare_all(cfg, got, fin, ref, steps, ids):
    assign, load, trace, cnt, fin_ref, procs = ref
    assert np.array_equal(got["assign"], assign)
    assert np.array_equal(got["load"], load)
    assert np.array_equal(got["trace"], trace)                       # maximum, minimum and sum
    assert np.array_equal(got["counters"].astype(np.int64), cnt)
    assert np.array_equal((got["status"] & 1) != 0, cnt[:, :, 0] > 0)
    for j, i in enumerate(ids):
        compare_state_dict(cfg, fin, fin_ref[j], i, steps)


@pytest.mark.parametrize("spl", [1, 16])
def test_c3_every_instance_every_array(spl):
    cfg = wlm.get_config("c3")
    steps = 112
    ref = oracle_batch("c3", cfg.N, steps)
    print(f"checker processes: {ref[5]}")
    got, fin = _gpu_run(cfg, steps, spl)
    _compare_all(cfg, got, fin, ref, steps, range(cfg.N))


@pytest.mark.parametrize("spl", [1, 4])
def test_c4_every_instance_every_array(spl):
    cfg = wlm.get_config("c4")
    steps = 20
    ref = oracle_batch("c4", cfg.N, steps)
    print(f"checker processes: {ref[5]}")
    got, fin = _gpu_run(cfg, steps, spl)
    _compare_all(cfg, got, fin, ref, steps, range(cfg.N))


def test_c4_full_length_across_the_bursts():
    """The whole batch of 1,024 instances runs its 1,000 steps, four per launch; instances
    0, 341, 682 and 1023 are compared with the checker at every step (the checker's instances are
    generated on their own: an instance's inputs do not depend on its batch)."""
    cfg = wlm.get_config("c4")
    steps, ids = 1000, [0, 341, 682, 1023]
    import multiprocessing as mp
    from helpers import oracle_chunk
    with mp.get_context("spawn").Pool(len(ids)) as pool:
        pending = pool.map_async(oracle_chunk, [("c4", {}, i, 1, steps) for i in ids])
        got, fin = _gpu_run(cfg, steps, 4, keep=ids)
        res = pending.get()
    dropped = 0
    for j, (first, assign, load, trace, cnt, fin_ref) in enumerate(res):
        assert np.array_equal(got["assign"][:, j], assign[:, 0])
        assert np.array_equal(got["load"][:, j], load[:, 0])
        assert np.array_equal(got["trace"][:, j], trace[:, 0])
        assert np.array_equal(got["counters"][:, j].astype(np.int64), cnt[:, 0])
        compare_state_dict(cfg, fin, fin_ref[0], ids[j], steps)
        dropped += int(cnt[[250, 500, 750], 0, 0].sum())
    assert dropped >= 3 * 150 * len(ids)          # the bursts arrived (and overflowed the full queue)
