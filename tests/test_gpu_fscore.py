"""br_fscore (the F-score matrix and the pool-bypass arg-max) against the checker's Eq. 1 / Eq. 2."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from paper_2605_06113_b200 import workload as wlm
from paper_2605_06113_b200.binding import Router

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,H", [("c3", 0), ("c4", 8), ("c2", 4), ("h80", 80), ("c4", 33)])
def test_fscore_matrix_and_best_worker(name, H):
    cfg = wlm.get_config(name, H=H)
    wl = wlm.make_workload(cfg, n_instances=2)
    r = Router(wl, device="cuda:0")
    rng = np.random.default_rng(3 + H)
    N, G, n_req = 3, cfg.G, 2052                      # two full tiles and a ragged tail
    s = rng.integers(1, 60000, (N, n_req)).astype(np.int32)
    Lh = rng.integers(100000, 400000, (N, G, H + 1)).astype(np.int64)
    cap = rng.integers(0, 3, (N, G)).astype(np.int32)
    cap[2] = 0                                        # no worker has room: best_g = -1
    st, Lt, ct = (torch.from_numpy(x).cuda() for x in (s, Lh, cap))
    F = torch.zeros((N, n_req, G), dtype=torch.float64, device="cuda")
    best = torch.full((N, n_req), -7, dtype=torch.int32, device="cuda")
    r.fscore(st, Lt, F, cap=ct, best_g=best)
    torch.cuda.synchronize()
    Fh, bh = F.cpu().numpy(), best.cpu().numpy()
    M = Lh.max(axis=1)                                # envelope per offset
    for n in range(N):
        for i in list(range(0, 40)) + list(range(n_req - 40, n_req)) + [int(x) for x in rng.integers(0, n_req, 60)]:
            ref = np.empty(G)
            for g in range(G):
                m = M[n] - Lh[n, g]
                if cfg.score_mode == 0:
                    ref[g] = oracle.f_br0(G, int(s[n, i]), int(m[0]))
                else:
                    ref[g] = oracle.f_brh(H, cfg.alpha, cfg.beta, cfg.gamma, int(s[n, i]), m)
            err = np.abs(Fh[n, i] - ref) / np.maximum(1.0, np.abs(ref))
            assert err.max() <= 1e-6                  # stated tolerance
            assert np.array_equal(Fh[n, i], ref)      # same arithmetic, same order: equality
            ok = np.nonzero(cap[n] > 0)[0]
            want = -1 if len(ok) == 0 else int(ok[np.argmax(ref[ok])])
            assert bh[n, i] == want
    r.close()


@pytest.mark.parametrize("G,score_mode", [(32, 0), (64, 0), (5, 0), (16, 1)])
def test_pool_bypass_dispatch(G, score_mode):
    """br_bypass_dispatch against the checker: workers, virtual loads and inflight counts."""
    kw = dict(G=G, init_active=8, init_queue=0)
    if score_mode == 1:
        kw.update(score_mode=1, alpha=1.0, beta=7.5, gamma=1.0)
    cfg = wlm.get_config("c3", **kw)
    wl = wlm.make_workload(cfg, n_instances=1)
    r = Router(wl, device="cuda:0")
    rng = np.random.default_rng(71 + G)
    N, n_req = 9, 150
    s = rng.integers(1, 40000, (N, n_req)).astype(np.int32)
    s[0] = 1000                                            # equal lengths: ties between workers
    L = rng.integers(0, 300000, (N, G)).astype(np.int64)
    L[1] = 5000                                            # equal loads
    infl = rng.integers(0, 10, (N, G)).astype(np.int32)
    cap = rng.integers(8, 14, (N, G)).astype(np.int32)     # tight caps: some instances fill up
    cap[2] = 0
    st, Lt, it, ct = (torch.from_numpy(x.copy()).cuda() for x in (s, L, infl, cap))
    out = torch.full((N, n_req), -7, dtype=torch.int32, device="cuda")
    r.bypass_dispatch(st, Lt, it, ct, out)
    torch.cuda.synchronize()
    for n in range(N):
        want, Lw, nw = oracle.bypass(G, s[n], L[n], infl[n], cap[n], score_mode=score_mode, alpha=cfg.alpha,
                                     beta=float(G) if score_mode == 0 else cfg.beta)
        assert np.array_equal(out[n].cpu().numpy(), want), n
        assert np.array_equal(Lt[n].cpu().numpy(), Lw) and np.array_equal(it[n].cpu().numpy(), nw), n
    assert (out[2] == -1).all()
    r.close()


def test_empirical_survival_estimator():
    """br_survival_chat against the checker's counting definition (same fp64 operations: equality)."""
    cfg = wlm.get_config("c4")                              # H = 8
    wl = wlm.make_workload(cfg, n_instances=1)
    r = Router(wl, device="cuda:0")
    rng = np.random.default_rng(83)
    hist = np.sort(rng.geometric(1 / 600.0, 5000).astype(np.int32))
    prefix = np.concatenate([[0], np.cumsum(hist.astype(np.int64))]).astype(np.int64)
    age = np.concatenate([rng.integers(0, 3000, 3000), [0, int(hist[-1]) - 1, int(hist[-1]), int(hist[-1]) + 9,
                                                        int(hist[0]) - 1, int(hist[0])]]).astype(np.int32)
    ht, pt, at = (torch.from_numpy(x).cuda() for x in (hist, prefix, age))
    c = torch.empty(len(age), dtype=torch.float32, device="cuda")
    p = torch.empty(len(age), dtype=torch.float64, device="cuda")
    mu = torch.empty(len(age), dtype=torch.float64, device="cuda")
    r.survival_chat(ht, pt, at, c, p, mu)
    torch.cuda.synchronize()
    ch, ph, mh = c.cpu().numpy(), p.cpu().numpy(), mu.cpu().numpy()
    shuffled = rng.permutation(hist)                        # the definition does not need the order
    for i in list(range(400)) + list(range(len(age) - 6, len(age))):
        wc, wp, wm = oracle.survival(shuffled, cfg.H, int(age[i]))
        assert ch[i] == np.float32(wc) and ph[i] == wp and mh[i] == wm, i
    r.close()
