"""br_best_subset (the Stage-2 subproblem on windows of up to 32 requests) against the checker's
exhaustive enumeration, and beyond its reach against the reachable sums per subset size."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_06113_b200 import workload as wlm
from paper_2605_06113_b200.binding import Router

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,H", [("c3", 0), ("c2", 4), ("c4", 8)])
def test_best_subset_matches_exhaustive_enumeration(name, H):
    cfg = wlm.get_config(name)
    wl = wlm.make_workload(cfg, n_instances=1)
    r = Router(wl, device="cuda:0")
    rng = np.random.default_rng(17 + H)
    for R in [1, 2, 5, 8, 9, 12, 13, 16, 17, 20, 23]:
        N = 24 if R <= 16 else 6
        # small value ranges make equal sums (ties between masks) common
        hi = 40 if R % 2 else 3000
        win = rng.integers(1, hi, (N, R)).astype(np.int32)
        m = rng.integers(0, hi * max(1, R // 2), (N, H + 1)).astype(np.int64)
        lim = rng.integers(0, R + 2, N).astype(np.int32)
        lim[0] = 0; lim[1] = 1; lim[2] = R
        wt, mt, lt = (torch.from_numpy(x).cuda() for x in (win, m, lim))
        mask = torch.full((N,), 0xFFFF, dtype=torch.int32, device="cuda")
        F = torch.zeros((N,), dtype=torch.float64, device="cuda")
        r.best_subset(wt, mt, lt, mask, F)
        torch.cuda.synchronize()
        mh, Fh = mask.cpu().numpy(), F.cpu().numpy()
        for n in range(N):
            want_mask, want_f = oracle.best_subset(cfg.score_mode, cfg.G, H, cfg.alpha, cfg.beta, cfg.gamma,
                                                   m[n], win[n], int(min(lim[n], R)))
            if lim[n] < 1:
                want_mask, want_f = 0, 0.0
            assert int(mh[n]) == want_mask, (R, n)
            assert Fh[n] == want_f, (R, n)
    r.close()


def test_best_subset_twenty_entries():
    """The largest window: 2^20 - 1 subsets per problem, checked through the property that pins the
    optimum for Eq. 1 (largest reachable sum at or below the margin, or smallest above it)."""
    cfg = wlm.get_config("c3")
    wl = wlm.make_workload(cfg, n_instances=1)
    r = Router(wl, device="cuda:0")
    rng = np.random.default_rng(29)
    R, N = 20, 3
    win = rng.integers(50, 4000, (N, R)).astype(np.int32)
    m = rng.integers(1000, 30000, (N, 1)).astype(np.int64)
    lim = np.array([R, 4, 7], dtype=np.int32)
    wt, mt, lt = (torch.from_numpy(x).cuda() for x in (win, m, lim))
    mask = torch.zeros((N,), dtype=torch.int32, device="cuda")
    F = torch.zeros((N,), dtype=torch.float64, device="cuda")
    r.best_subset(wt, mt, lt, mask, F)
    torch.cuda.synchronize()
    for n in range(N):
        reach = [set() for _ in range(int(lim[n]) + 1)]
        reach[0].add(0)
        for s in win[n]:
            for j in range(int(lim[n]), 0, -1):
                reach[j] |= {x + int(s) for x in reach[j - 1]}
        sums = set().union(*reach[1:])
        best = max(oracle.f_br0(cfg.G, d, int(m[n, 0])) for d in sums)
        got = int(mask[n].item())
        assert 0 < got < (1 << R) and bin(got).count("1") <= lim[n]
        delta = sum(int(win[n, j]) for j in range(R) if got >> j & 1)
        assert oracle.f_br0(cfg.G, delta, int(m[n, 0])) == best == int(F[n].item())
    r.close()


@pytest.mark.parametrize("name,H", [("c3", 0), ("c4", 8)])
def test_best_subset_thirty_two_entries(name, H):
    """Windows of 25 to 32 requests (the halves meet in the middle).  The reachable sums per subset
    size come from the shift-or recurrence of Appendix "Bit-set subset selection" on Python
    integers; the best score over them is the optimum, and the returned subset must reach it."""
    cfg = wlm.get_config(name)
    wl = wlm.make_workload(cfg, n_instances=1)
    r = Router(wl, device="cuda:0")
    rng = np.random.default_rng(31 + H)
    for R in (25, 29, 32):
        N = 4
        win = rng.integers(20, 1500, (N, R)).astype(np.int32)
        win[3, : R // 2] = win[3, 0]                       # many equal entries
        m = rng.integers(500, 12000, (N, H + 1)).astype(np.int64)
        lim = np.array([R, 3, 11, R // 2], dtype=np.int32)
        wt, mt, lt = (torch.from_numpy(x).cuda() for x in (win, m, lim))
        mask = torch.zeros((N,), dtype=torch.int32, device="cuda")
        F = torch.zeros((N,), dtype=torch.float64, device="cuda")
        r.best_subset(wt, mt, lt, mask, F)
        torch.cuda.synchronize()
        for n in range(N):
            dp = [0] * (int(lim[n]) + 1)                   # dp[c] bit d: some c entries sum to d
            dp[0] = 1
            for s in win[n]:
                for c in range(int(lim[n]), 0, -1):
                    dp[c] |= dp[c - 1] << int(s)
            reach = 0
            for c in range(1, int(lim[n]) + 1):
                reach |= dp[c]
            sums = [d for d in range(reach.bit_length()) if reach >> d & 1]
            if H == 0:
                best = max(float(oracle.f_br0(cfg.G, d, int(m[n, 0]))) for d in sums)
            else:
                best = max(oracle.f_brh(H, cfg.alpha, cfg.beta, cfg.gamma, d, m[n]) for d in sums)
            got = int(mask[n].item()) & 0xFFFFFFFF
            assert 0 < got < (1 << R) and bin(got).count("1") <= lim[n], (R, n)
            delta = sum(int(win[n, j]) for j in range(R) if got >> j & 1)
            f = float(oracle.f_br0(cfg.G, delta, int(m[n, 0]))) if H == 0 else \
                oracle.f_brh(H, cfg.alpha, cfg.beta, cfg.gamma, delta, m[n])
            assert f == best == float(F[n].item()), (R, n)
    r.close()


def test_large_windows_need_the_two_probe_rule():
    """Without a strictly falling side (Eq. 1 with one worker; Eq. 2 with alpha = beta = gamma = 1) only
    enumeration is exact: windows beyond 20 requests are refused, smaller ones still solved."""
    from paper_2605_06113_b200.binding import BrError, BR_EINVAL
    for cfg in (wlm.get_config("c3", G=1), wlm.get_config("c2", alpha=1.0, beta=1.0, gamma=1.0)):
        wl = wlm.make_workload(cfg, n_instances=1)
        r = Router(wl, device="cuda:0")
        H = cfg.H
        for R, ok in ((16, True), (24, False)):
            win = torch.randint(1, 50, (2, R), dtype=torch.int32, device="cuda")
            m = torch.randint(0, 200, (2, H + 1), dtype=torch.int64, device="cuda")
            lim = torch.full((2,), R, dtype=torch.int32, device="cuda")
            mask = torch.zeros((2,), dtype=torch.int32, device="cuda")
            F = torch.zeros((2,), dtype=torch.float64, device="cuda")
            if ok:
                r.best_subset(win, m, lim, mask, F)
                torch.cuda.synchronize()
                for n in range(2):
                    wm, wf = oracle.best_subset(cfg.score_mode, cfg.G, H, cfg.alpha, cfg.beta, cfg.gamma,
                                                m[n].cpu().numpy(), win[n].cpu().numpy(), R)
                    assert int(mask[n].item()) == wm and float(F[n].item()) == wf
            else:
                with pytest.raises(BrError) as e:
                    r.best_subset(win, m, lim, mask, F)
                assert e.value.status == BR_EINVAL
        r.close()
