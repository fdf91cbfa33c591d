"""Pins for the CPU reference checker: closed forms, identities and brute force
that the paper and the mathematics fix, so that a dropped term, a wrong sign or a
wrong index in the checker fails here before anything is compared with it."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2605_06113_b200 import workload as wlm

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
EMPTY = oracle.EMPTY


# ---------------------------------------------------------------- Philox
def _philox_py(ctr, key):
    """Independent big-integer restatement of Philox4x32-10 (SC'11, Section 5.3)."""
    c = list(ctr); k = list(key)
    for _ in range(10):
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [((p1 >> 32) ^ c[1] ^ k[0]) & 0xFFFFFFFF, p1 & 0xFFFFFFFF,
             ((p0 >> 32) ^ c[3] ^ k[1]) & 0xFFFFFFFF, p0 & 0xFFFFFFFF]
        k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
    return c


def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        out = oracle.philox4x32_10(v[0:4], v[4:6])
        assert [int(x) for x in out] == v[6:10]


def test_philox_against_bigint_and_uniformity():
    rng = np.random.default_rng(7)
    for _ in range(200):
        ctr = [int(x) for x in rng.integers(0, 2 ** 32, 4)]
        key = [int(x) for x in rng.integers(0, 2 ** 32, 2)]
        assert [int(x) for x in oracle.philox4x32_10(ctr, key)] == _philox_py(ctr, key)
    # consecutive counters give words that look uniform: mean and a 16-bin chi-square
    words = np.concatenate([oracle.philox4x32_10([i, 0, 2, 0], [5, 0]) for i in range(5000)])
    u = words.astype(np.float64) / 2 ** 32
    assert abs(u.mean() - 0.5) < 4 * (1 / np.sqrt(12 * u.size))
    hist = np.bincount((words >> 28).astype(np.int64), minlength=16)
    chi2 = ((hist - u.size / 16) ** 2 / (u.size / 16)).sum()
    assert chi2 < 45.0           # 15 dof, p ~ 1e-4


# ---------------------------------------------------------------- Eq. 1
@pytest.mark.parametrize("G", [2, 3, 8, 64])
def test_eq1_closed_forms(G):
    for m in [0, 1, 5, 17, 1000]:
        for d in range(0, 3 * m + 40):
            F = oracle.f_br0(G, d, m)
            if d <= m:
                assert F == d                                   # safe regime
            else:
                assert F == G * m - (G - 1) * d                 # overflow regime
            # sign: F > 0  <=>  Delta < G m / (G - 1), Delta > 0
            assert (F > 0) == (d > 0 and Fraction(d) < Fraction(G * m, G - 1))
        assert oracle.f_br0(G, m, m) == m                       # the two branches meet at the kink
        for delta in [1, 2, 7]:
            if m - delta >= 0:
                assert oracle.f_br0(G, m, m) - oracle.f_br0(G, m - delta, m) == delta
            assert oracle.f_br0(G, m + delta, m) - oracle.f_br0(G, m, m) == -(G - 1) * delta


def test_eq1_is_minus_delta_imbalance():
    """F_g(Q) = -(I_after - I_before) with I recomputed from the definition."""
    rng = np.random.default_rng(11)
    for _ in range(2000):
        G = int(rng.integers(2, 12))
        L = rng.integers(0, 5000, G).astype(np.int64)
        g = int(rng.integers(0, G))
        d = int(rng.integers(0, 6000))
        I0 = G * int(L.max()) - int(L.sum())
        L2 = L.copy(); L2[g] += d
        I1 = G * int(L2.max()) - int(L2.sum())
        m = int(L.max() - L[g])
        assert oracle.f_br0(G, d, m) == -(I1 - I0)
        assert oracle.imbalance(L) == I0


# ---------------------------------------------------------------- Eq. 2
def _f_brh_exact(H, alpha, beta, gamma, delta, m):
    """Eq. 2 in exact rational arithmetic."""
    a, b, g = Fraction(alpha), Fraction(beta), Fraction(gamma)
    d = [g ** h for h in range(H + 1)]
    pen = sum(d[h] * max(delta - int(m[h]), 0) for h in range(H + 1))
    return a * sum(d) * delta - b * pen


def test_eq2_reduces_to_eq1_at_h0():
    rng = np.random.default_rng(3)
    for _ in range(2000):
        G = int(rng.integers(2, 65))
        m = int(rng.integers(0, 10 ** 6)); d = int(rng.integers(0, 10 ** 6))
        assert oracle.f_brh(0, 1.0, float(G), 0.64, d, [m]) == float(oracle.f_br0(G, d, m))


def test_eq2_against_exact_rationals_and_regimes():
    rng = np.random.default_rng(5)
    for _ in range(1500):
        H = int(rng.integers(0, 17))
        alpha = float(rng.choice([1.0, 0.5, 2.0])); beta = float(rng.choice([14.67, 43.0, 48.0, 8.0]))
        gamma = float(rng.choice([0.64, 0.86, 0.9, 1.0]))
        m = rng.integers(0, 200000, H + 1)
        d = int(rng.integers(0, 400000))
        F = oracle.f_brh(H, alpha, beta, gamma, d, m)
        exact = _f_brh_exact(H, alpha, beta, gamma, d, m)
        scale = max(1.0, abs(float(exact)), alpha * (H + 1) * d)
        assert abs(F - float(exact)) <= 1e-12 * scale
        dvec, D = oracle.discount(H, gamma)
        if d <= m.min():                                   # horizon-safe: penalty vanishes
            assert F == (alpha * D) * d
    # gamma = 1 and equal margins: (H+1)(alpha Delta - beta (Delta - m)_+), exactly
    for H in [1, 4, 8]:
        for d in [0, 10, 99, 100, 101, 500]:
            F = oracle.f_brh(H, 1.0, 8.0, 1.0, d, [100] * (H + 1))
            assert F == (H + 1) * (d - 8.0 * max(d - 100, 0))


def test_eq2_kinks_and_slopes():
    """Piecewise linear with kinks at the distinct margins; slope after passing the
    set P of kinks is alpha 1^T d - beta sum_{h in P} gamma^h."""
    H, alpha, beta, gamma = 3, 1.0, 4.0, 0.5          # dyadic: every value exact in fp64
    m = [40, 10, 30, 20]
    d = [gamma ** h for h in range(H + 1)]
    for delta in range(0, 60):
        slope = oracle.f_brh(H, alpha, beta, gamma, delta + 1, m) - oracle.f_brh(H, alpha, beta, gamma, delta, m)
        passed = [h for h in range(H + 1) if m[h] <= delta]
        assert slope == alpha * sum(d) - beta * sum(d[h] for h in passed)


# ---------------------------------------------------------------- c_hat
def test_chat_identity_eq4_and_special_cases():
    rng = np.random.default_rng(9)
    for _ in range(500):
        H = int(rng.integers(1, 17))
        q = rng.beta(2, 20, H).astype(np.float32)
        c, p = oracle.chat_star(q)
        c2, p2, mu = oracle.chat_two_stage(q)
        assert abs(c - c2) < 1e-12 * H and abs(p - p2) < 1e-12
        assert 0.0 < mu <= H and 0.0 <= c <= H
        # exact rational evaluation of E[min(r, H)]
        qs = [Fraction(float(x)) for x in q]
        surv, tot = Fraction(1), Fraction(0)
        for h in range(H):
            tot += surv; surv *= 1 - qs[h]
        assert abs(c - float(tot)) < 1e-13 * H
    for H in [1, 2, 4, 8, 16]:
        assert oracle.chat_star([0.0] * H) == (float(H), 0.0)             # never finishes: anchor H
        c, p = oracle.chat_star([1.0] + [0.3] * (H - 1))
        assert (c, p) == (1.0, 1.0)                                       # finishes at the first step
        c, p = oracle.chat_star([0.5] * H)                                # all q = 1/2: closed forms
        assert c == 2.0 - 2.0 ** (1 - H) and p == 1.0 - 2.0 ** (-H)


def test_chat_matches_simulated_expectation():
    rng = np.random.default_rng(21)
    H = 6
    q = np.array([0.1, 0.3, 0.05, 0.2, 0.4, 0.15], dtype=np.float32)
    n = 400000
    alive = np.ones(n, dtype=bool); r = np.full(n, H + 5)
    for h in range(1, H + 1):
        fin = alive & (rng.random(n) < q[h - 1])
        r[fin] = h; alive &= ~fin
    mc = np.minimum(r, H).mean()
    c, p = oracle.chat_star(q)
    assert abs(mc - c) < 5 * np.minimum(r, H).std() / np.sqrt(n)
    assert abs((r <= H).mean() - p) < 5 * 0.5 / np.sqrt(n)


def _mk(G=2, H=4, B=4, W=8, **kw):
    return oracle.Instance(G=G, H=H, B=B, W=W, **kw)


def test_refresh_rules_branch_table():
    """Periodic refresh, confidence gate, floor (Appendix 'Refresh logic')."""
    H, dT = 8, 4
    o = _mk(G=1, H=H, B=8, W=4, delta_T=dT, gate=0.5, c_floor=1.0, beta=14.67, gamma=0.64)
    base = np.full((1, 8), EMPTY, dtype=np.int32); base[0, :6] = 100
    chat = np.array([[8.0, 5.0, 1.5, 8.0, 3.25, 2.0, 0, 0]], dtype=np.float32)
    tau = np.array([[0, 1, 0, 3, 2, 3, 0, 0]], dtype=np.int32)
    o.set_state(0, 0, base, None, chat, tau, None, None, 0)
    hi = np.full(H, 0.5, dtype=np.float32)            # p_fin = 1 - 2^-8 >= gate, c* = 2 - 2^-7
    lo = np.full(H, 0.01, dtype=np.float32)           # p_fin ~ 0.077 < gate
    probs = np.stack([hi, hi, hi, hi, lo, lo, hi, hi])[None]
    o.predict_only(probs)
    st = o.get_state()
    cs = 2.0 - 2.0 ** -7
    # slot0: tau 0->1 < dT, 8-1=7 >= floor: plain decrement
    assert (st["chat"][0, 0], st["tau"][0, 0]) == (7.0, 1)
    # slot1: decrement to 4, tau 2
    assert (st["chat"][0, 1], st["tau"][0, 1]) == (4.0, 2)
    # slot2: 1.5-1 = 0.5 < floor -> immediate refresh, gate open -> c*
    assert (st["chat"][0, 2], st["tau"][0, 2]) == (np.float32(cs), 0)
    # slot3: tau 3->4 = dT -> periodic refresh, gate open
    assert (st["chat"][0, 3], st["tau"][0, 3]) == (np.float32(cs), 0)
    # slot4: no refresh due (tau 3 < 4, 2.25 >= 1): decrement
    assert (st["chat"][0, 4], st["tau"][0, 4]) == (2.25, 3)
    # slot5: periodic refresh but gate closed -> anchor H
    assert (st["chat"][0, 5], st["tau"][0, 5]) == (float(H), 0)
    # clip to the floor: q_1 = 1 gives c* = 1; with floor 2 it is raised to 2
    o2 = _mk(G=1, H=H, B=8, W=4, delta_T=1, gate=0.5, c_floor=2.0)
    o2.set_state(0, 0, base, None, chat, tau, None, None, 0)
    one = np.zeros((1, 8, H), dtype=np.float32); one[..., 0] = 1.0
    o2.predict_only(one)
    assert np.all(o2.get_state()["chat"][0, :6] == 2.0)


def test_projection_closed_form_and_eq6():
    rng = np.random.default_rng(4)
    G, H, B = 3, 5, 6
    o = _mk(G=G, H=H, B=B, W=4, delta_T=100)
    base = np.full((G, B), EMPTY, dtype=np.int32)
    occ = rng.random((G, B)) < 0.7
    base[occ] = rng.integers(16, 5000, occ.sum())
    k = 37
    # all c_hat = H: L_g(k+h) = L_g(k) + h n_g
    o.set_state(k, 0, base, None, np.full((G, B), H, np.float32), np.zeros((G, B), np.int32), None, None, 0)
    Lh, Mh, m = o.projection()
    cur = np.where(occ, base.astype(np.int64) + k, 0)
    for h in range(H + 1):
        assert np.array_equal(Lh[:, h], cur.sum(1) + h * occ.sum(1))
    assert np.array_equal(Mh, Lh.max(0)) and np.array_equal(m, Mh[None] - Lh) and (m >= 0).all()
    # general c_hat: a request is counted at offset h iff h = 0 or h <= c_hat
    chat = rng.uniform(1, H, (G, B)).astype(np.float32)
    o.set_state(k, 0, base, None, chat, np.zeros((G, B), np.int32), None, None, 0)
    Lh, Mh, m = o.projection()
    for h in range(H + 1):
        inw = occ & ((h == 0) | (h <= chat))
        assert np.array_equal(Lh[:, h], ((cur + h) * inw).sum(1))
    assert np.array_equal(Lh[:, 0], cur.sum(1))          # offset 0 is L_g(k)


# ---------------------------------------------------------------- Stage 2 subproblem
@pytest.mark.parametrize("mode", [0, 1])
def test_best_subset_is_brute_force_optimum(mode):
    rng = np.random.default_rng(13 + mode)
    for _ in range(400):
        G = int(rng.integers(2, 20)); H = 0 if mode == 0 else int(rng.integers(1, 6))
        alpha, beta, gamma = (1.0, float(G), 1.0) if mode == 0 else (1.0, 4.0, 0.5)
        nw = int(rng.integers(1, 5)); lim = int(rng.integers(1, 5))
        win = sorted((int(x) for x in rng.integers(1, 300, nw)), reverse=True)
        m = rng.integers(0, 600, H + 1)
        mask, f = oracle.best_subset(mode, G, H, alpha, beta, gamma, m, win, lim)
        best = None
        for r in range(1, min(lim, nw) + 1):
            for comb in itertools.combinations(range(nw), r):
                d = sum(win[j] for j in comb)
                val = _f_brh_exact(H, alpha, beta, gamma, d, m)
                mk = sum(1 << j for j in comb)
                if best is None or val > best[0] or (val == best[0] and mk < best[1]):
                    best = (val, mk)
        assert float(best[0]) == f and best[1] == mask


# ---------------------------------------------------------------- whole routing round
def _random_snapshot(rng, G, B, W, H=0, full=0.6, nq=None, smax=400):
    base = np.full((G, B), EMPTY, dtype=np.int32)
    for g in range(G):
        n = int(rng.integers(0, B + 1)) if full is None else int(rng.binomial(B, full))
        idx = rng.permutation(B)[:n]
        base[g, idx] = rng.integers(1, smax, n)
    nq = int(rng.integers(0, W + 1)) if nq is None else nq
    qs = np.zeros(W, dtype=np.int32); qs[:nq] = rng.integers(1, smax, nq)
    return base, qs, nq


@pytest.mark.parametrize("H", [0, 3])
def test_round_invariants(H):
    """Feasibility, liveness (no idle slot while requests wait), stickiness of the
    running set, and for BR-0 the telescoped identity sum F = I_before - I_after."""
    rng = np.random.default_rng(17 + H)
    for trial in range(300):
        G = int(rng.integers(2, 7)); B = int(rng.integers(1, 6)); W = 12
        S_greedy = int(rng.choice([0, G, 2 * G, G * B]))
        o = oracle.Instance(G=G, H=H, B=B, W=W, S_greedy=S_greedy, R_max=int(rng.integers(1, 5)),
                            beta=(None if H == 0 else 4.0), gamma=0.5, delta_T=50)
        base, qs, nq = _random_snapshot(rng, G, B, W, H)
        o.set_state(0, 0, base, None, np.full((G, B), H, np.float32), np.zeros((G, B), np.int32),
                    qs, None, nq)
        L0 = np.where(base != EMPTY, base, 0).astype(np.int64).sum(1)
        cap0 = (base == EMPTY).sum(1)
        assign, L1 = o.route_only()
        st = o.get_state()
        adm = np.nonzero(assign >= 0)[0]
        assert len(adm) == min(int(cap0.sum()), nq)                  # liveness
        assert np.all(assign[nq:] == -1)
        slots = assign[adm]
        assert len(set(slots.tolist())) == len(slots)                # one request per slot
        assert np.all(base.reshape(-1)[slots] == EMPTY)              # only free slots are used
        keep = base != EMPTY
        assert np.array_equal(st["act_base"][keep], base[keep])      # running requests never move
        add = np.zeros(G, dtype=np.int64)
        np.add.at(add, slots // B, qs[adm])
        assert np.array_equal(L1, L0 + add)
        assert np.all(cap0 - np.bincount(slots // B, minlength=G) >= 0)
        assert np.array_equal(st["wq_s"][:st["wq_n"]], np.delete(qs[:nq], adm))   # stable removal
        # lowest free slot first, per worker
        for g in range(G):
            used = sorted(s % B for s in slots if s // B == g)
            free = [b for b in range(B) if base[g, b] == EMPTY]
            assert used == free[:len(used)]


def _exhaustive_min_imbalance(L, caps, qs, n_fill):
    """Smallest I over all assignments that fill n_fill slots (tiny instances only)."""
    G = len(L); best = None
    for subset in itertools.combinations(range(len(qs)), n_fill):
        for dest in itertools.product(range(G), repeat=n_fill):
            cnt = np.bincount(dest, minlength=G)
            if np.any(cnt > caps):
                continue
            L2 = L.copy()
            for i, g in zip(subset, dest):
                L2[g] += qs[i]
            I = G * L2.max() - L2.sum()
            if best is None or I < best:
                best = I
    return best


def test_br0_against_exhaustive_assignment_tiny():
    """BR is a heuristic: it can not beat the exhaustive optimum and is usually close."""
    rng = np.random.default_rng(23)
    gaps = []
    for _ in range(60):
        G = int(rng.integers(2, 4)); B = 3; W = 6
        o = oracle.Instance(G=G, H=0, B=B, W=W, S_greedy=int(rng.choice([0, G])))
        base = np.full((G, B), EMPTY, dtype=np.int32)
        caps = rng.integers(0, 3, G)
        for g in range(G):
            base[g, :B - caps[g]] = rng.integers(1, 200, B - caps[g])
        nq = int(rng.integers(1, 6)); qs = np.zeros(W, np.int32); qs[:nq] = rng.integers(1, 200, nq)
        o.set_state(0, 0, base, None, None, None, qs, None, nq)
        L0 = np.where(base != EMPTY, base, 0).astype(np.int64).sum(1)
        assign, L1 = o.route_only()
        n_fill = int((assign >= 0).sum())
        assert n_fill == min(int(caps.sum()), nq)
        I_br = G * L1.max() - L1.sum()
        I_opt = _exhaustive_min_imbalance(L0, caps, qs[:nq].astype(np.int64), n_fill)
        assert I_br >= I_opt
        gaps.append(I_br - I_opt)
    assert np.mean(np.array(gaps) == 0) > 0.3       # often optimal on tiny cases


def test_single_admission_is_the_argmax_of_eq1():
    """One free slot: the admitted request maximises F over R_wait, i.e. minimises
    the imbalance after admission (brute force), earliest arrival on ties."""
    rng = np.random.default_rng(29)
    for _ in range(300):
        G = int(rng.integers(2, 8)); B = 2; W = 10
        o = oracle.Instance(G=G, H=0, B=B, W=W, S_greedy=0)
        base = rng.integers(1, 300, (G, B)).astype(np.int32)
        g_free = int(rng.integers(0, G)); base[g_free, 1] = EMPTY
        nq = int(rng.integers(1, W + 1)); qs = np.zeros(W, np.int32); qs[:nq] = rng.integers(1, 300, nq)
        o.set_state(0, 0, base, None, None, None, qs, None, nq)
        L0 = np.where(base != EMPTY, base, 0).astype(np.int64).sum(1)
        assign, L1 = o.route_only()
        I_after = []
        for i in range(nq):
            L2 = L0.copy(); L2[g_free] += qs[i]
            I_after.append(G * L2.max() - L2.sum())
        # S_greedy = 0 sends the one slot through Stage 1, whose choice is the F-argmax
        assert int(np.nonzero(assign >= 0)[0][0]) == int(np.argmin(I_after))


def test_brh_path_at_h0_equals_br0_on_whole_runs():
    """Running the horizon code path with H = 0 and (alpha, beta) = (1, G) reproduces
    BR-0 step for step (Section 4.1, 'Reduction to BR-0')."""
    for name, steps in [("c0", 300), ("c1", 400)]:
        cfg = wlm.get_config(name)
        wl = wlm.make_workload(cfg)
        a = oracle.instance_from_workload(wl, 0)
        b = oracle.instance_from_workload(wl, 0, score_mode=1, alpha=1.0, beta=float(cfg.G), gamma=0.64)
        for k in range(steps):
            ra = a.step(); rb = b.step()
            assert np.array_equal(ra[0], rb[0]) and np.array_equal(ra[1], rb[1])
            assert np.array_equal(ra[2], rb[2])


# ---------------------------------------------------------------- model / advance
def test_advance_growth_and_loads_from_scratch():
    cfg = wlm.get_config("c0", term_mode=0)
    wl = wlm.make_workload(cfg)
    o = oracle.instance_from_workload(wl, 0)
    prev_load, prev_n = None, None
    for k in range(60):
        st0 = o.get_state()
        assign, load, trace, _ = o.step()
        st1 = o.get_state()
        occ1 = st1["act_base"] != EMPTY
        # no terminations: every running request grew by one token, so base = cur - k is constant
        keep = st0["act_base"] != EMPTY
        assert np.array_equal(st1["act_base"][keep], st0["act_base"][keep])
        cur_k = np.where(occ1, st1["act_base"].astype(np.int64) + k, 0)   # loads at step k
        assert np.array_equal(load, cur_k.sum(1))
        assert (trace[0], trace[1], trace[2]) == (load.max(), load.min(), load.sum())
        if prev_load is not None:
            adm = np.zeros(cfg.G, np.int64)
            sl = assign[assign >= 0]
            np.add.at(adm, sl // cfg.B, st1["act_base"].reshape(-1)[sl].astype(np.int64) + k)
            assert np.array_equal(load, prev_load + prev_n + adm)        # L(k) = L(k-1) + n + admitted
        prev_load, prev_n = load, occ1.sum(1)
        # a request admitted at k enters with load s_i: base = s_i - k
        for pos in np.nonzero(assign >= 0)[0]:
            assert st1["act_base"].reshape(-1)[assign[pos]] + k == _queue_after_arrive(st0, st1, wl, k)[pos]


def _queue_after_arrive(st0, st1, wl, k):
    """Queue contents right after ARRIVE of step k, rebuilt from the Philox definition."""
    key = [int(wl.seeds[0]) & 0xFFFFFFFF, int(wl.seeds[0]) >> 32]
    u = _philox_py([k, 0, 0, 0], key)[0]
    row = wl.arr_rows_for(0)[k % wl.arr_period]
    n = int((u >= row.astype(np.int64)).sum())
    q = list(st0["wq_s"][:st0["wq_n"]])
    for j in range(n):
        r = _philox_py([k, j // 4, 1, 0], key)[j % 4]
        if len(q) < wl.cfg.W:
            q.append(int(wl.len_tab[r >> 16]))
    return q


def test_terminations_follow_the_hazard():
    cfg = wlm.get_config("c1")
    wl = wlm.make_workload(cfg)
    o = oracle.instance_from_workload(wl, 0)
    fin = 0; exposure = 0
    for k in range(600):
        o.step()
        st = o.get_state()
        exposure += 1024
    # workers stay (nearly) full, so terminations = admissions ~ hazard * exposure
    adm = int(o.get_state()["counters"][1])
    assert abs(adm - exposure / 400.0) < 5 * np.sqrt(exposure / 400.0) + 20


def test_bernoulli_terminations_use_the_step_probability():
    """term_mode 2: a slot with probability 0 never ends, with probability 1 ends at once."""
    G, B, H = 2, 4, 2
    o = oracle.Instance(G=G, H=H, B=B, W=4, term_mode=2, beta=4.0, gamma=0.5)
    base = np.full((G, B), 50, dtype=np.int32)
    o.set_state(0, 0, base, None, np.full((G, B), H, np.float32), np.zeros((G, B), np.int32), None, None, 0)
    probs = np.zeros((G, B, H), dtype=np.float32); probs[0, :, 0] = 1.0
    o.step(probs)
    st = o.get_state()
    assert np.all(st["act_base"][0] == EMPTY) and np.all(st["act_base"][1] == 50)


# ---------------------------------------------------------------- comparison routers
def test_round_robin_and_least_loaded():
    rng = np.random.default_rng(31)
    G, B, W = 5, 8, 23
    base = np.full((G, B), EMPTY, dtype=np.int32)
    qs = rng.integers(1, 500, W).astype(np.int32)
    rr = oracle.Instance(G=G, H=0, B=B, W=W, router=1)
    rr.set_state(0, 0, base, None, None, None, qs, None, W)
    assign, L = rr.route_only()
    cnt = np.bincount(assign[assign >= 0] // B, minlength=G)
    assert cnt.max() - cnt.min() <= 1 and cnt.sum() == W
    assert np.array_equal(assign[:G] // B, np.arange(G))          # cyclic order from worker 0
    # least-loaded on equal sizes is greedy list scheduling: loads differ by at most one job
    ll = oracle.Instance(G=G, H=0, B=B, W=W, router=2)
    ll.set_state(0, 0, base, None, None, None, np.full(W, 7, np.int32), None, W)
    assign, L = ll.route_only()
    assert L.max() - L.min() <= 7 and L.sum() == 7 * W
    # general sizes: textbook greedy (each job to the currently least loaded machine)
    ll2 = oracle.Instance(G=G, H=0, B=B, W=W, router=2)
    ll2.set_state(0, 0, base, None, None, None, qs, None, W)
    assign, L = ll2.route_only()
    ref = np.zeros(G, np.int64)
    for i in range(W):
        g = int(np.argmin(ref)); ref[g] += qs[i]
        assert assign[i] // B == g
    assert np.array_equal(L, ref)


def test_balanceroute_beats_baselines_on_imbalance():
    """Context check of the paper's headline ordering on a synthetic trace: average
    max-min load of BR-0 is below least-loaded and round-robin (Table 1 ordering)."""
    cfg = wlm.get_config("c1")
    wl = wlm.make_workload(cfg)
    res = {}
    for router in (0, 1, 2):
        o = oracle.instance_from_workload(wl, 0, router=router)
        gaps = []
        for k in range(800):
            _, _, tr, _ = o.step()
            gaps.append(tr[0] - tr[1])
        res[router] = float(np.mean(gaps[200:]))
    assert res[0] < res[2] and res[0] < res[1]


# ---------------------------------------------------------------- input tables
def test_workload_tables_match_their_distributions():
    t = wlm.lognormal_table(7.0, 1.0, 1, 10 ** 9).astype(np.float64)
    assert abs(np.log(t).mean() - 7.0) < 0.01 and abs(np.log(t).std() - 1.0) < 0.01
    b = wlm.beta_table(2.0, 50.0).astype(np.float64)
    assert abs(b.mean() - 2 / 52) < 1e-4
    assert abs(b.var() - (2 * 50) / (52 ** 2 * 53)) < 1e-5
    for lam in [2.0, 8.0, 20.0]:
        thr = wlm.poisson_thresholds([lam])[0].astype(np.float64)
        pmf = np.diff(np.concatenate([[0.0], thr / 2 ** 32]))
        mean = (np.arange(len(pmf)) * pmf).sum()
        assert abs(mean - lam) < 1e-3
    # gap thresholds of the constant hazard: P(gap = j) = p (1 - p)^j on the 32-bit scale
    for p, B in [(1 / 500, 64), (1 / 400, 64), (0.05, 16), (0.5, 8)]:
        t = wlm.termination_gap_thresholds(p, B).astype(np.float64)
        assert t[0] == np.floor(p * 2 ** 32) and np.all(np.diff(t) >= 0)
        pmf = np.diff(np.concatenate([[0.0], t])) / 2 ** 32
        assert np.abs(pmf - p * (1 - p) ** np.arange(B)).max() < 2.0 ** -31
    assert not wlm.termination_gap_thresholds(0.0, 8).any()
    # numpy and torch flavours of the counter mixer agree
    import torch
    seeds = np.arange(5, dtype=np.uint64) + np.uint64(2 ** 63 + 12345)
    idx = np.arange(1000, dtype=np.uint64)[None, :]
    a = wlm.mix_np(seeds[:, None], 4, idx)
    bt = wlm.mix_torch(torch.from_numpy(seeds.astype(np.int64))[:, None], 4,
                       torch.arange(1000, dtype=torch.int64)[None, :])
    assert np.array_equal(a.astype(np.int64), bt.numpy())
    cfg = wlm.get_config("c2")
    wl = wlm.make_workload(cfg)
    assert np.array_equal(wlm.term_probs_np(wl, 17), wlm.term_probs_torch(wl, 17, "cpu").numpy())


def test_stored_traces_are_reproduced():
    """The stored traces (written from the checker by tests/golden/make_golden.py) guard
    against unintended changes of the checker's arithmetic."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(GOLDEN, "make_golden.py"))
    mg = importlib.util.module_from_spec(spec); spec.loader.exec_module(mg)
    for name, steps in (("c0", 300), ("c2", 200)):
        want = [tuple(int(x) for x in l.split()) for l in open(os.path.join(GOLDEN, f"{name}_trace.txt"))
                if not l.startswith("#")]
        assert mg.run(name, steps) == want


def test_gap_of_a_word_is_the_count_of_thresholds_at_or_below_it():
    """A uniform word u skips gap = #{j : u >= t[j]} slots: gap <= j exactly when u < t[j], so
    P(gap <= j) = t[j] / 2^32 (the table is that CDF)."""
    rng = np.random.default_rng(41)
    for p, B in [(1 / 500, 64), (0.05, 16), (0.5, 8), (0.0, 8), (1.0, 8)]:
        t = wlm.termination_gap_thresholds(p, B)
        us = [0, 1, 0xFFFFFFFF] + [int(x) for x in rng.integers(0, 2 ** 32, 40)]
        for j in range(B):
            us += [int(t[j]), max(int(t[j]) - 1, 0), min(int(t[j]) + 1, 0xFFFFFFFF)]
        for u in us:
            gap = oracle.term_gap(t, u)
            assert 0 <= gap <= B
            for j in range(B):
                assert (gap <= j) == (u < int(t[j]))


def test_constant_hazard_slots_end_independently_with_probability_p():
    """term_mode 1 realises independent Bernoulli(p) endings per slot and step (Section 2.2: each
    running request ends with a fixed probability per step).  Checked on the law itself: per-slot
    frequencies, the number ending per worker-step (binomial mean and variance), joint endings of
    slot pairs, and the realised ending sets rebuilt from the Philox definition."""
    G, B, p, steps = 3, 16, 0.08, 6000
    t = wlm.termination_gap_thresholds(p, B)
    seed = 0x1234_5678_9ABC_DEF1
    o = oracle.Instance(G=G, H=0, B=B, W=4, term_mode=1, term_cdf=t, seed=seed)
    base = np.full((G, B), 1000, dtype=np.int32)
    ended = np.zeros((steps, G, B), dtype=bool)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for k in range(steps):
        o.set_state(k, 0, base - k, None, None, None, None, None, 0)     # all slots running again
        o.step()
        ended[k] = o.get_state()["act_base"] == EMPTY
        if k < 40:
            for g in range(G):       # the same sets from the definition: walk the gaps
                want = np.zeros(B, dtype=bool); pos = 0; d = 0
                while pos < B:
                    u = _philox_py([k, g, 2, d // 4], key)[d % 4]
                    slot = pos + int((u >= t.astype(np.int64)).sum())
                    if slot >= B:
                        break
                    want[slot] = True; pos = slot + 1; d += 1
                assert np.array_equal(ended[k, g], want)
    n = steps * G
    freq = ended.reshape(n, B).mean(0)
    assert np.abs(freq - p).max() < 5 * np.sqrt(p * (1 - p) / n)
    cnt = ended.reshape(n, B).sum(1)
    assert abs(cnt.mean() - B * p) < 5 * np.sqrt(B * p * (1 - p) / n)
    assert abs(cnt.var() - B * p * (1 - p)) < 0.1 * B * p * (1 - p)
    e = ended.reshape(n, B)
    for i, j in [(0, 1), (0, B - 1), (3, 4), (7, 12)]:
        both = (e[:, i] & e[:, j]).mean()
        assert abs(both - p * p) < 5 * np.sqrt(p * p / n)
    # a slot that is free when the step ends is unaffected, an occupied one follows the same draw
    o2 = oracle.Instance(G=G, H=0, B=B, W=4, term_mode=1, term_cdf=t, seed=seed)
    k7 = int(np.argmax(ended[:, :, 1::2].sum((1, 2))))                  # a step where odd slots end
    half = base - k7; half[:, ::2] = EMPTY
    o2.set_state(k7, 0, half, None, None, None, None, None, 0)
    o2.step()
    got = o2.get_state()["act_base"] == EMPTY
    assert ended[k7][:, 1::2].any()
    assert np.array_equal(got[:, 1::2], ended[k7][:, 1::2]) and got[:, ::2].all()


def test_best_subset_agrees_with_reachable_sums_and_two_probe_rule():
    """The Stage-2 subproblem depends on Q only through Delta(Q) (Appendix 'Bit-set subset
    selection'): a second, independent solver that enumerates the reachable sums per cardinality
    must find the same optimum, and for BR-0 the optimum is one of two probes: the largest
    reachable sum at or below the margin, or the smallest one above it."""
    rng = np.random.default_rng(47)
    for _ in range(300):
        G = int(rng.integers(2, 33)); nw = int(rng.integers(1, 6)); lim = int(rng.integers(1, 6))
        win = sorted((int(x) for x in rng.integers(1, 400, nw)), reverse=True)
        m = int(rng.integers(0, 900))
        reach = [set() for _ in range(lim + 1)]        # reach[j] = sums of exactly j window entries
        reach[0].add(0)
        for s in win:
            for j in range(min(lim, nw), 0, -1):
                reach[j] |= {x + s for x in reach[j - 1]}
        sums = sorted(set().union(*reach[1:]))
        mask, f = oracle.best_subset(0, G, 0, 1.0, float(G), 1.0, [m], win, lim)
        assert f == max(oracle.f_br0(G, d, m) for d in sums)
        below = [d for d in sums if d <= m]
        above = [d for d in sums if d > m]
        probes = ([max(below)] if below else []) + ([min(above)] if above else [])
        assert f == max(oracle.f_br0(G, d, m) for d in probes)
        assert sum(win[j] for j in range(nw) if mask >> j & 1) in sums
        # horizon score: same statement with the reachable sums (no two-probe shortcut)
        H = int(rng.integers(1, 5)); mh = rng.integers(0, 900, H + 1)
        mask, f = oracle.best_subset(1, G, H, 1.0, 4.0, 0.5, mh, win, lim)
        assert f == max(oracle.f_brh(H, 1.0, 4.0, 0.5, d, mh) for d in sums)


def test_eq2_single_request_argmax_sits_next_to_the_peak():
    """Eq. 2 is concave and piecewise linear in Delta with kinks at the margins m_{g,h}: it rises
    until the slope alpha D - beta sum_{m_h <= Delta} gamma^h turns non-positive and falls after.
    With every such slope well away from zero, the fp64 values at integer lengths are strictly
    ordered on either side of that kink s*, so the best single request is the largest s <= s* or
    the smallest s > s*.  (The CUDA path relies on this for its single-request arg-max.)"""
    rng = np.random.default_rng(53)
    for alpha, beta, gamma in [(1.0, 14.67, 0.64), (1.0, 43.0, 0.86), (1.0, 48.0, 0.9), (2.0, 3.0, 0.5)]:
        for _ in range(60):
            H = int(rng.integers(1, 9))
            m = np.sort(rng.integers(0, 5000, H + 1))[rng.permutation(H + 1)]
            d, D = oracle.discount(H, gamma)
            # the statement needs every segment slope clearly off zero (the library checks the same
            # at br_create and otherwise scans every request): e.g. (2, 3, 0.5) has a flat segment at H = 1
            slopes = [alpha * D - beta * sum(d[h] for h in range(H + 1) if mask >> h & 1)
                      for mask in range(1 << (H + 1))]
            if min(abs(x) for x in slopes) < 1e-9:
                continue
            # s*: smallest kink whose passed weight makes the slope non-positive
            order = np.argsort(m, kind="stable")
            sstar = None
            for i in order:
                w = d[m <= m[i]].sum()
                if alpha * D - beta * w <= 0:
                    sstar = int(m[i]); break
            sizes = [int(x) for x in rng.integers(1, 9000, 40)]
            f = [oracle.f_brh(H, alpha, beta, gamma, s, m) for s in sizes]
            best = max(range(len(sizes)), key=lambda i: (f[i], -i))           # earliest on ties
            below = [i for i in range(len(sizes)) if sstar is None or sizes[i] <= sstar]
            above = [i for i in range(len(sizes)) if sstar is not None and sizes[i] > sstar]
            cand = []
            if below:
                top = max(sizes[i] for i in below); cand.append(min(i for i in below if sizes[i] == top))
            if above:
                low = min(sizes[i] for i in above); cand.append(min(i for i in above if sizes[i] == low))
            pick = max(cand, key=lambda i: (f[i], -i))
            assert pick == best
            # strict order of the fp64 values on either side of the peak
            grid = sorted(set(sizes))
            vals = [oracle.f_brh(H, alpha, beta, gamma, s, m) for s in grid]
            for a_, b_, fa, fb in zip(grid, grid[1:], vals, vals[1:]):
                if sstar is None or b_ <= sstar:
                    assert fb > fa
                elif a_ >= sstar:
                    assert fb < fa


def test_pool_bypass_sends_each_request_where_imbalance_grows_least():
    """Pool-bypass BR-0 (Appendix "Pool-bypass deployment path for BR-0"): each request goes to
    argmax_g F_g(s) on the virtual loads, and F = -Delta I (Section 3.1), so the chosen worker is
    the one whose admission raises I = G max L - sum L the least among the workers below their
    inflight cap (lowest g on ties); loads and inflight counts move before the next request."""
    rng = np.random.default_rng(59)
    for _ in range(40):
        G = int(rng.integers(1, 12)); n = int(rng.integers(1, 30))
        L = rng.integers(0, 3000, G).astype(np.int64)
        infl = rng.integers(0, 4, G).astype(np.int32)
        cap = rng.integers(1, 7, G).astype(np.int32)
        s = rng.integers(1, 1500, n).astype(np.int32)
        got, L_out, n_out = oracle.bypass(G, s, L, infl, cap)
        Lr, nr = L.copy(), infl.copy()
        for i in range(n):
            ok = [g for g in range(G) if nr[g] < cap[g]]
            if not ok:
                assert got[i] == -1
                continue
            def grow(g):
                after = Lr.copy(); after[g] += s[i]
                return oracle.imbalance(after) - oracle.imbalance(Lr)
            want = min(ok, key=lambda g: (grow(g), g))
            assert got[i] == want
            Lr[want] += s[i]; nr[want] += 1
        assert np.array_equal(L_out, Lr) and np.array_equal(n_out, nr)
    # one worker, or everything at its cap
    got, _, _ = oracle.bypass(1, [5, 6], [10], [0], [1])
    assert list(got) == [0, -1]


def test_empirical_survival_estimator_is_the_truncated_expectation():
    """The empirical-survival c_hat is Eq. 3 on the empirical distribution: the two-stage form
    (1 - p_fin) H + p_fin mu_rem (Eqs. 4-5) must equal E[min(o - a, H) | o > a] taken directly over
    the history, in exact rationals; plus the closed forms of a one-point history."""
    from fractions import Fraction
    rng = np.random.default_rng(61)
    for _ in range(60):
        n = int(rng.integers(1, 200)); H = int(rng.integers(1, 17))
        hist = rng.integers(1, 120, n)
        for age in [0, 1, int(rng.integers(0, 130)), int(hist.max()) - 1, int(hist.max()), int(hist.max()) + 5]:
            c, p, mu = oracle.survival(hist, H, age)
            alive = [int(o) for o in hist if o > age]
            inside = [o for o in alive if o <= age + H]
            if not inside:
                assert (c, p, mu) == (float(H), 0.0, float(H))
                # nothing recorded ends inside the window: every survivor contributes the full H
                continue
            want = Fraction(sum(min(o - age, H) for o in alive), len(alive))
            assert abs(Fraction(c) - want) < Fraction(1, 10 ** 12)
            assert abs(Fraction(p) - Fraction(len(inside), len(alive))) < Fraction(1, 10 ** 14)
            assert abs(Fraction(mu) - Fraction(sum(o - age for o in inside), len(inside))) < Fraction(1, 10 ** 12)
            assert 0.0 <= c <= H
    # one recorded length v: inside the window the request surely ends after v - a more steps
    assert oracle.survival([50] * 7, 8, 45) == (5.0, 1.0, 5.0)
    assert oracle.survival([50] * 7, 8, 41)[0] == 8.0 and oracle.survival([50] * 7, 8, 50)[0] == 8.0


# ---------------------------------------------------------------- lifetimes and perfect lookahead
def test_requests_with_lifetimes_run_for_exactly_their_output_length():
    """term_mode 3 (Section 2.2): a request admitted at step x with output length o runs at steps
    x .. x + o - 1, its load growing by one token per step from s_i, and is gone at step x + o."""
    G, B, W = 2, 3, 8
    o = oracle.Instance(G=G, H=0, B=B, W=W, term_mode=3, S_greedy=0)
    base = np.full((G, B), EMPTY, dtype=np.int32)
    base[0, 0] = 40; base[1, 0] = 70                      # two running requests ...
    qs = np.array([11, 22, 33, 0, 0, 0, 0, 0], np.int32)  # ... three waiting ones
    o.set_state(0, 0, base, None, None, None, qs, None, 3)
    end = np.zeros((G, B), np.int32); end[0, 0] = 2; end[1, 0] = 0      # last steps of the running ones
    o.set_lifetimes(end, np.array([1, 3, 5, 0, 0, 0, 0, 0], np.int32))
    seen = {}                                             # (worker, slot) -> loads step by step
    for k in range(8):
        st0 = o.get_state()
        assign, load, _, _ = o.step()
        st1 = o.get_state()
        occ_after_admit = (st1["act_base"] != EMPTY)
        # loads recorded at step k include everything that ran at step k
        running = {}
        for g in range(G):
            for b in range(B):
                was = st0["act_base"][g, b] != EMPTY
                adm = bool((assign == g * B + b).any())
                if was or adm:
                    running[(g, b)] = True
        for key in running:
            seen.setdefault(key, []).append(k)
    # the two initial requests: last steps 2 and 0
    assert seen[(0, 0)] == [0, 1, 2] and seen[(1, 0)] == [0]
    # admissions at step 0 (Stage 1 fills the emptiest worker first; both have two free slots, worker 0
    # is lighter): whatever the placement, each admitted request runs for exactly o steps
    lifetimes = sorted(len(v) for key, v in seen.items() if key not in ((0, 0), (1, 0)))
    assert lifetimes == [1, 3, 5]


def test_lifetime_loads_grow_by_one_token_per_step():
    G, B = 1, 2
    o = oracle.Instance(G=G, H=0, B=B, W=4, term_mode=3)
    base = np.full((G, B), EMPTY, dtype=np.int32); base[0, 0] = 100
    o.set_state(0, 0, base, None, None, None, np.array([7, 0, 0, 0], np.int32), None, 1)
    o.set_lifetimes(np.array([[3, 0]], np.int32), np.array([2, 0, 0, 0], np.int32))
    loads = [int(o.step()[1][0]) for _ in range(6)]
    # step 0: 100 + 7; step 1: 101 + 8 (the admitted request's second and last step); step 2: 102;
    # step 3: 103 (last step of the first request); then nothing runs
    assert loads == [107, 109, 102, 103, 0, 0]


def test_perfect_lookahead_is_min_of_remaining_steps_and_h():
    """pred_mode 1 (Section 5.1 "Our methods", BR-H oracle): c_hat = min(r_i(k), H); with the offset
    convention of the projection a request is counted at offsets h <= c_hat."""
    G, B, H, k = 2, 4, 5, 10
    o = oracle.Instance(G=G, H=H, B=B, W=4, term_mode=3, pred_mode=1, beta=4.0, gamma=0.5)
    base = np.full((G, B), EMPTY, dtype=np.int32)
    base[0, :3] = [100 - k, 200 - k, 300 - k]            # loads 100, 200, 300 at step k
    base[1, :2] = [50 - k, 60 - k]
    o.set_state(k, 0, base, None, None, None, None, None, 0)
    end = np.zeros((G, B), np.int32)
    end[0, :3] = [k, k + 2, k + 40]                       # r = 1, 3, 41
    end[1, :2] = [k + 4, k + 5]                           # r = 5, 6
    o.set_lifetimes(end, np.zeros(4, np.int32))
    o.predict_only(None)
    st = o.get_state()
    assert st["chat"][0, :3].tolist() == [1.0, 3.0, 5.0] and st["chat"][1, :2].tolist() == [5.0, 5.0]
    Lh, Mh, m = o.projection()
    want0 = [100 + 200 + 300, 101 + 201 + 301, 202 + 302, 203 + 303, 304, 305]
    want1 = [110 + h * 2 for h in range(6)]
    assert Lh[0].tolist() == want0 and Lh[1].tolist() == want1
    assert Mh.tolist() == [max(a, b) for a, b in zip(want0, want1)]


def test_arrivals_carry_output_lengths_from_the_table():
    """term_mode 3: arrival j of step k gets out_tab[word j % 4 of Philox block (k, j / 4, 3, 0)]."""
    cfg = wlm.get_config("h80", arrival=("const", 6.0), init_queue=0, init_active=64)
    wl = wlm.make_workload(cfg, n_instances=1)
    o = oracle.instance_from_workload(wl, 0)
    o.set_lifetimes(np.full((cfg.G, cfg.B), 10 ** 6, np.int32), wl.state["wq_o"][0])   # nobody leaves: no admissions
    key = [int(wl.seeds[0]) & 0xFFFFFFFF, int(wl.seeds[0]) >> 32]
    for k in range(5):
        n0 = o.get_state()["wq_n"]
        o.step(None)
        st = o.get_state()
        _, qo = o.get_lifetimes()
        u = _philox_py([k, 0, 0, 0], key)[0]
        n = int((u >= wl.arr_rows_for(0)[0].astype(np.int64)).sum())
        # the workers are full and stay full, so every arrival stays in the queue
        assert st["wq_n"] == n0 + n
        for j in range(n):
            r_len = _philox_py([k, j // 4, 1, 0], key)[j % 4]
            r_out = _philox_py([k, j // 4, 3, 0], key)[j % 4]
            assert st["wq_s"][n0 + j] == wl.len_tab[r_len >> 16]
            assert qo[n0 + j] == wl.out_tab[r_out >> 16]
