"""Hand-built snapshots that pin the rules inside the checker's routing round: the worker order
of both stages, the Stage-2 window, the guard's boundary, the horizon update of an admission and
the subset choice as the round itself makes it.  Every expected value below is worked out by
hand (or by an independent exact restatement in this file) from Algorithms 1 and 2 and
Sections 3.2 / 4.1 / 4.2 -- none comes from the checker."""
import itertools
from fractions import Fraction

import numpy as np
import pytest

import oracle

EMPTY = oracle.EMPTY


def _snapshot(loads, B):
    """act_base [G][B] at k = 0: worker g runs the requests loads[g] in its lowest slots."""
    base = np.full((len(loads), B), EMPTY, dtype=np.int32)
    for g, row in enumerate(loads):
        base[g, :len(row)] = row
    return base


def _route(loads, B, queue, *, H=0, S_greedy=0, R_max=4, chat=None, W=8, **kw):
    G = len(loads)
    o = oracle.Instance(G=G, H=H, B=B, W=W, S_greedy=S_greedy, R_max=R_max, **kw)
    qs = np.zeros(W, dtype=np.int32); qs[:len(queue)] = queue
    ch = np.full((G, B), H, np.float32) if chat is None else np.asarray(chat, np.float32)
    o.set_state(0, 0, _snapshot(loads, B), None, ch, np.zeros((G, B), np.int32), qs, None, len(queue))
    assign, L1 = o.route_only()
    return o, assign, L1


def _worker_of(assign, pos, B):
    return int(assign[pos]) // B


# ---------------------------------------------------------------- Stage 1: worker order
@pytest.mark.parametrize("H", [0, 3])
def test_stage1_takes_the_worker_with_the_most_free_slots(H):
    """Algorithm 1 / 2, Stage 1: g = argmax cap.  Worker 1 has three free slots and by far the
    largest load; the one waiting request still goes there."""
    kw = {} if H == 0 else dict(beta=4.0, gamma=0.5, delta_T=50)
    _, assign, L1 = _route([[10, 10, 10], [500], [20, 20]], 4, [7], H=H, S_greedy=0, **kw)
    assert _worker_of(assign, 0, 4) == 1
    assert L1.tolist() == [30, 507, 40]


@pytest.mark.parametrize("H", [0, 3])
def test_stage1_breaks_equal_free_slots_by_the_smallest_load(H):
    """Algorithm 1 / 2, Stage 1, the tie-break comment of the arg-max line: smallest L_g(k)."""
    kw = {} if H == 0 else dict(beta=4.0, gamma=0.5, delta_T=50)
    _, assign, L1 = _route([[150, 150], [50, 50], [100, 100]], 4, [7], H=H, S_greedy=0, **kw)
    assert _worker_of(assign, 0, 4) == 1
    assert L1.tolist() == [300, 107, 200]
    # and the other way round: the light worker is now worker 2
    _, assign, _ = _route([[150, 150], [100, 100], [50, 50]], 4, [7], H=H, S_greedy=0, **kw)
    assert _worker_of(assign, 0, 4) == 2


# ---------------------------------------------------------------- Stage 2: key order
def test_stage2_pops_the_larger_margin_among_equal_free_slots():
    """Section 3.2: the queue is keyed (cap, m_g) and favours the larger safe margin.  Caps are
    equal; worker 1 has m = 200, worker 0 (the envelope) m = 0.  Popping worker 1 admits the
    request with F = 7 > 0; popping worker 0 first would push it there through the guard."""
    o, assign, L1 = _route([[150, 150], [50, 50], [100, 100]], 4, [7], S_greedy=1 << 20)
    assert _worker_of(assign, 0, 4) == 1
    assert o.get_state()["counters"][4] == 0            # no guard involved
    assert L1.tolist() == [300, 107, 200]


def test_stage2_pops_the_larger_cap_before_the_larger_margin():
    """Section 3.2: cap comes first in the key.  Worker 1 has the most free slots and margin 0
    (it is the envelope); it is popped first, every subset scores below zero, and the guard
    admits the request there."""
    o, assign, L1 = _route([[10, 10, 10], [500], [20, 20]], 4, [7], S_greedy=1 << 20)
    assert _worker_of(assign, 0, 4) == 1
    assert o.get_state()["counters"][4] == 1            # F = 7 - 3 * 7 < 0: guard
    assert L1.tolist() == [30, 507, 40]


def test_stage2_key_of_brh_is_the_horizon_min_margin():
    """Section 4.2 (ii): BR-H keys the queue by min_h m_{g,h}.  H = 2.  Worker 2 is full and its
    requests leave the window after offset 0 (c_hat = 0): loads (200, 0, 0).  Worker 0's requests
    stay (c_hat = H): (100, 102, 104), margins (100, 0, 0).  Worker 1's leave: (120, 0, 0), margins
    (80, 102, 104).  At offset 0 worker 0 has the larger margin, over the horizon worker 1 has (80
    against 0): worker 1 is popped and the request of 10 tokens fits it without penalty.  Popping
    worker 0 would score 17.5 - 4 (5 + 2.5) < 0 and admit it there through the guard."""
    H, B = 2, 4
    o = oracle.Instance(G=3, H=H, B=B, W=8, S_greedy=1 << 20, R_max=4, alpha=1.0, beta=4.0, gamma=0.5,
                        delta_T=50)
    base = _snapshot([[50, 50], [60, 60], [50, 50, 50, 50]], B)
    ch = np.zeros((3, B), np.float32); ch[0, :] = H
    qs = np.zeros(8, np.int32); qs[0] = 10
    o.set_state(0, 0, base, None, ch, np.zeros((3, B), np.int32), qs, None, 1)
    Lh, Mh, m = o.projection()
    assert Lh.tolist() == [[100, 102, 104], [120, 0, 0], [200, 0, 0]]
    assert Mh.tolist() == [200, 102, 104]
    assert m[0].tolist() == [100, 0, 0] and m[1].tolist() == [80, 102, 104]
    assign, L1 = o.route_only()
    assert _worker_of(assign, 0, B) == 1
    assert o.get_state()["counters"][4] == 0
    assert L1.tolist() == [100, 130, 200]


# ---------------------------------------------------------------- Stage 2: window
def test_stage2_window_holds_the_largest_requests():
    """READING (the paper says 'sorted by s_i' without a direction; Stage 1's 'largest waiting
    request' motivates descending): the window is the R_max largest waiting requests.  One worker
    with two free slots and margin 998; R_max = 2.  Largest-first admits 400 and 300
    (F = 700); smallest-first would admit 10 and 20."""
    _, assign, L1 = _route([[1, 1], [250, 250, 250, 250]], 4, [10, 400, 20, 300, 30], S_greedy=1 << 20, R_max=2)
    assert [int(a >= 0) for a in assign[:5]] == [0, 1, 0, 1, 0]
    assert L1.tolist() == [702, 1000]


# ---------------------------------------------------------------- Stage 2: guard boundary
def test_guard_fires_on_a_best_subset_that_scores_exactly_zero():
    """Algorithm 1, starvation-guard line: F_g(Q*) <= 0.  G = 2, m_0 = 50, R_max = 1: the window
    is the request of 100 tokens, F = 100 - 2 (100 - 50) = 0, so the guard takes over and admits
    the single best request of all of R_wait (READING: all of it, not the window): 30 tokens, F = 30."""
    o, assign, L1 = _route([[950], [500, 500]], 2, [100, 30], S_greedy=1 << 20, R_max=1)
    assert assign[0] == -1 and assign[1] == 1           # slot 1 of worker 0
    assert o.get_state()["counters"][4] == 1
    assert L1.tolist() == [980, 1000]


def test_guard_stays_out_on_a_best_subset_that_scores_plus_one():
    """Same snapshot with 99 tokens: F = 99 - 2 * 49 = +1 > 0, the subset is admitted as it is."""
    o, assign, L1 = _route([[950], [500, 500]], 2, [99, 30], S_greedy=1 << 20, R_max=1)
    assert assign[0] == 1 and assign[1] == -1
    assert o.get_state()["counters"][4] == 0
    assert L1.tolist() == [1049, 1000]


def test_guard_boundary_of_the_horizon_score():
    """Algorithm 2 has the same line.  H = 1, gamma = 1, (alpha, beta) = (1, 2), every c_hat = H:
    worker 0 runs one request of 950 -> loads (950, 951); worker 1 is full -> (1000, 1002); margins
    of worker 0: (50, 51).  For D >= 51: F(D) = 2 D - 2 ((D - 50) + (D - 51)) = 202 - 2 D, which is
    0 at D = 101 and +2 at D = 100 (integers: fp64 is exact)."""
    kw = dict(H=1, alpha=1.0, beta=2.0, gamma=1.0, delta_T=50)
    o, assign, L1 = _route([[950], [500, 500]], 2, [101, 30], S_greedy=1 << 20, R_max=1, **kw)
    assert assign[0] == -1 and assign[1] == 1 and o.get_state()["counters"][4] == 1
    assert L1.tolist() == [980, 1000]
    o, assign, L1 = _route([[950], [500, 500]], 2, [100, 30], S_greedy=1 << 20, R_max=1, **kw)
    assert assign[0] == 1 and assign[1] == -1 and o.get_state()["counters"][4] == 0
    assert L1.tolist() == [1050, 1000]


# ---------------------------------------------------------------- BR-H: an admission over the horizon
def test_admission_adds_its_length_at_every_offset_and_moves_the_envelope():
    """Section 4.1: an admitted request counts as a constant s_i at every offset h = 0..H; the
    envelope and all margins follow (Algorithm 2, the update line of both stages)."""
    H, B = 3, 4
    o = oracle.Instance(G=3, H=H, B=B, W=8, S_greedy=0, R_max=4, beta=4.0, gamma=0.5, delta_T=50)
    base = _snapshot([[100, 100, 100, 100], [40], [90, 90, 90, 90]], B)   # only worker 1 has room
    ch = np.full((3, B), H, np.float32)
    qs = np.zeros(8, np.int32); qs[0] = 500
    o.set_state(0, 0, base, None, ch, np.zeros((3, B), np.int32), qs, None, 1)
    L0, M0, m0 = o.projection()
    assert L0.tolist() == [[400, 404, 408, 412], [40, 41, 42, 43], [360, 364, 368, 372]]
    assign, _ = o.route_only()
    assert _worker_of(assign, 0, B) == 1
    L1, M1, m1 = o.round_projection()
    assert L1[1].tolist() == [540, 541, 542, 543]            # + 500 at every offset
    assert L1[0].tolist() == L0[0].tolist() and L1[2].tolist() == L0[2].tolist()
    assert M1.tolist() == [540, 541, 542, 543]               # worker 1 is the new envelope
    assert m1.tolist() == (M1[None] - L1).tolist()
    assert m1[0].tolist() == [140, 137, 134, 131]


def test_later_pop_sees_the_horizon_update_of_an_earlier_admission():
    """The same fact through behaviour.  H = 1, gamma = 1, (alpha, beta) = (1, 8), Stage 2 only,
    R_max = 1, every c_hat = H.  Loads: worker 0 (100, 101) with two free slots, worker 1
    (100, 102) with one, worker 2 full at (400, 403).  Queue 250, 120, 60, 52.
      pop 1: worker 0 (most free slots), margins (300, 302): 250 fits, F = 500 -> admitted;
             worker 0 is now at (350, 351), margins (50, 52)
      pop 2: equal free slots, worker 1 has the larger horizon-min margin (300): 120 fits
      pop 3: worker 0, window {60}: F = 120 - 8 (10 + 8) = -24 <= 0 -> guard -> 52 (F = 104 - 16)
    Had the first admission raised offset 0 only, pop 3 would see margins (50, 302), score
    F(60) = 120 - 80 > 0 and admit the 60."""
    B = 3
    kw = dict(H=1, alpha=1.0, beta=8.0, gamma=1.0, delta_T=50)
    o, assign, L1 = _route([[100], [50, 50], [134, 133, 133]], B, [250, 120, 60, 52],
                           S_greedy=1 << 20, R_max=1, **kw)
    assert assign[:4].tolist() == [0 * B + 1, 1 * B + 2, -1, 0 * B + 2]
    assert L1.tolist() == [402, 220, 400]
    assert o.get_state()["counters"][4] == 1


# ---------------------------------------------------------------- admission: prediction state (reading)
def test_admitted_request_is_anchored_at_h_and_refreshed_at_the_next_step():
    """READING (the refresh rules give no timing for a new request): on admission c_hat = H and
    the refresh age is Delta_T - 1, so the next PREDICT takes its classifier row."""
    H, dT = 4, 3
    o = oracle.Instance(G=1, H=H, B=2, W=4, S_greedy=0, beta=4.0, gamma=0.5, delta_T=dT, gate=0.5)
    base = _snapshot([[10]], 2)
    o.set_state(0, 0, base, None, np.full((1, 2), 2.0, np.float32), np.zeros((1, 2), np.int32),
                np.array([33, 0, 0, 0], np.int32), None, 1)
    assign, _ = o.route_only()
    st = o.get_state()
    assert assign[0] == 1 and st["chat"][0, 1] == float(H) and st["tau"][0, 1] == dT - 1
    probs = np.full((1, 2, H), 0.5, np.float32)              # gate open: c* = 1 + 1/2 + 1/4 + 1/8
    o.predict_only(probs)
    st = o.get_state()
    assert st["chat"][0, 1] == np.float32(1.875) and st["tau"][0, 1] == 0
    assert st["chat"][0, 0] == 1.0 and st["tau"][0, 0] == 1  # the older request only ages


# ---------------------------------------------------------------- Stage 2: the subset choice inside the round
def _exact_score(H, alpha, beta, gamma, delta, m):
    d = [Fraction(gamma) ** h for h in range(H + 1)]
    pen = sum(d[h] * max(0, delta - int(m[h])) for h in range(H + 1))
    return Fraction(alpha) * sum(d) * delta - Fraction(beta) * pen


@pytest.mark.parametrize("H", [0, 2])
def test_stage2_round_equals_an_exact_restatement_on_one_open_worker(H):
    """All workers but one are full, so Stage 2 pops that worker until it is full or the queue is
    empty.  Each pop is restated here in exact rationals: window = the R_max largest (earliest
    first on ties), best subset over all combinations (lowest mask on ties), guard on F <= 0 over
    all of R_wait, loads and envelope updated at every offset."""
    rng = np.random.default_rng(71 + H)
    alpha, beta, gamma = (1.0, None, 1.0) if H == 0 else (1.0, 3.0, 0.5)
    for _ in range(250):
        G = int(rng.integers(2, 6)); B = int(rng.integers(2, 7)); W = 12
        R_max = int(rng.integers(1, 5))
        g_open = int(rng.integers(0, G)); n_open = int(rng.integers(0, B))
        loads = [list(rng.integers(1, 200, B)) for _ in range(G)]
        loads[g_open] = list(rng.integers(1, 200, n_open))
        nq = int(rng.integers(1, 9)); queue = [int(x) for x in rng.integers(1, 250, nq)]
        kw = {} if H == 0 else dict(alpha=alpha, beta=beta, gamma=gamma, delta_T=50)
        o, assign, L1 = _route(loads, B, queue, H=H, S_greedy=1 << 20, R_max=R_max, W=W, **kw)
        # exact restatement; every c_hat = H, so L_g(k+h) = L_g + h n_g
        b_eff = float(G) if H == 0 else beta
        Lh = np.array([[sum(r) + h * len(r) for h in range(H + 1)] for r in loads], dtype=np.int64)
        cap = B - n_open
        waiting = list(range(nq)); expect = {}
        slot = n_open
        while cap > 0 and waiting:
            Mh = Lh.max(0); m = Mh - Lh[g_open]
            win = sorted(waiting, key=lambda i: (-queue[i], i))[:R_max]
            best = None
            for r in range(1, min(cap, R_max, len(win)) + 1):
                for comb in itertools.combinations(range(len(win)), r):
                    f = _exact_score(H, alpha, b_eff, gamma, sum(queue[win[j]] for j in comb), m)
                    mk = sum(1 << j for j in comb)
                    if best is None or f > best[0] or (f == best[0] and mk < best[1]):
                        best = (f, mk)
            if best[0] <= 0:
                pick = max(waiting, key=lambda i: (_exact_score(H, alpha, b_eff, gamma, queue[i], m), -i))
                chosen = [pick]
            else:
                chosen = [win[j] for j in range(len(win)) if best[1] >> j & 1]
            for i in chosen:
                expect[i] = g_open * B + slot; slot += 1; cap -= 1
                Lh[g_open] += queue[i]
                waiting.remove(i)
        got = {i: int(assign[i]) for i in range(nq) if assign[i] >= 0}
        assert got == expect
