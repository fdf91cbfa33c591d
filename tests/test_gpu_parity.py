"""CUDA library against the CPU checker, element by element, through the C ABI."""
import numpy as np
import pytest

from paper_2605_06113_b200 import workload as wlm
from helpers import run_parity

pytestmark = pytest.mark.gpu


def test_c0_br0_full_run():
    run_parity(wlm.get_config("c0"), 1, 300, check_every=10, fscore=True)


@pytest.mark.parametrize("threads", [32, 64, 256])
def test_c1_br0_thread_shapes(threads):
    run_parity(wlm.get_config("c1"), 1, 150, threads=threads, check_every=25)


def test_c1_br0_full_run():
    run_parity(wlm.get_config("c1"), 1, 2000, check_every=100)


def test_c2_brh_full_run():
    run_parity(wlm.get_config("c2"), 1, 2000, check_every=100)


def test_c2_brh_fscore_matrix():
    run_parity(wlm.get_config("c2"), 1, 60, check_every=10, fscore=True)


def test_c2_brh_open_gate_every_step():
    # the probability path exercised at scale: gate open for everyone, refresh every step
    run_parity(wlm.get_config("c2", gate=0.0, delta_T=1), 2, 300, check_every=20)


def test_c2_brh_low_gate_period_two():
    run_parity(wlm.get_config("c2", gate=0.12, delta_T=2, beta=43.0, gamma=0.86), 2, 300, check_every=20)


def test_c3_br0_batched_slice():
    run_parity(wlm.get_config("c3"), 6, 200, check_every=20)


def test_c4_brh_batched_slice():
    run_parity(wlm.get_config("c4"), 3, 260, check_every=20)


def test_c4_brh_hazard_informative_probs():
    # classifier output that is confident for some requests: gate opens request by request
    run_parity(wlm.get_config("c4", beta_ab=(0.5, 2.0), gate=0.5, term_mode=2), 2, 80, check_every=10)


@pytest.mark.parametrize("S_greedy", [0, 16, 1 << 20])
def test_stage_split_sweep(S_greedy):
    # 0: Stage 1 admits everything; huge: Stage 2 only
    run_parity(wlm.get_config("c1", S_greedy=S_greedy), 1, 120, check_every=20)


@pytest.mark.parametrize("R_max", [1, 2, 5])
def test_window_sizes(R_max):
    run_parity(wlm.get_config("c1", R_max=R_max), 1, 120, check_every=20)


def test_brh_code_path_at_h0_matches_br0():
    cfg = wlm.get_config("c1")
    a = run_parity(cfg, 1, 200, check_every=50)
    b = run_parity(wlm.get_config("c1", score_mode=1, alpha=1.0, beta=float(cfg.G), gamma=0.64), 1, 200,
                   check_every=50)
    assert np.array_equal(a, b)


def test_multi_step_launch_and_graph_replay():
    run_parity(wlm.get_config("c1"), 2, 120, launch_steps=8, check_every=1)
    run_parity(wlm.get_config("c2"), 1, 96, launch_steps=4, check_every=1)
    run_parity(wlm.get_config("c1"), 1, 100, graph=True, check_every=10)
    run_parity(wlm.get_config("c2"), 1, 100, graph=True, check_every=10)


def test_ragged_shapes():
    # odd worker counts, B not a multiple of 32 or 64, tiny, odd and maximal queue capacities
    for G, B, W, H in [(1, 8, 4, 0), (3, 24, 20, 0), (5, 16, 36, 3), (7, 40, 100, 2), (64, 8, 64, 16),
                       (33, 72, 200, 5), (2, 256, 4096, 1)]:
        cfg = wlm.get_config("c0", G=G, B=B, W=W, H=H, init_active=B // 2, init_queue=W // 2,
                             hazard=0.05, term_mode=1, arrival=("const", 3.0), S_greedy=-1,
                             score_mode=-1, delta_T=-1, gate=0.1)
        run_parity(cfg, 3, 80, check_every=10)


def test_empty_and_saturated_edges():
    # nothing waiting and nothing arriving; then full workers with a full queue and no terminations
    cfg = wlm.get_config("c0", init_queue=0, arrival=("const", 1e-9))
    run_parity(cfg, 1, 20)
    cfg = wlm.get_config("c1", term_mode=0, hazard=0.0)
    run_parity(cfg, 1, 20)
    # empty fleet, long queue: first step admits min(S_tot, n_w)
    cfg = wlm.get_config("c1", init_active=0)
    run_parity(cfg, 1, 10)


# ---- the one-warp-per-instance BR-0 kernel (G <= 32, B <= 64, W <= 256; threads=32 selects it) ----
def test_small_fleet_c3_slice_full_length():
    run_parity(wlm.get_config("c3"), 8, 500, threads=32, check_every=50)


def test_small_fleet_c0_full_run():
    run_parity(wlm.get_config("c0"), 1, 300, threads=32, check_every=25)


@pytest.mark.parametrize("kw", [dict(R_max=1), dict(R_max=2), dict(R_max=5), dict(S_greedy=0),
                                dict(S_greedy=16), dict(S_greedy=1 << 20)])
def test_small_fleet_window_and_stage_split(kw):
    run_parity(wlm.get_config("c3", **kw), 4, 260, threads=32, check_every=20)


def test_small_fleet_multi_step_and_graph():
    run_parity(wlm.get_config("c3"), 5, 240, threads=32, launch_steps=8, check_every=1)
    run_parity(wlm.get_config("c3"), 2, 100, threads=32, graph=True, check_every=10)


def test_small_fleet_ragged_and_busy_shapes():
    # odd worker counts and slot counts, queues that are not a multiple of 128, a hazard high
    # enough that several requests of a worker end in one step (some at the step they were
    # admitted), arrival rates that overflow the queue
    for G, B, W, lam, hz in [(1, 8, 4, 3.0, 0.05), (5, 16, 36, 3.0, 0.05), (7, 40, 100, 6.0, 0.2),
                             (32, 64, 256, 30.0, 0.3), (31, 56, 252, 12.0, 0.02), (32, 8, 128, 40.0, 0.5)]:
        cfg = wlm.get_config("c3", G=G, B=B, W=W, init_active=B // 2, init_queue=W // 2, hazard=hz,
                             arrival=("const", lam), S_greedy=-1)
        run_parity(cfg, 3, 120, threads=32, check_every=10)


def test_brh_flat_slope_takes_the_full_scan():
    # alpha D = beta (d_0 + d_1): one segment of Eq. 2 is flat, scores tie across lengths, and the
    # single-request arg-max must scan every request (earliest arrival among equal scores)
    run_parity(wlm.get_config("c2", H=1, alpha=1.0, beta=1.0, gamma=1.0, gate=0.0, delta_T=1), 2, 150,
               check_every=25)
    run_parity(wlm.get_config("c4", H=2, alpha=1.0, beta=1.0, gamma=1.0), 1, 60, check_every=20)


@pytest.mark.parametrize("name,n_inst", [("c3", 600), ("c3", 2100), ("c2", 520)])
def test_host_buffer_step_in_chunks_matches_device_step(name, n_inst):
    """br_step_host on batches large enough to go through in chunks of instances (uploads, kernels
    and downloads of different chunks overlap on three streams): state and outputs must equal those
    of br_step on device buffers, for three steps in a row."""
    import torch
    from paper_2605_06113_b200.binding import Router, state_to_numpy
    cfg = wlm.get_config(name)
    wl = wlm.make_workload(cfg, n_instances=n_inst)
    r = Router(wl, device="cuda:0")
    st_h = {k: np.ascontiguousarray(v).copy() for k, v in wl.state.items()}
    out_h = {k: v.numpy() for k, v in r.outputs(n_inst, device="cpu").items()}
    st_d = r.device_state()
    out_d = r.outputs(n_inst)
    for k in range(3):
        probs = np.ascontiguousarray(wlm.term_probs_np(wl, k)) if cfg.H > 0 else None
        r.step_host(st_h, out_h, probs)
        r.step(st_d, out_d, None if probs is None else torch.from_numpy(probs).cuda())
        torch.cuda.synchronize()
        for key in out_h:
            assert np.array_equal(out_h[key], out_d[key].cpu().numpy()), (name, k, key)
        ref = state_to_numpy(st_d)
        for key in st_h:
            assert np.array_equal(st_h[key], ref[key]), (name, k, key)
    r.close()


@pytest.mark.parametrize("name", ["c3", "c2"])
def test_row_offset_batches(name):
    """first_instance selects a range of rows of every array, state and outputs alike: stepping
    rows [5, 12) of a 16-row allocation must leave the other rows untouched and give what a
    7-instance batch of the same seeds gives."""
    import torch
    from paper_2605_06113_b200.binding import Router, state_to_numpy
    cfg = wlm.get_config(name)
    wl = wlm.make_workload(cfg, n_instances=16)
    r = Router(wl, device="cuda:0", threads=32 if name == "c3" else 0)
    st = r.device_state(); out = r.outputs(16)
    for v in out.values():
        v.fill_(-9)
    wl7 = wlm.make_workload(cfg, n_instances=7, first_instance=5)
    r7 = Router(wl7, device="cuda:0", threads=32 if name == "c3" else 0)
    st7 = r7.device_state(); out7 = r7.outputs(7)
    before = state_to_numpy({k: v.clone() for k, v in st.items()})
    for k in range(3):
        probs16 = probs7 = None
        if cfg.H > 0:
            probs16 = torch.from_numpy(wlm.term_probs_np(wl, k)).cuda()
            probs7 = torch.from_numpy(wlm.term_probs_np(wl7, k)).cuda()
        r.step(st, out, probs16, N=7, first=5)
        r7.step(st7, out7, probs7)
        torch.cuda.synchronize()
        for key in out7:
            assert torch.equal(out[key][0, 5:12], out7[key][0]), (name, k, key)
            assert bool((out[key][0, :5] == -9).all()) and bool((out[key][0, 12:] == -9).all()), (name, k, key)
    after = state_to_numpy(st); ref = state_to_numpy(st7)
    for key in after:
        if key == "seed":
            continue
        assert np.array_equal(after[key][5:12], ref[key]), key
        assert np.array_equal(after[key][:5], before[key][:5]) and np.array_equal(after[key][12:], before[key][12:]), key
    r.close(); r7.close()


def test_small_fleet_random_shapes():
    """Thirty seeded random fleet shapes inside the small-fleet kernel's range (G <= 32, B <= 64,
    W <= 512) with random window sizes, stage splits, hazards and arrival rates."""
    rng = np.random.default_rng(2024)
    for case in range(30):
        G = int(rng.integers(1, 33)); B = 8 * int(rng.integers(1, 9)); W = 4 * int(rng.integers(1, 129))
        cfg = wlm.get_config("c3", G=G, B=B, W=W, R_max=int(rng.integers(1, 6)),
                             S_greedy=int(rng.choice([-1, 0, 3, G, 4 * G, 1 << 20])),
                             init_active=int(rng.integers(0, B + 1)), init_queue=int(rng.integers(0, W + 1)),
                             hazard=float(rng.choice([0.0, 0.002, 0.05, 0.3, 1.0])),
                             arrival=("const", float(rng.choice([0.01, 1.0, 5.0, 20.0, 45.0]))),
                             first_seed=1000 * case)
        run_parity(cfg, 2, 50, threads=32, check_every=10, launch_steps=int(rng.choice([1, 1, 5])))


def test_brh_random_shapes():
    """Seeded random BR-H shapes (H up to 16, G up to 64, ragged B and W), open and closed gates,
    both termination modes."""
    rng = np.random.default_rng(4048)
    for case in range(14):
        G = int(rng.integers(1, 65)); B = 8 * int(rng.integers(1, 13)); W = 4 * int(rng.integers(1, 151))
        H = int(rng.integers(1, 17))
        cfg = wlm.get_config("c2", G=G, B=B, W=W, H=H, R_max=int(rng.integers(1, 6)),
                             S_greedy=int(rng.choice([-1, 0, G, 1 << 20])), delta_T=int(rng.choice([-1, 1, 2, 5])),
                             gate=float(rng.choice([0.0, 0.1, 0.5])), beta=float(rng.choice([3.0, 14.67, 43.0])),
                             gamma=float(rng.choice([0.5, 0.64, 0.9, 1.0])),
                             init_active=int(rng.integers(0, B + 1)), init_queue=int(rng.integers(0, W + 1)),
                             term_mode=int(rng.choice([1, 2])), hazard=float(rng.choice([0.002, 0.05, 0.3])),
                             beta_ab=(2.0, float(rng.choice([4.0, 20.0, 50.0]))),
                             arrival=("const", float(rng.choice([1.0, 8.0, 30.0]))), first_seed=5000 * case)
        run_parity(cfg, 2, 40, threads=int(rng.choice([0, 32, 64, 128])), check_every=10,
                   launch_steps=int(rng.choice([1, 1, 4])))


@pytest.mark.parametrize("H,G,kw", [
    (80, 8, dict(beta=48.0, gamma=0.9, W=256, init_queue=256)),                       # the paper's deployed lookahead and fleet
    (80, 16, dict(gate=0.0, delta_T=1)),                              # every request refreshed every step
    (40, 64, dict(B=32, init_active=30, W=400, init_queue=390, term_mode=1, hazard=0.01, gate=0.3)),  # two workers per router lane
    (17, 5, dict(B=16, init_active=9, W=64, init_queue=40, S_greedy=0)),                           # just beyond the register-resident horizons
])
def test_long_horizons(H, G, kw):
    """Horizons beyond 16 offsets keep projected loads, envelope and margins in shared memory."""
    run_parity(wlm.get_config("c2", H=H, G=G, **kw), 2, 60, check_every=10, fscore=(G == 8))


def test_long_horizon_multi_step_and_random_shapes():
    rng = np.random.default_rng(808)
    for case in range(6):
        G = int(rng.integers(1, 65)); B = 8 * int(rng.integers(1, 9)); W = 4 * int(rng.integers(1, 100))
        H = int(rng.integers(17, 81))
        cfg = wlm.get_config("c2", G=G, B=B, W=W, H=H, R_max=int(rng.integers(1, 6)),
                             S_greedy=int(rng.choice([-1, 0, G, 1 << 20])), delta_T=int(rng.choice([-1, 1, 7])),
                             gate=float(rng.choice([0.0, 0.5, 0.9])), beta=float(rng.choice([1.0, 24.0, 96.0])),
                             gamma=float(rng.choice([0.5, 0.9, 1.0])),
                             init_active=int(rng.integers(0, B + 1)), init_queue=int(rng.integers(0, W + 1)),
                             term_mode=int(rng.choice([1, 2])), hazard=float(rng.choice([0.002, 0.05])),
                             beta_ab=(2.0, float(rng.choice([20.0, 50.0, 200.0]))),
                             arrival=("const", float(rng.choice([1.0, 8.0]))), first_seed=7000 * case)
        run_parity(cfg, 2, 30, threads=int(rng.choice([0, 32, 128])), check_every=10,
                   launch_steps=int(rng.choice([1, 3])))


@pytest.mark.parametrize("name,R_max,kw", [("c1", 6, {}), ("c1", 16, dict(S_greedy=1 << 20)), ("c2", 9, {}),
                                           ("c2", 16, dict(gate=0.0, delta_T=1, S_greedy=1 << 20)),
                                           ("c4", 12, {}), ("c3", 7, dict(hazard=0.05))])
def test_large_stage2_windows(name, R_max, kw):
    """Windows of 6 to 16 requests: Stage 2 picks its subset by meeting in the middle."""
    run_parity(wlm.get_config(name, R_max=R_max, **kw), 2, 60, check_every=10)


def test_large_stage2_windows_random_shapes():
    rng = np.random.default_rng(1616)
    for case in range(8):
        G = int(rng.integers(2, 65)); B = 8 * int(rng.integers(1, 9)); W = 4 * int(rng.integers(2, 100))
        H = int(rng.choice([0, 0, 3, 8, 16]))
        cfg = wlm.get_config("c2" if H else "c1", G=G, B=B, W=W, H=H, R_max=int(rng.integers(6, 17)),
                             S_greedy=int(rng.choice([-1, 0, 1 << 20])), hazard=float(rng.choice([0.02, 0.2])),
                             term_mode=1, init_active=int(rng.integers(0, B + 1)), init_queue=int(rng.integers(0, W + 1)),
                             arrival=("const", float(rng.choice([2.0, 12.0]))), first_seed=3100 * case)
        run_parity(cfg, 2, 30, threads=int(rng.choice([0, 32, 128])), check_every=10,
                   launch_steps=int(rng.choice([1, 4])))


def test_long_horizon_large_fleet_needs_more_than_48k_of_shared_memory():
    """H = 80 on G = 64 workers with 1,024 waiting requests: about 60 KB of shared memory per instance,
    beyond the default limit, so the kernel is opted in at launch."""
    run_parity(wlm.get_config("c4", H=80, term_mode=1, gate=0.3, beta=48.0, gamma=0.9), 2, 12, check_every=4)
    run_parity(wlm.get_config("h80", G=64, W=1024, init_queue=1000, arrival=("const", 5.0)), 2, 12, check_every=4,
               threads=256)
    run_parity(wlm.get_config("h80", G=64, W=1024, init_queue=1000, arrival=("const", 5.0)), 1, 8, check_every=4,
               graph=True)                             # the opt-in also happens while a graph is captured


def test_more_requests_end_in_a_step_than_the_lists_hold():
    # single-warp BR-H instances resolve the step's terminations before routing; with hundreds of
    # requests ending at once the surplus must still count in that step's projection
    for kw, threads, n, ls in [
            (dict(G=47, B=72, W=36, H=8, init_active=42, init_queue=21, hazard=0.1, delta_T=7, gate=0.1, S_greedy=0,
                  arrival=("const", 20.0)), 32, 3, 2),
            (dict(G=32, B=72, W=256, H=16, init_active=48, init_queue=159, hazard=0.3, delta_T=2, gate=0.3,
                  S_greedy=16, gamma=0.9, arrival=("const", 8.0)), 32, 8, 1),
            (dict(G=8, B=64, W=1000, H=80, init_active=49, init_queue=737, hazard=0.3, delta_T=2, gate=0.3,
                  S_greedy=0, beta=3.0, gamma=1.0, beta_ab=(1.0, 8.0), arrival=("const", 1.0)), 0, 5, 5),
            (dict(G=32, B=64, W=256, H=0, init_active=60, init_queue=200, hazard=0.3, arrival=("const", 20.0)), 32, 4, 3)]:
        cfg = wlm.get_config("c0", term_mode=1, score_mode=-1, **kw)
        run_parity(cfg, n, 6 * ls, threads=threads, launch_steps=ls, check_every=1)
