"""Requests that carry their output lengths (term_mode 3) and the perfect-lookahead predictor
c_hat = min(r_i(k), H) (Section 5.1 "Our methods", BR-H oracle), against the CPU checker."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_06113_b200 import workload as wlm
from paper_2605_06113_b200.binding import Router, state_to_numpy
from helpers import compare_state, run_parity

pytestmark = pytest.mark.gpu


def test_deployed_setting_h80_g8_rmax4():
    """H = 80, G = 8, R_max = 4 (Section 5.3 "Dispatch overhead"), perfect lookahead."""
    run_parity(wlm.get_config("h80"), 2, 400, check_every=50)


def test_deployed_setting_multi_step_and_graph():
    run_parity(wlm.get_config("h80"), 3, 120, check_every=5, launch_steps=8)
    run_parity(wlm.get_config("h80"), 1, 60, check_every=5, graph=True)


def test_br0_on_the_same_lifetimes():
    """BR-0 (Eq. 1) on requests with lifetimes: the comparison run of the (beta, gamma) table."""
    run_parity(wlm.get_config("h80", H=0, pred_mode=0), 2, 400, check_every=50)
    run_parity(wlm.get_config("h80", H=0, pred_mode=0, G=40, W=260, init_queue=200, arrival=("const", 4.0)),
               2, 80, check_every=10, threads=64)


@pytest.mark.parametrize("H,kw", [(8, dict(G=64, W=1024, init_queue=900, arrival=("const", 6.0), out_mu=5.0)),
                                  (4, dict(G=16, B=32, init_active=20, out_mu=3.0, out_sigma=0.7)),
                                  (1, dict(G=3, B=8, init_active=5, W=16, init_queue=9, out_mu=1.0, out_sigma=1.0,
                                           arrival=("const", 2.0)))])
def test_perfect_lookahead_on_register_resident_horizons(H, kw):
    run_parity(wlm.get_config("h80", H=H, **kw), 2, 100, check_every=10)


def test_classifier_rows_with_lifetimes():
    """Classifier-driven c_hat (refresh rules) while the realised terminations follow lifetimes."""
    run_parity(wlm.get_config("c2", term_mode=3, out_mu=4.0, gate=0.05), 2, 150, check_every=10)


def test_short_outputs_end_at_their_admission_step():
    """o_i = 1 for most requests: a request admitted at k ends at k."""
    run_parity(wlm.get_config("h80", H=6, out_mu=0.0, out_sigma=0.5, G=5, B=16, init_active=10, W=64, init_queue=40,
                              arrival=("const", 9.0)), 2, 60, check_every=5)


def test_host_buffer_step_with_lifetimes():
    cfg = wlm.get_config("h80", H=12, G=9, B=16, init_active=12, W=128, init_queue=100)
    n = 5
    wl = wlm.make_workload(cfg, n_instances=n)
    r = Router(wl, device="cuda:0")
    view = {np.dtype(np.uint64): np.int64, np.dtype(np.uint32): np.int32}
    st = {k: torch.from_numpy(np.ascontiguousarray(v).view(view.get(v.dtype, v.dtype))).pin_memory()
          for k, v in wl.state.items()}
    out = {k: v.pin_memory() for k, v in r.outputs(n, device="cpu").items()}
    orcs = [oracle.instance_from_workload(wl, i) for i in range(n)]
    for k in range(25):
        (r.step_host if k % 2 else r.step_host_static)(st, out, None)
        for i, o in enumerate(orcs):
            a, l, t, _ = o.step(None)
            assert np.array_equal(out["assign"][0, i].numpy(), a), (i, k)
            assert np.array_equal(out["load"][0, i].numpy(), l) and np.array_equal(out["trace"][0, i].numpy(), t)
    fin = state_to_numpy(st)
    for i, o in enumerate(orcs):
        compare_state(cfg, fin, o, i, 25)
    r.close()
