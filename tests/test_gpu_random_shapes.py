"""Seeded random fleets, queues, horizons, predictors, termination models, window sizes, stage
splits, refresh rules, thread counts and launch shapes through the routing step, every step and
every snapshot compared with the checker (run_parity).  Shapes the library refuses at br_create
(outside its compiled limits or range proofs) are skipped; the run must still cover most draws."""
import numpy as np
import pytest

from paper_2605_06113_b200 import workload as wlm
from paper_2605_06113_b200.binding import BrError
from helpers import run_parity

pytestmark = pytest.mark.gpu


def _draw(rng):
    G = int(rng.choice([1, 2, 3, 5, 8, 16, 31, 32, 33, 47, 64]))
    B = int(rng.choice([8, 16, 24, 40, 64, 72, 128]))
    if G * B > 8192:
        B = 64
    W = int(rng.choice([4, 20, 36, 100, 128, 256, 512, 1000, 1024, 2048]))
    H = int(rng.choice([0, 0, 1, 2, 3, 4, 5, 8, 11, 16, 17, 33, 80]))
    term_mode = int(rng.choice([0, 1, 1, 2, 3])) if H > 0 else int(rng.choice([0, 1, 1, 3]))
    pred_mode = int(rng.choice([0, 1])) if (H > 0 and term_mode == 3) else 0
    R_max = int(rng.choice([1, 2, 3, 4, 4, 5, 6, 9, 12, 16]))
    if H > 16 and R_max > 5:
        R_max = 4
    ab = [(2.0, 50.0), (0.5, 2.0), (1.0, 8.0)][int(rng.integers(0, 3))]
    kw = dict(G=G, B=B, W=W, H=H, init_active=int(rng.integers(0, B + 1)), init_queue=int(rng.integers(0, W + 1)),
              hazard=float(rng.choice([0.002, 0.02, 0.1, 0.3])), term_mode=term_mode, pred_mode=pred_mode,
              arrival=("const", float(rng.choice([0.2, 1.0, 3.0, 8.0, 20.0]))), R_max=R_max,
              S_greedy=int(rng.choice([-1, 0, 4, 16, 1 << 20])), score_mode=int(rng.choice([-1, -1, 1])),
              delta_T=int(rng.choice([-1, 1, 2, 3, 7])), gate=float(rng.choice([0.0, 0.1, 0.3, 0.5])),
              c_floor=float(rng.choice([1.0, 1.0, 2.5])), beta_ab=ab,
              beta=float(rng.choice([14.67, 48.0, 1.0, 3.0])), gamma=float(rng.choice([0.64, 0.9, 1.0])),
              burst_every=int(rng.choice([0, 0, 3, 7])), burst_size=int(rng.choice([5, 50, 300])),
              out_mu=float(rng.choice([2.0, 4.0, 6.5])))
    threads = int(rng.choice([0, 0, 32, 64, 96, 128, 256]))
    n_inst = int(rng.choice([1, 2, 3, 5, 8]))
    ls = int(rng.choice([1, 1, 2, 3, 5]))
    return kw, threads, n_inst, ls, ls * int(rng.integers(3, 9)), bool(rng.random() < 0.15)


@pytest.mark.parametrize("block", range(4))
def test_random_shapes(block):
    ran = 0
    for case in range(60):
        kw, threads, n_inst, ls, steps, graph = _draw(np.random.default_rng(7000 + 100 * block + case))
        try:
            run_parity(wlm.get_config("c0", **kw), n_inst, steps, threads=threads, launch_steps=ls, check_every=1,
                       graph=graph)
            ran += 1
        except BrError as e:
            assert "br_create" in str(e), (block, case, kw)
    assert ran >= 40
