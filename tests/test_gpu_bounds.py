"""The range-checked build of the library (libbr_dbg.so, -DBR_BOUNDS): ragged, random and edge shapes
of both step kernels run through it with every index into a per-instance array checked; the run
must match the CPU checker as usual and the count of out-of-range indexes must stay at zero.  The
counter itself is shown to count by the library's self-test, which indexes a four-element span
out of range three times (into a sink: nothing outside the array is touched)."""
import numpy as np
import pytest
import torch

from paper_2605_06113_b200 import binding, build, workload as wlm
from helpers import run_parity

pytestmark = pytest.mark.gpu


@pytest.fixture()
def checked_library():
    path = build.build_debug()
    binding.use_library(path)
    assert binding.lib().br_debug_bounds_hits() >= 0          # this is the checked build
    yield binding.lib()
    binding.use_library(None)


def test_normal_build_has_no_range_checks():
    binding.use_library(None)
    assert binding.lib().br_debug_bounds_hits() == -1


def test_counter_counts(checked_library):
    four = torch.zeros(4, dtype=torch.int32, device="cuda")
    before = checked_library.br_debug_bounds_hits()
    assert checked_library.br_debug_bounds_selftest(four.data_ptr()) == 3
    assert four.tolist() == [0, 0, 0, 7]                      # only the in-range write arrived
    assert checked_library.br_debug_bounds_hits() == before + 3


def test_ragged_and_random_shapes_stay_in_range(checked_library):
    L = checked_library
    start = L.br_debug_bounds_hits()
    rng = np.random.default_rng(77)
    # small-fleet kernel (one warp per instance)
    for case in range(8):
        G = int(rng.integers(1, 33)); B = 8 * int(rng.integers(1, 9)); W = 4 * int(rng.integers(1, 129))
        cfg = wlm.get_config("c3", G=G, B=B, W=W, R_max=int(rng.integers(1, 6)),
                             S_greedy=int(rng.choice([-1, 0, G, 1 << 20])),
                             init_active=int(rng.integers(0, B + 1)), init_queue=int(rng.integers(0, W + 1)),
                             hazard=float(rng.choice([0.0, 0.05, 1.0])),
                             arrival=("const", float(rng.choice([0.01, 5.0, 45.0]))), first_seed=900 * case)
        run_parity(cfg, 3, 25, threads=32, check_every=5, launch_steps=int(rng.choice([1, 5])))
    # general kernel: BR-H, ragged sizes, both register- and shared-memory horizons, large windows, lifetimes
    for case in range(8):
        G = int(rng.integers(1, 65)); B = 8 * int(rng.integers(1, 10)); W = 4 * int(rng.integers(1, 120))
        H = int(rng.choice([1, 4, 8, 16, 17, 40, 80]))
        big = H <= 16 and G >= 2 and case % 2 == 0
        cfg = wlm.get_config("c2", G=G, B=B, W=W, H=H, R_max=int(rng.integers(6, 17)) if big else int(rng.integers(1, 6)),
                             S_greedy=int(rng.choice([-1, 0, 1 << 20])), delta_T=int(rng.choice([-1, 1, 5])),
                             gate=float(rng.choice([0.0, 0.5])), init_active=int(rng.integers(0, B + 1)),
                             init_queue=int(rng.integers(0, W + 1)), term_mode=int(rng.choice([1, 2, 3])),
                             hazard=0.05, out_mu=2.0, arrival=("const", float(rng.choice([1.0, 20.0]))),
                             first_seed=1300 * case)
        run_parity(cfg, 2, 20, threads=int(rng.choice([0, 32, 96, 256])), check_every=5,
                   launch_steps=int(rng.choice([1, 3])))
    # the five configurations' own shapes, a few steps each, and the deployed H = 80 setting
    for name, n in (("c0", 1), ("c1", 1), ("c2", 1), ("c3", 5), ("c4", 2), ("h80", 2)):
        run_parity(wlm.get_config(name), n, 12, check_every=4)
    run_parity(wlm.get_config("c1", G=40, W=1024, init_queue=1000), 2, 10, check_every=5)     # BR-0 on the general kernel
    assert L.br_debug_bounds_hits() == start
