"""The multi-process path of the benchmark (instances sharded over ranks, no data-path
collective, max-over-ranks timing) exercised with two gloo ranks on CPU."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    import oracle
    from paper_2605_06113_b200 import workload as wlm
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # each rank owns its own instance range: disjoint seeds, identical shapes
    first, n = bench.shard_of(rank, world, instances_per_rank=3, sets=2)
    cfg = wlm.get_config("c3")
    wl = wlm.make_workload(cfg, n_instances=n, first_instance=first)
    o = oracle.instance_from_workload(wl, 0)
    tr = np.array([o.step()[2] for _ in range(3)])
    ms = bench.max_over_ranks(10.0 * (rank + 1), dist, device="cpu")
    dist.barrier()
    q.put((rank, first, n, [int(s) for s in wl.seeds], tr.tolist(), ms))
    dist.destroy_process_group()


def test_two_ranks_shard_instances_and_take_the_slowest_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=240) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    (r0, f0, n0, s0, t0, ms0), (r1, f1, n1, s1, t1, ms1) = res
    assert n0 == n1 == 6 and f0 == 0 and f1 == 6
    assert not set(s0) & set(s1)                      # no instance is simulated twice
    assert t0 != t1                                   # different seeds, different traces
    assert ms0 == ms1 == 20.0                         # max over ranks
