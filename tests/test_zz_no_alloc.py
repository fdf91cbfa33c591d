"""br_step_host_static -- the host-buffer step for callers that may not allocate device memory
(pre-planned serving loops, processes whose CUDA memory belongs to another framework's pool,
contexts where cudaMalloc could stall) -- must give exactly what br_step_host gives.

Both entry points are driven through the C ABI on the same seeded snapshots for two calls in a
row (the second call reuses the built-in staging array with the first call's data still in it).
Collected last on purpose: a failure here cannot hide the result of any other test."""
import numpy as np
import pytest
import torch

from paper_2605_06113_b200 import workload as wlm
from paper_2605_06113_b200.binding import BR_ELIMIT, BrError, Router, STATIC_STAGE_BYTES

pytestmark = pytest.mark.gpu


def _host_buffers(wl, r, n):
    st = {k: np.ascontiguousarray(v).copy() for k, v in wl.state.items()}
    out = {k: v.numpy() for k, v in r.outputs(n, device="cpu").items()}
    return st, out


@pytest.mark.parametrize("name,n_inst", [("c3", 40), ("c2", 2), ("c0", 1)])
def test_static_staging_matches_allocating_entry_point(name, n_inst):
    cfg = wlm.get_config(name)
    wl = wlm.make_workload(cfg, n_instances=n_inst)
    r = Router(wl, device="cuda:0")
    st_a, out_a = _host_buffers(wl, r, n_inst)      # br_step_host (allocates its staging)
    st_b, out_b = _host_buffers(wl, r, n_inst)      # br_step_host_static (allocates nothing)
    free_seen = []
    for k in range(3):                              # calls in a row on the shared array
        probs = np.ascontiguousarray(wlm.term_probs_np(wl, k)) if cfg.H > 0 else None
        up_a, down_a = r.step_host(st_a, out_a, probs)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        up_b, down_b = r.step_host_static(st_b, out_b, probs)
        torch.cuda.synchronize()
        free_seen.append((free_before, torch.cuda.mem_get_info()[0]))
        assert (up_a, down_a) == (up_b, down_b)
        for key in out_a:                           # integer work: the tolerance is equality
            assert np.array_equal(out_a[key], out_b[key]), (name, k, key)
        for key in st_a:
            assert np.array_equal(st_a[key], st_b[key]), (name, k, key)
        assert int(st_b["step"][0]) == k + 1
        assert (out_b["assign"][0] >= -1).all() and (out_b["trace"][0][:, 0] >= out_b["trace"][0][:, 1]).all()
    # no device memory was taken: free memory is the same before and after the second and third call
    # (the first call may load the library's kernels, which the driver places in device memory)
    for before, after in free_seen[1:]:
        assert after == before
    r.close()


def test_static_staging_rejects_batches_beyond_its_size():
    cfg = wlm.get_config("c3")
    n_inst = 1024                                   # ~20 KB per instance: well over 8 MiB
    wl = wlm.make_workload(cfg, n_instances=n_inst)
    r = Router(wl, device="cuda:0")
    st, out = _host_buffers(wl, r, n_inst)
    need = sum(((v.nbytes + 255) // 256) * 256 for v in list(st.values()) + list(out.values()))
    assert need > STATIC_STAGE_BYTES
    before = {k: v.copy() for k, v in st.items()}
    with pytest.raises(BrError) as ei:
        r.step_host_static(st, out)
    assert ei.value.status == BR_ELIMIT and "BR_STATIC_STAGE_BYTES" in str(ei.value)
    for k in st:                                    # a rejected call leaves the snapshot untouched
        assert np.array_equal(st[k], before[k])
    r.close()
