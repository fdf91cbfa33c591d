"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every entry
point that include/br.h declares, and rejects bad arguments with status codes before any
CUDA call."""
import ctypes as C
import os
import re

import pytest

from paper_2605_06113_b200 import binding
from paper_2605_06113_b200.binding import (BR_EINVAL, BR_ERANGE, BR_ESTATE, BR_OK, BrInstanceBatch,
                                           BrLoadOut, BrParams, BrWaitingQueue, BrWorkerState)

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "br.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(br_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_entry_point():
    names = _declared()
    assert {"br_create", "br_step", "br_destroy"} <= set(names)
    L = binding.lib()
    for n in names:
        assert hasattr(L, n), n
    assert sorted(binding.EXPORTS) == names
    assert L.br_version() == 102
    assert L.br_strerror(BR_OK) == b"ok"
    assert b"invalid" in L.br_strerror(BR_EINVAL)


def _params(**kw):
    p = BrParams(B=64, W=256, R_max=0, S_greedy=-1, alpha=1.0, beta=14.67, gamma=0.64, delta_T=0,
                 gate=-1.0, c_floor=-1.0, score_mode=-1, term_mode=1, term_cdf=0x1000, arr_cdf=None,
                 arr_len=0, arr_period=0, arr_inst_stride=0, len_tab=None, len_tab_log2=0,
                 burst_every=0, burst_size=0, s_max=131072, threads=0, inst_per_block=0)
    for k, v in kw.items():
        setattr(p, k, v)
    return p


def _create(G, H, p):
    h = C.c_void_p()
    rc = binding.lib().br_create(G, H, C.byref(p), C.byref(h))
    return rc, h


def test_create_validates_sizes_and_ranges():
    L = binding.lib()
    rc, h = _create(32, 0, _params())
    assert rc == BR_OK and h.value
    assert L.br_graph_step(h) == BR_ESTATE              # nothing captured yet
    assert L.br_destroy(h) == BR_OK
    assert L.br_destroy(None) == BR_OK
    for G, H, kw in [(0, 0, {}), (65, 0, {}), (32, 81, {}), (32, -1, {}), (32, 0, dict(B=12)),
                     (32, 0, dict(B=264)), (32, 0, dict(W=6)), (32, 0, dict(W=8192)),
                     (32, 0, dict(R_max=17)), (32, 4, dict(score_mode=0)), (32, 0, dict(term_mode=2)),
                     (32, 0, dict(term_mode=4)), (32, 4, dict(pred_mode=1)), (32, 0, dict(term_mode=3, pred_mode=1)), (32, 0, dict(term_cdf=None)), (32, 4, dict(gamma=0.0)), (32, 4, dict(gamma=1.5)),
                     (32, 4, dict(alpha=-1.0)), (32, 0, dict(threads=48)), (32, 0, dict(threads=512)),
                     (32, 4, dict(delta_T=200))]:
        rc, h = _create(G, H, _params(**kw))
        assert rc == BR_EINVAL, (G, H, kw)
        assert not h.value
    # value ranges the 32-bit device arithmetic cannot hold
    for kw in [dict(s_max=1 << 23), dict(W=4096, s_max=1 << 19), dict(B=256, s_max=1 << 22)]:
        rc, h = _create(64, 0, _params(**kw))
        assert rc == BR_ERANGE, kw
    assert L.br_create(32, 0, None, None) == BR_EINVAL


def test_step_rejects_null_and_misaligned_pointers_without_touching_the_gpu():
    L = binding.lib()
    rc, h = _create(8, 0, _params(W=64))
    assert rc == BR_OK
    b = BrInstanceBatch(n_instances=1, first_instance=0, n_steps=1, stream=None)
    ws, wq, lo = BrWorkerState(), BrWaitingQueue(), BrLoadOut()
    assert L.br_step(h, C.byref(b), C.byref(ws), C.byref(wq), None, None, C.byref(lo)) == BR_EINVAL
    assert L.br_step(None, C.byref(b), C.byref(ws), C.byref(wq), None, None, C.byref(lo)) == BR_EINVAL
    fake = 0x1000                      # never dereferenced: validation fails first
    for f in ("load", "nact", "occ", "act_base", "step", "seed", "next_id"):
        setattr(ws, f, fake)
    wq.s, wq.id, wq.n = fake, fake, fake
    lo.load, lo.trace = fake, fake
    ws.act_base = fake + 4             # not 16-byte aligned
    assert L.br_step(h, C.byref(b), C.byref(ws), C.byref(wq), None, fake, C.byref(lo)) == BR_EINVAL
    ws.act_base = fake
    b.n_instances = -1
    assert L.br_step(h, C.byref(b), C.byref(ws), C.byref(wq), None, fake, C.byref(lo)) == BR_EINVAL
    b.n_instances, b.n_steps, b.first_instance = 4, 2, 1     # multi-step launches start at row 0
    assert L.br_step(h, C.byref(b), C.byref(ws), C.byref(wq), None, fake, C.byref(lo)) == BR_EINVAL
    b.n_instances, b.n_steps, b.first_instance = 0, 1, 0     # empty batch: a no-op
    assert L.br_step(h, C.byref(b), C.byref(ws), C.byref(wq), None, fake, C.byref(lo)) == BR_OK
    assert L.br_fscore(h, C.byref(b), None, 4, None, None, None, None) == BR_EINVAL
    L.br_destroy(h)
    # BR-H needs the predictor state and the classifier output
    rc, h = _create(8, 4, _params(W=64))
    assert rc == BR_OK
    b.n_instances = 1
    assert L.br_step(h, C.byref(b), C.byref(ws), C.byref(wq), None, fake, C.byref(lo)) == BR_EINVAL
    L.br_destroy(h)
