"""ctypes front end of the CPU reference checker (TEST INFRASTRUCTURE).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It takes its inputs in the same array formats as the CUDA
library's boundary so the two can be compared field by field, but shares no
code with it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "br_oracle.c")
_LIB = os.path.join(_HERE, "libbr_oracle.so")
EMPTY = -(2 ** 31)


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared",
                               "-Wall", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class OrcParams(C.Structure):
    _fields_ = [
        ("G", C.c_int32), ("H", C.c_int32), ("B", C.c_int32), ("W", C.c_int32),
        ("R_max", C.c_int32), ("S_greedy", C.c_int32),
        ("alpha", C.c_double), ("beta", C.c_double), ("gamma", C.c_double),
        ("delta_T", C.c_int32), ("gate", C.c_float), ("c_floor", C.c_float),
        ("score_mode", C.c_int32), ("term_mode", C.c_int32), ("term_cdf", C.c_void_p),
        ("arr_cdf", C.c_void_p), ("arr_len", C.c_int32), ("arr_period", C.c_int32),
        ("len_tab", C.c_void_p), ("len_tab_log2", C.c_int32),
        ("burst_every", C.c_int32), ("burst_size", C.c_int32), ("router", C.c_int32),
        ("pred_mode", C.c_int32), ("out_tab", C.c_void_p), ("out_tab_log2", C.c_int32),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_create.restype = C.c_void_p
        L.orc_create.argtypes = [C.POINTER(OrcParams), C.c_uint64]
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_set_state.argtypes = [C.c_void_p, C.c_int32, C.c_uint32] + [C.c_void_p] * 6 + [C.c_int32]
        L.orc_get_state.argtypes = [C.c_void_p] + [C.c_void_p] * 10
        L.orc_set_lifetimes.argtypes = [C.c_void_p] * 3
        L.orc_get_lifetimes.argtypes = [C.c_void_p] * 3
        L.orc_step.argtypes = [C.c_void_p] + [C.c_void_p] * 5
        L.orc_route_only.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_projection.argtypes = [C.c_void_p] + [C.c_void_p] * 3
        L.orc_round_projection.argtypes = [C.c_void_p] + [C.c_void_p] * 3
        L.orc_predict_only.argtypes = [C.c_void_p, C.c_void_p]
        L.orc_philox4x32_10.argtypes = [C.c_void_p] * 3
        L.orc_term_gap.restype = C.c_int
        L.orc_term_gap.argtypes = [C.c_void_p, C.c_int32, C.c_uint32]
        L.orc_f_br0.restype = C.c_int64
        L.orc_f_br0.argtypes = [C.c_int32, C.c_int64, C.c_int64]
        L.orc_f_brh.restype = C.c_double
        L.orc_f_brh.argtypes = [C.c_int32, C.c_double, C.c_double, C.c_void_p, C.c_double,
                                C.c_int64, C.c_void_p]
        L.orc_discount.restype = C.c_double
        L.orc_discount.argtypes = [C.c_int32, C.c_double, C.c_void_p]
        L.orc_imbalance.restype = C.c_int64
        L.orc_imbalance.argtypes = [C.c_int32, C.c_void_p]
        L.orc_chat_star.restype = C.c_double
        L.orc_chat_star.argtypes = [C.c_int32, C.c_void_p, C.c_void_p]
        L.orc_chat_two_stage.restype = C.c_double
        L.orc_chat_two_stage.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_best_subset.restype = C.c_uint32
        L.orc_best_subset.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_double, C.c_double,
                                      C.c_double, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                      C.c_void_p]
        L.orc_bypass.argtypes = [C.c_int32, C.c_int32, C.c_double, C.c_double, C.c_void_p, C.c_int32,
                                 C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_survival.restype = C.c_double
        L.orc_survival.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


# ---- pure functions ------------------------------------------------------
def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32); k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def term_gap(term_cdf, u: int) -> int:
    """Slots skipped before the next ending one, from one uniform 32-bit word."""
    t = np.ascontiguousarray(term_cdf, dtype=np.uint32)
    return int(lib().orc_term_gap(_p(t), len(t), int(u)))


def f_br0(G: int, delta: int, m: int) -> int:
    return int(lib().orc_f_br0(G, delta, m))


def discount(H: int, gamma: float):
    d = np.zeros(H + 1, dtype=np.float64)
    D = lib().orc_discount(H, gamma, _p(d))
    return d, float(D)


def f_brh(H: int, alpha: float, beta: float, gamma: float, delta: int, m) -> float:
    d, D = discount(H, gamma)
    mm = np.ascontiguousarray(m, dtype=np.int64)
    assert mm.shape == (H + 1,)
    return float(lib().orc_f_brh(H, alpha, beta, _p(d), D, int(delta), _p(mm)))


def imbalance(L) -> int:
    a = np.ascontiguousarray(L, dtype=np.int64)
    return int(lib().orc_imbalance(len(a), _p(a)))


def chat_star(q):
    a = np.ascontiguousarray(q, dtype=np.float32)
    pf = C.c_double()
    v = lib().orc_chat_star(len(a), _p(a), C.addressof(pf))
    return float(v), float(pf.value)


def chat_two_stage(q):
    a = np.ascontiguousarray(q, dtype=np.float32)
    pf = C.c_double(); mu = C.c_double()
    v = lib().orc_chat_two_stage(len(a), _p(a), C.addressof(pf), C.addressof(mu))
    return float(v), float(pf.value), float(mu.value)


def best_subset(score_mode, G, H, alpha, beta, gamma, m, win, lim):
    mm = np.ascontiguousarray(m, dtype=np.int64)
    ww = np.ascontiguousarray(win, dtype=np.int32)
    f = C.c_double()
    mask = lib().orc_best_subset(score_mode, G, H, alpha, beta, gamma, _p(mm), _p(ww), len(ww),
                                 lim, C.addressof(f))
    return int(mask), float(f.value)


def survival(hist, H, age):
    """Empirical-survival (c_hat, p_fin, mu_rem) of a request of the given age."""
    h = np.ascontiguousarray(hist, dtype=np.int32)
    p = C.c_double(); mu = C.c_double()
    c = lib().orc_survival(_p(h), len(h), int(H), int(age), C.addressof(p), C.addressof(mu))
    return float(c), float(p.value), float(mu.value)


def bypass(G, s, vload, inflight, cap, score_mode=0, alpha=1.0, beta=None):
    """Pool-bypass dispatch of the requests s in order; returns (workers, virtual loads, inflight)."""
    ss = np.ascontiguousarray(s, dtype=np.int32)
    L = np.ascontiguousarray(vload, dtype=np.int64).copy()
    n = np.ascontiguousarray(inflight, dtype=np.int32).copy()
    c = np.ascontiguousarray(cap, dtype=np.int32)
    out = np.zeros(len(ss), dtype=np.int32)
    lib().orc_bypass(G, score_mode, alpha, float(G) if beta is None else beta, _p(ss), len(ss), _p(L), _p(n),
                     _p(c), _p(out))
    return out, L, n


# ---- one routing instance --------------------------------------------------
class Instance:
    """One routing instance.  ``arr_rows`` is that instance's [period, len]
    block of arrival thresholds, ``len_tab`` the prompt-length table."""

    def __init__(self, *, G, H, B, W, R_max=4, S_greedy=None, alpha=1.0, beta=None, gamma=1.0,
                 delta_T=None, gate=0.5, c_floor=1.0, score_mode=None, term_mode=0,
                 term_cdf=None, arr_rows=None, len_tab=None, burst_every=0, burst_size=0,
                 router=0, seed=0, pred_mode=0, out_tab=None):
        self.G, self.H, self.B, self.W = G, H, B, W
        self._arr = np.ascontiguousarray(
            arr_rows if arr_rows is not None else np.full((1, 1), 0xFFFFFFFF), dtype=np.uint32)
        self._len = np.ascontiguousarray(
            len_tab if len_tab is not None else np.ones(2, dtype=np.int32), dtype=np.int32)
        self._term = np.ascontiguousarray(
            term_cdf if term_cdf is not None else np.zeros(B, dtype=np.uint32), dtype=np.uint32)
        assert self._term.shape == (B,)
        log2 = int(self._len.size).bit_length() - 1
        assert 1 << log2 == self._len.size
        self._out = np.ascontiguousarray(
            out_tab if out_tab is not None else np.ones(2, dtype=np.int32), dtype=np.int32)
        olog2 = int(self._out.size).bit_length() - 1
        assert 1 << olog2 == self._out.size
        p = OrcParams(
            G=G, H=H, B=B, W=W, R_max=R_max, S_greedy=2 * G if S_greedy is None else S_greedy,
            alpha=alpha, beta=float(G) if beta is None else beta, gamma=gamma,
            delta_T=max(1, H // 2) if delta_T is None else delta_T, gate=gate, c_floor=c_floor,
            score_mode=(0 if H == 0 else 1) if score_mode is None else score_mode,
            term_mode=term_mode, term_cdf=self._term.ctypes.data,
            arr_cdf=self._arr.ctypes.data, arr_len=self._arr.shape[1],
            arr_period=self._arr.shape[0], len_tab=self._len.ctypes.data, len_tab_log2=log2,
            burst_every=burst_every, burst_size=burst_size, router=router,
            pred_mode=pred_mode, out_tab=self._out.ctypes.data, out_tab_log2=olog2)
        self.params = p
        self._h = lib().orc_create(C.byref(p), C.c_uint64(int(seed)))

    def __del__(self):
        if getattr(self, "_h", None):
            lib().orc_destroy(self._h)
            self._h = None

    # state in boundary format: act_base (EMPTY marker), chat/tau in explicit form
    def set_state(self, k, next_id, act_base, act_id=None, chat=None, tau=None,
                  wq_s=None, wq_id=None, wq_n=0):
        A = self.G * self.B
        assert 0 <= int(wq_n) <= self.W, "queue length beyond the capacity W"
        ab = np.ascontiguousarray(act_base, dtype=np.int32).reshape(A)
        ai = None if act_id is None else np.ascontiguousarray(act_id, dtype=np.uint32).reshape(A)
        ch = None if chat is None else np.ascontiguousarray(chat, dtype=np.float32).reshape(A)
        ta = None if tau is None else np.ascontiguousarray(tau, dtype=np.int32).reshape(A)
        qs = np.ascontiguousarray(wq_s if wq_s is not None else np.zeros(self.W), dtype=np.int32)
        qi = None if wq_id is None else np.ascontiguousarray(wq_id, dtype=np.uint32)
        lib().orc_set_state(self._h, int(k), int(next_id), _p(ab), _p(ai), _p(ch), _p(ta),
                            _p(qs), _p(qi), int(wq_n))

    def set_lifetimes(self, act_end, wq_o):
        """term_mode 3: the step at whose end each running request finishes, and the output
        lengths of the waiting requests (call after set_state)."""
        ae = np.ascontiguousarray(act_end, dtype=np.int32).reshape(self.G * self.B)
        qo = np.ascontiguousarray(wq_o, dtype=np.int32).reshape(self.W)
        lib().orc_set_lifetimes(self._h, _p(ae), _p(qo))

    def get_lifetimes(self):
        ae = np.zeros(self.G * self.B, dtype=np.int32); qo = np.zeros(self.W, dtype=np.int32)
        lib().orc_get_lifetimes(self._h, _p(ae), _p(qo))
        return ae.reshape(self.G, self.B), qo

    def get_state(self) -> Dict[str, np.ndarray]:
        A = self.G * self.B
        k = C.c_int32(); nid = C.c_uint32(); qn = C.c_int32()
        ab = np.zeros(A, dtype=np.int32); ai = np.zeros(A, dtype=np.uint32)
        ch = np.zeros(A, dtype=np.float32); ta = np.zeros(A, dtype=np.int32)
        qs = np.zeros(self.W, dtype=np.int32); qi = np.zeros(self.W, dtype=np.uint32)
        cnt = np.zeros(5, dtype=np.int64)
        lib().orc_get_state(self._h, C.addressof(k), C.addressof(nid), _p(ab), _p(ai), _p(ch),
                            _p(ta), _p(qs), _p(qi), C.addressof(qn), _p(cnt))
        return dict(step=k.value, next_id=nid.value, act_base=ab.reshape(self.G, self.B),
                    act_id=ai.reshape(self.G, self.B), chat=ch.reshape(self.G, self.B),
                    tau=ta.reshape(self.G, self.B), wq_s=qs, wq_id=qi, wq_n=qn.value,
                    counters=cnt)

    def step(self, probs=None, want_fscore=False):
        pr = None if probs is None else np.ascontiguousarray(probs, dtype=np.float32)
        assign = np.zeros(self.W, dtype=np.int32)
        load = np.zeros(self.G, dtype=np.int64)
        trace = np.zeros(3, dtype=np.int64)
        fs = np.zeros((self.W, self.G), dtype=np.float64) if want_fscore else None
        lib().orc_step(self._h, _p(pr), _p(assign), _p(load), _p(trace), _p(fs))
        return assign, load, trace, fs

    def route_only(self):
        assign = np.zeros(self.W, dtype=np.int32)
        loads = np.zeros(self.G, dtype=np.int64)
        lib().orc_route_only(self._h, _p(assign), _p(loads))
        return assign, loads

    def projection(self):
        H1 = self.H + 1
        Lh = np.zeros((self.G, H1), dtype=np.int64); Mh = np.zeros(H1, dtype=np.int64)
        m = np.zeros((self.G, H1), dtype=np.int64)
        lib().orc_projection(self._h, _p(Lh), _p(Mh), _p(m))
        return Lh, Mh, m

    def round_projection(self):
        """Projected loads, envelope and margins as the last routing round left them."""
        H1 = self.H + 1
        Lh = np.zeros((self.G, H1), dtype=np.int64); Mh = np.zeros(H1, dtype=np.int64)
        m = np.zeros((self.G, H1), dtype=np.int64)
        lib().orc_round_projection(self._h, _p(Lh), _p(Mh), _p(m))
        return Lh, Mh, m

    def predict_only(self, probs):
        pr = np.ascontiguousarray(probs, dtype=np.float32)
        lib().orc_predict_only(self._h, _p(pr))


# ---- glue: build an Instance from a generated workload ---------------------
def explicit_pred_state(act_chat0, act_kref, k):
    """(chat0, kref) storage of the boundary -> explicit (c_hat, tau) entering step k."""
    tau = ((int(k) - act_kref.astype(np.int64)) & 255) - 1
    chat = (act_chat0.astype(np.float32) - tau.astype(np.float32)).astype(np.float32)
    return chat, tau.astype(np.int32)


def instance_from_workload(wl, inst: int, router: int = 0, **overrides) -> Instance:
    cfg = wl.cfg
    kw = dict(G=cfg.G, H=cfg.H, B=cfg.B, W=cfg.W, R_max=cfg.R_max, S_greedy=cfg.S_greedy,
              alpha=cfg.alpha, beta=cfg.beta, gamma=cfg.gamma, delta_T=cfg.delta_T,
              gate=cfg.gate, c_floor=cfg.c_floor, score_mode=cfg.score_mode,
              term_mode=cfg.term_mode, term_cdf=wl.term_cdf, arr_rows=wl.arr_rows_for(inst),
              len_tab=wl.len_tab, burst_every=cfg.burst_every, burst_size=cfg.burst_size,
              router=router, seed=int(wl.seeds[inst]), pred_mode=cfg.pred_mode, out_tab=wl.out_tab)
    if cfg.score_mode == 0:
        kw["beta"] = float(cfg.G)
        kw["alpha"] = 1.0
    kw.update(overrides)
    o = Instance(**kw)
    st = wl.state
    k = int(st["step"][inst])
    chat, tau = explicit_pred_state(st["act_chat0"][inst], st["act_kref"][inst], k)
    o.set_state(k, int(st["next_id"][inst]), st["act_base"][inst], st["act_id"][inst], chat, tau,
                st["wq_s"][inst], st["wq_id"][inst], int(st["wq_n"][inst]))
    if "act_end" in st:
        o.set_lifetimes(st["act_end"][inst], st["wq_o"][inst])
    return o
