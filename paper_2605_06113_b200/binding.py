"""Thin ctypes binding of libbr.so: the same calls as include/br.h, argument
marshalling only.  Device memory and streams come from PyTorch; every step of the
routing path runs inside the library's CUDA kernels.  There is no fallback: if the
library is missing or a call fails, an exception is raised."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbr.so")

BR_OK, BR_EINVAL, BR_ERANGE, BR_ECUDA, BR_ENOMEM, BR_ESTATE, BR_ELIMIT = 0, -1, -2, -3, -4, -5, -6
STATIC_STAGE_BYTES = 8 << 20
ST_QUEUE_OVERFLOW, ST_ITER_CAP, ST_BAD_STATE = 1, 2, 4
EMPTY = -(2 ** 31)


class BrParams(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("W", C.c_int32), ("R_max", C.c_int32), ("S_greedy", C.c_int32),
        ("alpha", C.c_double), ("beta", C.c_double), ("gamma", C.c_double),
        ("delta_T", C.c_int32), ("gate", C.c_float), ("c_floor", C.c_float),
        ("score_mode", C.c_int32), ("term_mode", C.c_int32), ("term_cdf", C.c_void_p),
        ("arr_cdf", C.c_void_p), ("arr_len", C.c_int32), ("arr_period", C.c_int32),
        ("arr_inst_stride", C.c_int32),
        ("len_tab", C.c_void_p), ("len_tab_log2", C.c_int32),
        ("burst_every", C.c_int32), ("burst_size", C.c_int32),
        ("s_max", C.c_int32), ("threads", C.c_int32), ("inst_per_block", C.c_int32),
        ("pred_mode", C.c_int32), ("out_tab", C.c_void_p), ("out_tab_log2", C.c_int32),
    ]


class BrWorkerState(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("load", "nact", "occ", "act_base", "act_id", "act_chat0", "act_kref", "act_end",
                 "step", "seed", "next_id")]


class BrWaitingQueue(C.Structure):
    _fields_ = [("s", C.c_void_p), ("id", C.c_void_p), ("n", C.c_void_p), ("o", C.c_void_p)]


class BrInstanceBatch(C.Structure):
    _fields_ = [("n_instances", C.c_int32), ("first_instance", C.c_int32),
                ("n_steps", C.c_int32), ("stream", C.c_void_p)]


class BrLoadOut(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("load", "trace", "status", "counters", "fscore",
                                          "phase_cycles")]


EXPORTS = ["br_create", "br_step", "br_graph_capture", "br_graph_step", "br_step_host",
           "br_step_host_static", "br_debug_bounds_hits", "br_debug_bounds_selftest",
           "br_fscore", "br_best_subset", "br_bypass_dispatch", "br_survival_chat", "br_destroy", "br_strerror", "br_version"]

_lib = None


class BrError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().br_strerror(status).decode()
        super().__init__(f"{where}: status {status} ({msg})")


def lib():
    """Loads libbr.so.  Raises if it has not been built (python -m paper_2605_06113_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build the CUDA library first "
                               "(python paper_2605_06113_b200/build.py)")
        L = C.CDLL(LIB_PATH)
        step_args = [C.c_void_p, C.POINTER(BrInstanceBatch), C.POINTER(BrWorkerState),
                     C.POINTER(BrWaitingQueue), C.c_void_p, C.c_void_p, C.POINTER(BrLoadOut)]
        L.br_create.argtypes = [C.c_int32, C.c_int32, C.POINTER(BrParams), C.POINTER(C.c_void_p)]
        L.br_step.argtypes = step_args
        L.br_graph_capture.argtypes = step_args
        L.br_graph_step.argtypes = [C.c_void_p]
        L.br_step_host.argtypes = step_args + [C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.br_step_host_static.argtypes = step_args + [C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.br_fscore.argtypes = [C.c_void_p, C.POINTER(BrInstanceBatch), C.c_void_p, C.c_int32,
                                C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.br_best_subset.argtypes = [C.c_void_p, C.POINTER(BrInstanceBatch), C.c_void_p, C.c_int32,
                                     C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.br_bypass_dispatch.argtypes = [C.c_void_p, C.POINTER(BrInstanceBatch), C.c_void_p, C.c_int32,
                                         C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.br_survival_chat.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                       C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p]
        L.br_debug_bounds_hits.argtypes = []
        L.br_debug_bounds_selftest.argtypes = [C.c_void_p]
        L.br_destroy.argtypes = [C.c_void_p]
        L.br_strerror.restype = C.c_char_p
        L.br_strerror.argtypes = [C.c_int]
        for n in EXPORTS:
            if n != "br_strerror":
                getattr(L, n).restype = C.c_int
        _lib = L
    return _lib


def use_library(path: Optional[str] = None) -> None:
    """Makes lib() load another build of the library (the range-checked libbr_dbg.so); None goes
    back to libbr.so.  Contexts created earlier keep the library they were created with only as
    long as the caller keeps using them through it: close them first."""
    global _lib, LIB_PATH
    _lib = None
    LIB_PATH = os.path.join(_HERE, "libbr.so") if path is None else path


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _to_torch(a: np.ndarray, device):
    """numpy -> torch on `device`, keeping the bit pattern of unsigned types."""
    import torch
    if a.dtype == np.uint64:
        return torch.from_numpy(a.view(np.int64).copy()).to(device)
    if a.dtype == np.uint32:
        return torch.from_numpy(a.view(np.int32).copy()).to(device)
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


_STATE_DTYPES = dict(load=np.int64, nact=np.int32, occ=np.uint64, act_base=np.int32,
                     act_id=np.uint32, act_chat0=np.float32, act_kref=np.uint8, step=np.int32,
                     seed=np.uint64, next_id=np.uint32, wq_s=np.int32, wq_id=np.uint32, wq_n=np.int32,
                     act_end=np.int32, wq_o=np.int32)


class Router:
    """br_create / br_step / br_destroy for one fleet shape, fed from a generated workload."""

    def __init__(self, wl, device="cuda:0", threads: int = 0, **overrides):
        import torch
        self.torch = torch
        self.wl = wl
        cfg = wl.cfg
        self.cfg = cfg
        self.device = torch.device(device)
        self.len_tab = _to_torch(wl.len_tab, self.device)
        self.arr_cdf = _to_torch(wl.arr_cdf, self.device)
        self.term_cdf = _to_torch(wl.term_cdf, self.device)
        self.out_tab = _to_torch(wl.out_tab, self.device) if wl.out_tab is not None else None
        p = BrParams(
            B=cfg.B, W=cfg.W, R_max=cfg.R_max, S_greedy=cfg.S_greedy, alpha=cfg.alpha,
            beta=cfg.beta, gamma=cfg.gamma, delta_T=cfg.delta_T, gate=cfg.gate, c_floor=cfg.c_floor,
            score_mode=cfg.score_mode, term_mode=cfg.term_mode, term_cdf=self.term_cdf.data_ptr(),
            arr_cdf=self.arr_cdf.data_ptr(), arr_len=wl.arr_cdf.shape[1], arr_period=wl.arr_period,
            arr_inst_stride=wl.arr_inst_stride, len_tab=self.len_tab.data_ptr(),
            len_tab_log2=int(wl.len_tab.size).bit_length() - 1, burst_every=cfg.burst_every,
            burst_size=cfg.burst_size, s_max=int(max(cfg.len_clip[1], cfg.ctx_clip[1])),
            threads=threads, pred_mode=cfg.pred_mode,
            out_tab=self.out_tab.data_ptr() if self.out_tab is not None else None,
            out_tab_log2=int(wl.out_tab.size).bit_length() - 1 if wl.out_tab is not None else 0)
        for k, v in overrides.items():
            setattr(p, k, v)
        self.params = p
        h = C.c_void_p()
        rc = lib().br_create(cfg.G, cfg.H, C.byref(p), C.byref(h))
        if rc != BR_OK:
            raise BrError(rc, "br_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib().br_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- buffers -----------------------------------------------------------
    def device_state(self, state: Optional[Dict[str, np.ndarray]] = None) -> Dict[str, "object"]:
        st = self.wl.state if state is None else state
        return {k: _to_torch(np.ascontiguousarray(v, dtype=_STATE_DTYPES[k]), self.device)
                for k, v in st.items()}

    def outputs(self, N: int, n_steps: int = 1, fscore: bool = False, device=None):
        t = self.torch
        dev = self.device if device is None else device
        cfg = self.cfg
        o = dict(
            assign=t.empty((n_steps, N, cfg.W), dtype=t.int32, device=dev),
            load=t.empty((n_steps, N, cfg.G), dtype=t.int64, device=dev),
            trace=t.empty((n_steps, N, 3), dtype=t.int64, device=dev),
            status=t.zeros((n_steps, N), dtype=t.int32, device=dev),
            counters=t.zeros((n_steps, N, 4), dtype=t.int32, device=dev),
        )
        if fscore:
            o["fscore"] = t.zeros((n_steps, N, cfg.W, cfg.G), dtype=t.float64, device=dev)
        return o

    def _structs(self, st, out, N, first, n_steps, stream):
        ws = BrWorkerState(**{k: _ptr(st.get(k)) for k in
                              ("load", "nact", "occ", "act_base", "act_id", "act_chat0", "act_kref", "act_end",
                               "step", "seed", "next_id")})
        wq = BrWaitingQueue(s=_ptr(st["wq_s"]), id=_ptr(st["wq_id"]), n=_ptr(st["wq_n"]), o=_ptr(st.get("wq_o")))
        lo = BrLoadOut(load=_ptr(out["load"]), trace=_ptr(out["trace"]), status=_ptr(out.get("status")),
                       counters=_ptr(out.get("counters")), fscore=_ptr(out.get("fscore")),
                       phase_cycles=_ptr(out.get("phase_cycles")))
        b = BrInstanceBatch(n_instances=N, first_instance=first, n_steps=n_steps, stream=stream)
        return b, ws, wq, lo

    def _stream(self, stream):
        if stream is None:
            return self.torch.cuda.current_stream(self.device).cuda_stream
        return stream.cuda_stream if hasattr(stream, "cuda_stream") else stream

    # ---- the calls of include/br.h -------------------------------------------
    def step(self, st, out, term_probs=None, N=None, first=0, n_steps=1, stream=None):
        N = st["step"].shape[0] - first if N is None else N
        b, ws, wq, lo = self._structs(st, out, N, first, n_steps, self._stream(stream))
        rc = lib().br_step(self._h, C.byref(b), C.byref(ws), C.byref(wq), _ptr(term_probs),
                           _ptr(out["assign"]), C.byref(lo))
        if rc != BR_OK:
            raise BrError(rc, "br_step")

    def prepare(self, st, out, term_probs=None, N=None, first=0, n_steps=1, stream=None):
        """Marshals the arguments of br_step once; the returned callable repeats the same call
        (same buffers, same stream) without rebuilding the argument structures."""
        N = st["step"].shape[0] - first if N is None else N
        b, ws, wq, lo = self._structs(st, out, N, first, n_steps, self._stream(stream))
        fn, h = lib().br_step, self._h
        args = (h, C.byref(b), C.byref(ws), C.byref(wq), _ptr(term_probs), _ptr(out["assign"]), C.byref(lo))
        keep = (b, ws, wq, lo, st, out, term_probs)

        def call(_fn=fn, _args=args, _keep=keep):
            rc = _fn(*_args)
            if rc != BR_OK:
                raise BrError(rc, "br_step")
        return call

    def graph_capture(self, st, out, term_probs=None, N=None, first=0, n_steps=1, stream=None):
        N = st["step"].shape[0] - first if N is None else N
        b, ws, wq, lo = self._structs(st, out, N, first, n_steps, self._stream(stream))
        rc = lib().br_graph_capture(self._h, C.byref(b), C.byref(ws), C.byref(wq), _ptr(term_probs),
                                    _ptr(out["assign"]), C.byref(lo))
        if rc != BR_OK:
            raise BrError(rc, "br_graph_capture")

    def graph_step(self):
        rc = lib().br_graph_step(self._h)
        if rc != BR_OK:
            raise BrError(rc, "br_graph_step")

    def step_host(self, st, out, term_probs=None, N=None, stream=None):
        """st / out / term_probs are host tensors or numpy arrays (pinned for async copies)."""
        N = st["step"].shape[0] if N is None else N
        b, ws, wq, lo = self._structs(st, out, N, 0, 1, self._stream(stream))
        up, down = C.c_int64(), C.c_int64()
        rc = lib().br_step_host(self._h, C.byref(b), C.byref(ws), C.byref(wq), _ptr(term_probs),
                                _ptr(out["assign"]), C.byref(lo), C.byref(up), C.byref(down))
        if rc != BR_OK:
            raise BrError(rc, "br_step_host")
        return up.value, down.value

    def step_host_static(self, st, out, term_probs=None, N=None, stream=None):
        """br_step_host_static: like step_host, but the device staging is the library's built-in
        array, so nothing is allocated; raises BrError(BR_ELIMIT) if the batch does not fit."""
        N = st["step"].shape[0] if N is None else N
        b, ws, wq, lo = self._structs(st, out, N, 0, 1, self._stream(stream))
        up, down = C.c_int64(), C.c_int64()
        rc = lib().br_step_host_static(self._h, C.byref(b), C.byref(ws), C.byref(wq), _ptr(term_probs),
                                       _ptr(out["assign"]), C.byref(lo), C.byref(up), C.byref(down))
        if rc != BR_OK:
            raise BrError(rc, "br_step_host_static")
        return up.value, down.value

    def fscore(self, s, Lh, F, cap=None, best_g=None, N=None, first=0, stream=None):
        N = s.shape[0] - first if N is None else N
        b = BrInstanceBatch(n_instances=N, first_instance=first, n_steps=1, stream=self._stream(stream))
        rc = lib().br_fscore(self._h, C.byref(b), _ptr(s), int(s.shape[1]), _ptr(Lh), _ptr(cap),
                             _ptr(F), _ptr(best_g))
        if rc != BR_OK:
            raise BrError(rc, "br_fscore")


    def bypass_dispatch(self, s, virtual_load, inflight, inflight_cap, worker_out, N=None, first=0, stream=None):
        N = s.shape[0] - first if N is None else N
        b = BrInstanceBatch(n_instances=N, first_instance=first, n_steps=1, stream=self._stream(stream))
        rc = lib().br_bypass_dispatch(self._h, C.byref(b), _ptr(s), int(s.shape[1]), _ptr(virtual_load),
                                      _ptr(inflight), _ptr(inflight_cap), _ptr(worker_out))
        if rc != BR_OK:
            raise BrError(rc, "br_bypass_dispatch")

    def survival_chat(self, hist_sorted, hist_prefix, age, c_hat, p_fin=None, mu_rem=None, stream=None):
        rc = lib().br_survival_chat(self._h, self._stream(stream), _ptr(hist_sorted), _ptr(hist_prefix),
                                    int(hist_sorted.numel()), _ptr(age), int(age.numel()), _ptr(c_hat),
                                    _ptr(p_fin), _ptr(mu_rem))
        if rc != BR_OK:
            raise BrError(rc, "br_survival_chat")

    def best_subset(self, win, margins, lim, best_mask, best_F=None, N=None, first=0, stream=None):
        N = win.shape[0] - first if N is None else N
        b = BrInstanceBatch(n_instances=N, first_instance=first, n_steps=1, stream=self._stream(stream))
        rc = lib().br_best_subset(self._h, C.byref(b), _ptr(win), int(win.shape[1]), _ptr(margins), _ptr(lim),
                                  _ptr(best_mask), _ptr(best_F))
        if rc != BR_OK:
            raise BrError(rc, "br_best_subset")


def state_to_numpy(st) -> Dict[str, np.ndarray]:
    """Device (or host) torch state -> numpy with the boundary's unsigned types restored."""
    out = {}
    for k, v in st.items():
        a = v.detach().cpu().numpy() if not isinstance(v, np.ndarray) else v
        want = _STATE_DTYPES[k]
        if a.dtype != want and a.dtype.itemsize == np.dtype(want).itemsize:
            a = a.view(want)
        out[k] = a
    return out
