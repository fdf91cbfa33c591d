"""Seeded synthetic inputs for the BalanceRoute routing step.

This module only *generates inputs*: distribution tables, initial cluster
snapshots and the stand-in classifier probabilities.  It contains none of the
router's arithmetic (no F-score, no selection, no load update) and is the one
module that both the CUDA path and the CPU checker read their inputs from.

Every value is a pure function of ``(instance seed, stream, index)`` through a
64-bit counter mixer (the SplitMix64 output function), so an instance's inputs
do not depend on which batch it is generated in.  Distributions are realised
through fp64-built lookup tables indexed by the top 16 bits of the mixed word:
the consumers only ever see integers and fp32 table entries, never libm.

Workload shapes follow the paper's evaluation regime (heavy-tailed prompt
lengths, near-saturation load, non-stationary and bursty arrivals; Section 5.1
"Datasets"); the traces themselves are not available and are not reproduced.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import Dict, Optional, Tuple

import numpy as np

EMPTY = np.int32(-(2 ** 31))          # act_base marker for a free slot
TAB_LOG2 = 16                          # all inverse-CDF tables have 2**16 entries
ARR_LEN = 64                           # thresholds per Poisson row

# mixer streams (one per kind of generated input)
STREAM_INIT_CTX = 1
STREAM_INIT_QUEUE = 2
STREAM_INIT_TAU = 3
STREAM_PROBS = 4
STREAM_RATE = 5
STREAM_INIT_END = 6
STREAM_INIT_QO = 7

_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_GOLD = 0x9E3779B97F4A7C15
_STREAM_MUL = 0xD6E8FEB86659FD93
_U64 = (1 << 64) - 1


# --------------------------------------------------------------------------
# counter mixer, numpy (uint64) and torch (int64, wrap-around) flavours
# --------------------------------------------------------------------------
def mix_np(seed, stream: int, idx) -> np.ndarray:
    """SplitMix64 output function applied to seed ^ stream-tag + idx * golden."""
    seed = np.asarray(seed, dtype=np.uint64)
    idx = np.asarray(idx, dtype=np.uint64)
    with np.errstate(over="ignore"):
        tag = np.uint64((stream * _STREAM_MUL) & _U64)
        z = (seed ^ tag) + idx * np.uint64(_GOLD)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(_M1)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(_M2)
        z = z ^ (z >> np.uint64(31))
    return z


def _s64(x: int) -> int:
    x &= _U64
    return x - (1 << 64) if x >= (1 << 63) else x


def mix_torch(seed, stream: int, idx):
    """Same function as :func:`mix_np` on torch int64 tensors (two's complement
    wrap-around; logical shifts emulated by masking)."""
    import torch

    def lsr(z, n):
        return (z >> n) & ((1 << (64 - n)) - 1)

    tag = _s64(stream * _STREAM_MUL)
    z = (seed ^ tag) + idx * _s64(_GOLD)
    z = (z ^ lsr(z, 30)) * _s64(_M1)
    z = (z ^ lsr(z, 27)) * _s64(_M2)
    z = z ^ lsr(z, 31)
    return z


# --------------------------------------------------------------------------
# tables
# --------------------------------------------------------------------------
def lognormal_table(mu: float, sigma: float, lo: int, hi: int) -> np.ndarray:
    """int32 inverse-CDF table of round(exp(mu + sigma z)) clipped to [lo, hi]."""
    from scipy.special import ndtri

    q = (np.arange(1 << TAB_LOG2, dtype=np.float64) + 0.5) / float(1 << TAB_LOG2)
    v = np.rint(np.exp(mu + sigma * ndtri(q)))
    return np.clip(v, lo, hi).astype(np.int32)


def beta_table(a: float, b: float) -> np.ndarray:
    """fp32 inverse-CDF table of Beta(a, b)."""
    from scipy.stats import beta as beta_dist

    q = (np.arange(1 << TAB_LOG2, dtype=np.float64) + 0.5) / float(1 << TAB_LOG2)
    return beta_dist.ppf(q, a, b).astype(np.float32)


def poisson_thresholds(lam) -> np.ndarray:
    """uint32 rows t[j] = min(2^32-1, floor(P(N <= j) * 2^32)), j < ARR_LEN.

    A uniform 32-bit word u realises N = #{j : u >= t[j]}.
    """
    from scipy.stats import poisson

    lam = np.atleast_1d(np.asarray(lam, dtype=np.float64))
    j = np.arange(ARR_LEN, dtype=np.float64)[None, :]
    cdf = poisson.cdf(j, lam[:, None])
    t = np.floor(cdf * 4294967296.0)
    return np.minimum(t, 4294967295.0).astype(np.uint32)


def termination_gap_thresholds(p: float, B: int) -> np.ndarray:
    """uint32 t[j] = min(2^32-1, floor(P(gap <= j) * 2^32)), j < B, for slots that end
    independently with probability p each: the number of slots skipped before the next ending
    one is geometric, P(gap <= j) = 1 - (1 - p)^(j+1).  A uniform 32-bit word u realises
    gap = #{j : u >= t[j]}; gap = B means that no further slot of the worker ends.
    """
    j = np.arange(1, B + 1, dtype=np.float64)
    if p <= 0.0:
        cdf = np.zeros(B, dtype=np.float64)
    elif p >= 1.0:
        cdf = np.ones(B, dtype=np.float64)
    else:
        cdf = -np.expm1(j * math.log1p(-p))
    return np.minimum(np.floor(cdf * 4294967296.0), 4294967295.0).astype(np.uint32)


# --------------------------------------------------------------------------
# configurations (the five benchmark shapes)
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class Config:
    name: str
    N: int
    G: int
    W: int
    H: int
    steps: int
    first_seed: int
    init_active: int              # occupied slots per worker at k = 0
    init_queue: int               # waiting requests at k = 0
    len_mu: float
    len_sigma: float
    arrival: Tuple                # ("const", lam) | ("sin", base, amp, period) | ("uniform", lo, hi)
    hazard: float                 # per-step termination probability (term_mode 1)
    term_mode: int = 1            # 0 none, 1 constant hazard, 2 Bernoulli(term_probs[slot][0]),
                                  # 3 every request carries its output length (out_mu, out_sigma)
    B: int = 64
    R_max: int = 4
    S_greedy: int = -1            # -1 -> 2 G
    alpha: float = 1.0
    beta: float = 14.67
    gamma: float = 0.64
    delta_T: int = -1             # -1 -> max(1, H // 2)
    gate: float = 0.5
    c_floor: float = 1.0
    score_mode: int = -1          # -1 -> 0 (Eq. 1, integers) if H == 0 else 1 (Eq. 2, fp64)
    beta_ab: Tuple[float, float] = (2.0, 50.0)
    burst_every: int = 0
    burst_size: int = 0
    len_clip: Tuple[int, int] = (1, 131072)
    ctx_clip: Tuple[int, int] = (16, 32768)
    pred_mode: int = 0            # 0 classifier rows (term_probs), 1 perfect lookahead min(r_i, H) (needs term_mode 3)
    out_mu: float = 6.5           # output lengths (decode steps) of term_mode 3: lognormal, clipped
    out_sigma: float = 1.0
    out_clip: Tuple[int, int] = (1, 32768)

    def resolved(self) -> "Config":
        c = self
        if c.S_greedy < 0:
            c = replace(c, S_greedy=2 * c.G)
        if c.delta_T < 0:
            c = replace(c, delta_T=max(1, c.H // 2))
        if c.score_mode < 0:
            c = replace(c, score_mode=0 if c.H == 0 else 1)
        return c


CONFIGS: Dict[str, Config] = {
    # BR-0, one instance, G=4, 300 steps, Poisson(2) arrivals, hazard 1/500
    "c0": Config("c0", N=1, G=4, W=128, H=0, steps=300, first_seed=0, init_active=32,
                 init_queue=0, len_mu=7.0, len_sigma=1.0, arrival=("const", 2.0),
                 hazard=1.0 / 500.0),
    # BR-0 latency path, G=16, 512 waiting, sinusoidal arrivals, geometric mean 400
    "c1": Config("c1", N=1, G=16, W=512, H=0, steps=2000, first_seed=1, init_active=64,
                 init_queue=512, len_mu=7.0, len_sigma=1.0,
                 arrival=("sin", 8.0, 6.0, 500), hazard=1.0 / 400.0),
    # BR-H, H=4, Beta(2,50) classifier probabilities, terminations drawn from them
    "c2": Config("c2", N=1, G=16, W=512, H=4, steps=2000, first_seed=2, init_active=64,
                 init_queue=512, len_mu=7.0, len_sigma=1.0,
                 arrival=("sin", 8.0, 6.0, 500), hazard=0.0, term_mode=2,
                 beta_ab=(2.0, 50.0)),
    # BR-0 batched, 4096 instances, per-instance Poisson rate in [4, 16]
    "c3": Config("c3", N=4096, G=32, W=256, H=0, steps=500, first_seed=100, init_active=32,
                 init_queue=256, len_mu=7.5, len_sigma=1.2, arrival=("uniform", 4.0, 16.0),
                 hazard=1.0 / 500.0, ctx_clip=(16, 131072)),
    # The paper's deployed setting (Section 5.1 "Our methods", Section 5.3 "Dispatch overhead"):
    # BR-H with H = 80 on G = 8 workers, R_max = 4, perfect-lookahead predictor from simulated
    # lifetimes; prompt and output lengths shaped like its traces (mean prompt ~4,000, mean output
    # ~1,100 tokens), near saturation
    "h80": Config("h80", N=1, G=8, W=512, H=80, steps=2000, first_seed=9000, init_active=64,
                  init_queue=64, len_mu=8.0, len_sigma=0.8, arrival=("const", 0.7),
                  hazard=0.0, term_mode=3, pred_mode=1, beta=48.0, gamma=0.9,
                  out_mu=6.5, out_sigma=1.0, ctx_clip=(16, 131072)),
    # BR-H batched, H=8, bursts of 200 every 250 steps, geometric mean 600
    "c4": Config("c4", N=1024, G=64, W=1024, H=8, steps=1000, first_seed=5000,
                 init_active=64, init_queue=1024, len_mu=8.0, len_sigma=1.5,
                 arrival=("const", 20.0), hazard=1.0 / 600.0, term_mode=1,
                 beta_ab=(2.0, 60.0), burst_every=250, burst_size=200,
                 ctx_clip=(16, 131072)),
}


def get_config(name: str, **overrides) -> Config:
    return replace(CONFIGS[name], **overrides).resolved()


# --------------------------------------------------------------------------
# a generated workload: tables + initial snapshot, all numpy
# --------------------------------------------------------------------------
@dataclass
class Workload:
    cfg: Config
    seeds: np.ndarray             # uint64 [N]
    len_tab: np.ndarray           # int32 [2^16] prompt lengths
    beta_tab: np.ndarray          # fp32 [2^16] classifier probabilities
    arr_cdf: np.ndarray           # uint32 [rows, ARR_LEN]
    arr_period: int
    arr_inst_stride: int          # row(inst, k) = inst * stride + k % period
    term_cdf: np.ndarray          # uint32 [B] gap thresholds of the constant hazard
    out_tab: Optional[np.ndarray] = None   # int32 [2^16] output lengths (term_mode 3)
    state: Dict[str, np.ndarray] = field(default_factory=dict)

    def arr_rows_for(self, inst: int) -> np.ndarray:
        r0 = inst * self.arr_inst_stride
        return np.ascontiguousarray(self.arr_cdf[r0:r0 + self.arr_period])


def _top16(z: np.ndarray) -> np.ndarray:
    return (z >> np.uint64(64 - TAB_LOG2)).astype(np.int64)


def make_workload(cfg: Config, n_instances: Optional[int] = None,
                  first_instance: int = 0) -> Workload:
    """Tables and the k = 0 snapshot for instances
    ``first_instance .. first_instance + n_instances`` of ``cfg``."""
    cfg = cfg.resolved()
    N = cfg.N if n_instances is None else n_instances
    G, B, W, H = cfg.G, cfg.B, cfg.W, cfg.H
    seeds = (np.arange(N, dtype=np.uint64) + np.uint64(cfg.first_seed + first_instance))

    len_tab = lognormal_table(cfg.len_mu, cfg.len_sigma, *cfg.len_clip)
    ctx_tab = lognormal_table(cfg.len_mu, cfg.len_sigma, *cfg.ctx_clip)
    btab = beta_table(*cfg.beta_ab)

    kind = cfg.arrival[0]
    if kind == "const":
        arr = poisson_thresholds([cfg.arrival[1]])
        period, stride = 1, 0
    elif kind == "sin":
        _, base, amp, period = cfg.arrival
        k = np.arange(period, dtype=np.float64)
        arr = poisson_thresholds(base + amp * np.sin(2.0 * math.pi * k / period))
        stride = 0
    elif kind == "uniform":
        _, lo, hi = cfg.arrival
        u = mix_np(seeds, STREAM_RATE, 0).astype(np.float64) / 18446744073709551616.0
        arr = poisson_thresholds(lo + (hi - lo) * u)
        period, stride = 1, 1
    else:
        raise ValueError(kind)

    # ---- initial snapshot -------------------------------------------------
    A = G * B
    slot = np.arange(A, dtype=np.uint64)[None, :]
    ctx = ctx_tab[_top16(mix_np(seeds[:, None], STREAM_INIT_CTX, slot))].reshape(N, G, B)
    occupied = (np.arange(B)[None, None, :] < cfg.init_active)
    act_base = np.where(occupied, ctx, EMPTY).astype(np.int32)
    words = (B + 63) // 64
    occ = np.zeros((N, G, words), dtype=np.uint64)
    for b in range(min(cfg.init_active, B)):
        occ[:, :, b // 64] |= np.uint64(1) << np.uint64(b % 64)
    nact = np.full((N, G), min(cfg.init_active, B), dtype=np.int32)
    load = np.where(occupied, ctx, 0).astype(np.int64).sum(axis=2)
    act_id = np.where(occupied, np.arange(A, dtype=np.uint32).reshape(1, G, B),
                      np.uint32(0xFFFFFFFF)).astype(np.uint32)
    act_id = np.broadcast_to(act_id, (N, G, B)).copy()

    qpos = np.arange(W, dtype=np.uint64)[None, :]
    q_s = len_tab[_top16(mix_np(seeds[:, None], STREAM_INIT_QUEUE, qpos))].astype(np.int32)
    q_valid = np.arange(W)[None, :] < cfg.init_queue
    wq_s = np.where(q_valid, q_s, 0).astype(np.int32)
    wq_id = np.where(q_valid, (A + np.arange(W)).astype(np.uint32)[None, :],
                     np.uint32(0)).astype(np.uint32)
    wq_id = np.broadcast_to(wq_id, (N, W)).copy()
    wq_n = np.full((N,), cfg.init_queue, dtype=np.int32)

    # predictor state: every running request starts at the anchor H with a
    # staggered age since its last refresh (as if admitted at different steps)
    tau0 = (mix_np(seeds[:, None], STREAM_INIT_TAU, slot) >> np.uint64(40)).astype(np.int64)
    tau0 = (tau0 % max(1, cfg.delta_T)).reshape(N, G, B)
    act_chat0 = np.full((N, G, B), float(H), dtype=np.float32)
    act_kref = ((-tau0) & 255).astype(np.uint8)

    out_tab = None
    extra = {}
    if cfg.term_mode == 3:
        # every request carries its output length; a running request has a uniformly drawn part
        # of its own still ahead, a waiting one all of it
        out_tab = lognormal_table(cfg.out_mu, cfg.out_sigma, *cfg.out_clip)
        z = mix_np(seeds[:, None], STREAM_INIT_END, slot)
        o_run = out_tab[_top16(z)].astype(np.int64)
        frac = ((z >> np.uint64(16)) & np.uint64(0xFFFF)).astype(np.int64)
        act_end = ((o_run * frac) >> 16).reshape(N, G, B)            # last step of the request, in [0, o)
        extra["act_end"] = np.where(occupied, act_end, 0).astype(np.int32)
        q_o = out_tab[_top16(mix_np(seeds[:, None], STREAM_INIT_QO, qpos))].astype(np.int32)
        extra["wq_o"] = np.where(q_valid, q_o, 0).astype(np.int32)

    state = dict(
        act_base=act_base, occ=occ, nact=nact, load=load, act_id=act_id,
        act_chat0=act_chat0, act_kref=act_kref,
        wq_s=wq_s, wq_id=wq_id, wq_n=wq_n,
        step=np.zeros((N,), dtype=np.int32),
        seed=seeds.copy(),
        next_id=np.full((N,), A + cfg.init_queue, dtype=np.uint32),
    )
    state.update(extra)
    return Workload(cfg=cfg, seeds=seeds, len_tab=len_tab, beta_tab=btab, arr_cdf=arr,
                    arr_period=period, arr_inst_stride=stride,
                    term_cdf=termination_gap_thresholds(cfg.hazard, B), out_tab=out_tab, state=state)


# --------------------------------------------------------------------------
# stand-in termination classifier: probabilities for decode step k
# --------------------------------------------------------------------------
def term_probs_np(wl: Workload, k: int, instances=None) -> np.ndarray:
    """fp32 [n, G, B, H]: i.i.d. table draws per (instance, step, slot, h)."""
    cfg = wl.cfg
    seeds = wl.seeds if instances is None else wl.seeds[np.asarray(instances)]
    per_step = cfg.G * cfg.B * cfg.H
    idx = np.uint64(k) * np.uint64(per_step) + np.arange(per_step, dtype=np.uint64)[None, :]
    z = mix_np(seeds[:, None], STREAM_PROBS, idx)
    return wl.beta_tab[_top16(z)].reshape(len(seeds), cfg.G, cfg.B, cfg.H)


def term_probs_torch(wl: Workload, k: int, device, seeds_t=None, tab_t=None, out=None):
    """Same values as :func:`term_probs_np`, produced on ``device`` with torch
    integer ops (input generation only; not part of the routing path)."""
    import torch

    cfg = wl.cfg
    if seeds_t is None:
        seeds_t = torch.from_numpy(wl.seeds.astype(np.int64)).to(device)
    if tab_t is None:
        tab_t = torch.from_numpy(wl.beta_tab).to(device)
    per_step = cfg.G * cfg.B * cfg.H
    idx = torch.arange(per_step, dtype=torch.int64, device=device)[None, :] + k * per_step
    z = mix_torch(seeds_t[:, None], STREAM_PROBS, idx)
    sel = (z >> (64 - TAB_LOG2)) & ((1 << TAB_LOG2) - 1)
    res = tab_t[sel].reshape(seeds_t.shape[0], cfg.G, cfg.B, cfg.H)
    if out is not None:
        out.copy_(res)
        return out
    return res
