"""ORACLE (test infrastructure): the iterative denoising loop (Section 3.1, Eqs. 1-4) with the SlowFast
transition rule (Section 3.3, Algorithm 1), glued from forward.py, rowstats.py and scheduler.py.

`generate` runs the oracle's own predictor at every step; `generate_cached` does the same with the feature
cache of cache.py in front of the predictor (the combination of Table 4).  `replay` is the teacher-forced
variant: the logits of every step are supplied by the caller (e.g. read back from another implementation),
and only row statistics and selection are the oracle's.
"""
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np

from . import cache as C
from . import forward as F
from . import rowstats as RS
from .scheduler import (FAST, SlowFastParams, SlowFastState, StepRecord, rows_needed, slowfast_step)


def _stats_for(logits: np.ndarray, rows: Sequence[int]) -> Tuple[Dict[int, int], Dict[int, int]]:
    st = RS.row_stats(logits)
    a = {i: int(st["argmax"][j]) for j, i in enumerate(rows)}
    sq = {i: int(st["sq"][j]) for j, i in enumerate(rows)}
    return a, sq


def generate(cfg: F.ModelConfig, w: Dict, prompt: Sequence[int], L: int, p: SlowFastParams,
             dtype=np.float64, logits_hook: Optional[Callable] = None):
    """One sequence: prompt (list of ids), L response positions.  Returns (tokens[P+L], trace, states)."""
    P = len(prompt)
    y = list(prompt) + [cfg.mask_id] * L                     # y^(N): all [MASK]
    st = SlowFastState.fresh(L, p)
    trace: List[StepRecord] = []
    while not st.done:
        rows = rows_needed(st)
        logits = F.forward(cfg, w, np.asarray([y]), rows=[(0, P + i) for i in rows], dtype=dtype)
        logits32 = np.ascontiguousarray(logits, dtype=np.float32)
        if logits_hook is not None:
            logits_hook(len(trace), rows, logits32)
        a, sq = _stats_for(logits32, rows)
        rec = slowfast_step(st, a, sq, p)
        for i, t in zip(rec.positions, rec.tokens):
            y[P + i] = t
        trace.append(rec)
    return y, trace


def generate_cached(cfg: F.ModelConfig, w: Dict, prompt: Sequence[int], L: int, p: SlowFastParams,
                    k_prompt: int, k_response: int, rho: float, dtype=np.float64,
                    logits_hook: Optional[Callable] = None, select: Optional[Callable] = None,
                    record_hook: Optional[Callable] = None):
    """`generate` with the feature cache (cache.py) in front of the predictor: the cache's step counter starts at 0
    with the generation (so the first step recomputes everything); an accelerated step hands its span [s_cycle, hi)
    to the cache as the candidate set, an exploratory step the whole response.  `select(step, layer, sims, cand)`
    forces the adaptive sets of a step; `record_hook(step, record)` receives the per-layer sets and similarities."""
    P = len(prompt)
    y = list(prompt) + [cfg.mask_id] * L
    st = SlowFastState.fresh(L, p)
    cache = C.FeatureCache(cfg, P + L, dtype)
    trace: List[StepRecord] = []
    while not st.done:
        step = len(trace)
        rows = rows_needed(st)
        span = (st.s_cycle, st.hi) if st.phase == FAST else None
        rec_c: Dict = {}
        forced = (lambda l, sims, cand, _s=step: select(_s, l, sims, cand)) if select is not None else None
        logits = C.cached_forward(cfg, w, np.asarray(y), P, cache, k_prompt, k_response, rho, span=span,
                                  rows=[P + i for i in rows], select=forced, record=rec_c)
        if record_hook is not None:
            record_hook(step, rec_c)
        logits32 = np.ascontiguousarray(logits, dtype=np.float32)
        if logits_hook is not None:
            logits_hook(step, rows, logits32)
        a, sq = _stats_for(logits32, rows)
        rec = slowfast_step(st, a, sq, p)
        for i, t in zip(rec.positions, rec.tokens):
            y[P + i] = t
        trace.append(rec)
    return y, trace


def replay(L: int, p: SlowFastParams, logits_for_step: Callable[[int, List[int]], np.ndarray]):
    """Teacher-forced loop: logits_for_step(step, rows) -> [len(rows), V] float32 or uint16(bf16 bits)."""
    st = SlowFastState.fresh(L, p)
    y: List[Optional[int]] = [None] * L
    trace: List[StepRecord] = []
    while not st.done:
        rows = rows_needed(st)
        a, sq = _stats_for(logits_for_step(len(trace), rows), rows)
        rec = slowfast_step(st, a, sq, p)
        for i, t in zip(rec.positions, rec.tokens):
            y[i] = t
        trace.append(rec)
    return y, trace
