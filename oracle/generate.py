"""ORACLE (test infrastructure): the iterative denoising loop (Section 3.1, Eqs. 1-4) with the SlowFast
transition rule (Section 3.3, Algorithm 1), glued from forward.py, rowstats.py and scheduler.py.

`generate` runs the oracle's own predictor at every step.  `replay` is the teacher-forced variant: the
logits of every step are supplied by the caller (e.g. read back from another implementation), and only
row statistics and selection are the oracle's.
"""
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np

from . import forward as F
from . import rowstats as RS
from .scheduler import (SlowFastParams, SlowFastState, StepRecord, rows_needed, slowfast_step)


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
