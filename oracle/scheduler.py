"""ORACLE (test infrastructure): the SlowFast transition rule S of Section 3.3 / Algorithm 1, in pure Python.

Two statements of the same rule live here:

* `slowfast_loop`  — the whole sampling loop: cycles of an exploratory stage (`_Sampler.explore`) and an
  accelerated stage (`_Sampler.accelerate`), each asking a `predict` callback for the greedy tokens and
  confidences of the rows it reads (Algorithm 1; Section 3.3).
* `slowfast_step`  — the same rule as a one-step state machine (what a per-step entry point needs); the
  test-suite checks that driving it step by step reproduces `slowfast_loop` exactly.

Notation follows the paper, 0-based: response positions i in [0, L), window [s_cycle, L), span
[s_cycle, hi) with hi = e_cycle + 1.  Confidence comparisons are taken on the canonical fixed-point
softmax denominator S_q (see rowstats.c): "c_i > tau" is `float64(S_q) * float64(float32(tau)) < 2^28`,
and "larger confidence" is "smaller S_q", ties to the smaller position.

Readings where the paper is silent or at odds with itself (each is listed in the design notes):
  R1  Variance (Sec. 3.3 stability check) is the population variance of the window, evaluated exactly in
      integers:  n*sum(e^2) - (sum e)^2  <  sigma2 * n^2.
  R2  e_cycle = floor(mean(H_W)) on a stable exit (Eq. for e_cycle, Alg. 1 "Mean(H_W)"); the last
      e_cand when K_max is reached without stability (Alg. 1 fallback).
  R3  If no position exceeds tau_min_conf, e_cand is the first masked position of the window.
  R4  Only masked positions compete for e_cand and for the top-k; the statistics are those predicted
      before this step's unmasking.
  R5  H_W is cleared at the start of every exploratory stage.
  R6  The accelerated stage repeats until no masked position is left in [s_cycle, hi).
  R7  The outer loop runs while a masked position remains and k > 0.
  R8  The exploratory step's state update is the top-k_slow unmasking; on the last permitted step
      (k == 1) every position still masked is unmasked (n_un = L at k = 1 in the low-confidence rule).
  R9  Fast steps read only in-span rows, so predictions outside the span may be skipped.
  R10 k_slow = k_fast = 1 by default; R11 fallback iff |S_high| < min_high_count (default 1).
  R12 Both thresholds are strict ">", the variance test strict "<".
"""
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence, Tuple

QBITS = 28
SLOW, FAST = 0, 1


@dataclass
class SlowFastParams:
    tau_min_conf: float = 0.1      # Section 4.2 defaults
    tau_high_conf: float = 0.85
    sigma2_stable: float = 1.0
    k_max: int = 8
    w_hist: int = 2
    k_slow: int = 1
    k_fast: int = 1
    max_steps: int = 0             # N; 0 means N = L
    min_high_count: int = 1
    # Alternative readings of the passages where the paper is at odds with itself, honoured by `slowfast_loop` only (the
    # step machine, and every other implementation, use the defaults):
    e_cycle_rule: str = "floor_mean"   # R2: "floor_mean" (equation, Algorithm 1) or "last_candidate" (the prose after it)
    reset_history: bool = True         # R5: False keeps H_W across cycles, as Algorithm 1 initialises it only once
    fast_single_step: bool = False     # R6: True takes ONE accelerated step per cycle, as Algorithm 1 prints it; masked
                                       #     positions left behind s_cycle are then never revisited before the last step


def _f32(x: float) -> float:
    import struct
    return struct.unpack("f", struct.pack("f", x))[0]


def exceeds(sq: int, tau: float) -> bool:
    """c > tau on the canonical value: one IEEE double multiply, compared with 2^QBITS."""
    return float(int(sq)) * _f32(tau) < float(1 << QBITS)


def variance_below(H: Sequence[int], sigma2: float) -> bool:
    """Population variance of H strictly below sigma2, in exact integer arithmetic on the left."""
    n = len(H)
    num = n * sum(e * e for e in H) - sum(H) ** 2          # = n^2 * Var_pop(H), an integer
    return float(num) < _f32(sigma2) * float(n * n)


def top_k(cands: Sequence[int], sq: Dict[int, int], k: int) -> List[int]:
    """The k most confident candidates: smallest S_q first, equal S_q -> smaller position first."""
    return sorted(sorted(cands, key=lambda i: (int(sq[i]), i))[: max(k, 0)])


@dataclass
class StepRecord:
    step: int
    phase: int
    s: int
    hi: int                 # span end of the step (L for an exploratory step: its window is [s, L))
    e_cand: int             # -1 on accelerated steps and on the forced last step
    stable: int
    positions: List[int]
    tokens: List[int]

    def key(self) -> Tuple:
        return (self.step, self.phase, self.s, self.hi, self.e_cand, self.stable,
                tuple(self.positions), tuple(self.tokens))


Predict = Callable[[List[bool], List[int]], Tuple[Dict[int, int], Dict[int, int]]]
# predict(masked, rows) -> (a, sq): greedy token and S_q for (at least) the positions in `rows`.


class _Sampler:
    """Bookkeeping shared by the two stages of a cycle: which positions are still masked, the tokens
    written so far, the remaining step budget k and the trace."""

    def __init__(self, L: int, predict: Predict, p: SlowFastParams):
        self.L, self.predict, self.p = L, predict, p
        self.masked = [True] * L
        self.y: List[Optional[int]] = [None] * L
        self.k = p.max_steps if p.max_steps > 0 else L          # Algorithm 1, initialisation: k = N
        self.trace: List[StepRecord] = []
        self.H_kept: List[int] = []

    def open_positions(self, lo: int, hi: int) -> List[int]:
        return [i for i in range(lo, hi) if self.masked[i]]

    def commit(self, phase: int, s: int, hi: int, e_cand: int, stable: bool, chosen: List[int], a: Dict[int, int]):
        """Writes the greedy tokens of `chosen`, records the step and spends one step of the budget."""
        for i in chosen:
            assert self.masked[i], "a decoded position was selected again"
            self.masked[i] = False
            self.y[i] = int(a[i])
        self.trace.append(StepRecord(len(self.trace), phase, s, hi, e_cand, int(stable), chosen, [int(a[i]) for i in chosen]))
        self.k -= 1

    def last_step(self, phase: int, s: int, hi: int) -> None:
        """R8: the final permitted step decodes whatever is still masked."""
        rest = self.open_positions(0, self.L)
        a, _ = self.predict(list(self.masked), rest)
        self.commit(phase, s, hi, -1, False, rest, a)

    def explore(self, s: int) -> Optional[int]:
        """Section 3.3, exploratory stage from window start s.  Returns the span end hi = e_cycle + 1, or None when
        the sequence (or the budget) ended inside the stage."""
        p, L = self.p, self.L
        H: List[int] = [] if p.reset_history else self.H_kept     # R5: a fresh history per stage
        e_cand = -1
        for _ in range(p.k_max):
            if self.k == 0 or not any(self.masked) or not self.open_positions(s, L):
                return None
            if self.k == 1:
                self.last_step(SLOW, s, L)
                return None
            M = self.open_positions(s, L)
            a, sq = self.predict(list(self.masked), M)
            reach = [i for i in M if exceeds(sq[i], p.tau_min_conf)]
            e_cand = reach[-1] if reach else M[0]                 # end point of convergence; R3 when nothing reaches tau_min
            H = (H + [e_cand])[-p.w_hist:]
            self.H_kept = H
            stable = len(H) >= p.w_hist and variance_below(H, p.sigma2_stable)
            self.commit(SLOW, s, L, e_cand, stable, top_k(M, sq, p.k_slow), a)
            if stable:
                if p.e_cycle_rule == "last_candidate":
                    return e_cand + 1
                return sum(H) // len(H) + 1                       # R2: floor of the window's mean
        return e_cand + 1                                         # K_max steps without stability (Algorithm 1's fallback)

    def accelerate(self, s: int, hi: int) -> None:
        """Section 3.3, accelerated stage on the span [s, hi); R6: repeated until the span holds no mask."""
        p = self.p
        while self.k > 0 and any(self.masked[s:hi]):
            if self.k == 1:
                self.last_step(FAST, s, hi)
                return
            F = self.open_positions(s, hi)
            a, sq = self.predict(list(self.masked), F)
            high = [i for i in F if exceeds(sq[i], p.tau_high_conf)]
            chosen = high if len(high) >= p.min_high_count else top_k(F, sq, p.k_fast)
            self.commit(FAST, s, hi, -1, False, chosen, a)
            if p.fast_single_step:
                return


def slowfast_loop(L: int, predict: Predict, p: SlowFastParams) -> Tuple[List[Optional[int]], List[StepRecord]]:
    """The whole sampling loop of Algorithm 1 under the readings R1-R12: cycles of an exploratory stage that
    locates the span and an accelerated stage that decodes it.  Returns (tokens, trace)."""
    run = _Sampler(L, predict, p)
    s_cycle = 0
    while run.k > 0 and any(run.masked):                          # R7
        if not run.open_positions(s_cycle, L):
            # only reachable under fast_single_step: the window has run off the end with masks left behind it;
            # Algorithm 1 as printed stops here (s_cycle >= L) and returns a sequence that still holds masks
            break
        hi = run.explore(s_cycle)
        if hi is None or run.k == 0 or not any(run.masked):
            break
        run.accelerate(s_cycle, hi)
        s_cycle = hi                                              # the next cycle starts behind the decoded span
    return run.y, run.trace


# ----------------------------------------------------------------------------------------------------
# the same rule, one step at a time
# ----------------------------------------------------------------------------------------------------
@dataclass
class SlowFastState:
    L: int
    k: int                       # steps still permitted
    phase: int = SLOW
    s_cycle: int = 0
    hi: int = 0                  # meaningful in the fast phase
    step_count: int = 0          # exploratory steps taken in this cycle
    H: List[int] = field(default_factory=list)
    masked: List[bool] = field(default_factory=list)
    steps_done: int = 0
    done: bool = False

    @staticmethod
    def fresh(L: int, p: SlowFastParams) -> "SlowFastState":
        return SlowFastState(L=L, k=(p.max_steps if p.max_steps > 0 else L), masked=[True] * L, done=(L == 0))


def rows_needed(st: SlowFastState) -> List[int]:
    """Response positions whose prediction the next step reads."""
    if st.done:
        return []
    if st.k == 1:
        return [i for i in range(st.L) if st.masked[i]]
    if st.phase == SLOW:
        return [i for i in range(st.s_cycle, st.L) if st.masked[i]]
    return [i for i in range(st.s_cycle, st.hi) if st.masked[i]]


def slowfast_step(st: SlowFastState, a: Dict[int, int], sq: Dict[int, int], p: SlowFastParams) -> Optional[StepRecord]:
    """Apply one denoising step's decisions to `st` in place.  `a`, `sq` cover rows_needed(st)."""
    if st.done:
        return None
    assert p.e_cycle_rule == "floor_mean" and p.reset_history and not p.fast_single_step, "the step machine takes the default readings"
    L = st.L
    rec_step = st.steps_done
    if st.k == 1:
        rest = [i for i in range(L) if st.masked[i]]
        rec = StepRecord(rec_step, st.phase, st.s_cycle, L if st.phase == SLOW else st.hi, -1, 0,
                         rest, [int(a[i]) for i in rest])
        for i in rest:
            st.masked[i] = False
        st.k = 0
        st.steps_done += 1
        st.done = True
        return rec

    if st.phase == SLOW:
        M = [i for i in range(st.s_cycle, L) if st.masked[i]]
        above = [i for i in M if exceeds(sq[i], p.tau_min_conf)]
        e_cand = max(above) if above else min(M)
        chosen = top_k(M, sq, p.k_slow)
        for i in chosen:
            st.masked[i] = False
        st.H = (st.H + [e_cand])[-p.w_hist:]
        st.k -= 1
        st.step_count += 1
        stable = len(st.H) >= p.w_hist and variance_below(st.H, p.sigma2_stable)
        rec = StepRecord(rec_step, SLOW, st.s_cycle, L, e_cand, int(stable), chosen, [int(a[i]) for i in chosen])
        if stable:
            st.phase, st.hi = FAST, sum(st.H) // len(st.H) + 1
        elif st.step_count >= p.k_max:
            st.phase, st.hi = FAST, e_cand + 1
    else:
        F = [i for i in range(st.s_cycle, st.hi) if st.masked[i]]
        S_high = [i for i in F if exceeds(sq[i], p.tau_high_conf)]
        chosen = S_high if len(S_high) >= p.min_high_count else top_k(F, sq, p.k_fast)
        for i in chosen:
            st.masked[i] = False
        st.k -= 1
        rec = StepRecord(rec_step, FAST, st.s_cycle, st.hi, -1, 0, chosen, [int(a[i]) for i in chosen])

    st.steps_done += 1
    if not any(st.masked) or st.k == 0:
        st.done = True
    elif st.phase == FAST and not any(st.masked[st.s_cycle:st.hi]):
        # the span is fully decoded: next cycle starts behind it with an empty history
        st.s_cycle, st.phase, st.H, st.step_count = st.hi, SLOW, [], 0
    return rec
