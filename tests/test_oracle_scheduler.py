"""Pins for the oracle's SlowFast scheduler (Section 3.3, Algorithm 1): hand-derived traces, closed forms,
invariants, the step machine against the loop, and the special case that reduces to low-confidence
remasking (Section 3.1)."""
import glob
import math
import os
import random
import statistics

import pytest

from oracle.scheduler import (FAST, QBITS, SLOW, SlowFastParams, SlowFastState, exceeds, rows_needed,
                              slowfast_loop, slowfast_step, top_k, variance_below)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def sq_of(conf: float) -> int:
    return max(1 << QBITS, int(round((1 << QBITS) / conf)))


def parse_fixture(path):
    L, default, params, confs, expect = None, 0.01, {}, {}, []
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "L":
            L = int(tok[1])
        elif tok[0] == "default":
            default = float(tok[1])
        elif tok[0] == "param":
            params[tok[1]] = type(getattr(SlowFastParams(), tok[1]))(float(tok[2]))
        elif tok[0] == "conf":
            confs[int(tok[1])] = {int(a.split(":")[0]): float(a.split(":")[1]) for a in tok[2:]}
        elif tok[0] == "expect":
            bar = tok.index("|")
            expect.append((tuple(int(v) for v in tok[1:bar]), tuple(int(v) for v in tok[bar + 1:])))
    return L, default, SlowFastParams(**params), confs, expect


def scripted_predict(confs, default):
    step = [0]

    def predict(masked, rows):
        table = confs.get(step[0], {})
        step[0] += 1
        a = {i: 100 + i for i in rows}
        sq = {i: sq_of(table.get(i, default)) for i in rows}
        return a, sq
    return predict


@pytest.mark.parametrize("path", sorted(glob.glob(os.path.join(GOLDEN, "trace_*.txt"))))
def test_hand_traces(path):
    L, default, p, confs, expect = parse_fixture(path)
    y, trace = slowfast_loop(L, scripted_predict(confs, default), p)
    got = [((r.step, r.phase, r.s, r.hi, r.e_cand, r.stable), tuple(r.positions)) for r in trace]
    assert got == expect
    assert y == [100 + i for i in range(L)]


def test_variance_closed_form_w2():
    # W_hist = 2: population variance (a-b)^2/4, so "below 1" <=> |a-b| <= 1 (and the same for the sample variance (a-b)^2/2)
    for a in range(0, 40):
        for b in range(0, 40):
            assert variance_below([a, b], 1.0) == (abs(a - b) <= 1)


def test_variance_against_library():
    rng = random.Random(0)
    for _ in range(2000):
        n = rng.randint(1, 6)
        H = [rng.randint(0, 600) for _ in range(n)]
        sigma2 = rng.choice([0.3, 1.0, 2.5, 100.0, 5000.0])
        ref = statistics.pvariance(H)
        if abs(ref - sigma2) > 1e-9:
            assert variance_below(H, sigma2) == (ref < sigma2)
    assert variance_below([3], 1.0) and variance_below([0, 1000], math.inf)
    assert not variance_below([5, 5], 0.0)            # strict "<"


def test_thresholds_are_strict_and_canonical():
    one = 1 << QBITS
    assert exceeds(one, 0.85) and not exceeds(one, 1.0)            # c = 1 exceeds 0.85, not 1.0 (strict)
    assert exceeds(2 * one - 1, 0.5) and not exceeds(2 * one, 0.5)  # c = 1/2 does not exceed 0.5
    # the comparison uses float32(tau) widened to double, not the decimal literal
    import struct
    tau32 = struct.unpack("f", struct.pack("f", 0.1))[0]
    assert exceeds(10 * one, 0.1) == (float(10 * one) * tau32 < float(one))
    # around c = 0.1 the two readings part: float32(0.1) = 0.1 + 1.49e-9 moves the boundary by 40 units of S_q
    from fractions import Fraction
    flips = 0
    for sq in range(10 * one - 60, 10 * one + 5):
        want = Fraction(sq) * Fraction(tau32) < one               # exact rational arithmetic on the float the ABI carries
        assert exceeds(sq, 0.1) == want, sq
        flips += want != (Fraction(sq) * Fraction(1, 10) < one)
    assert flips >= 30                                            # the window really separates the readings


def test_top_k_ties_to_smaller_position():
    sq = {3: 50, 1: 50, 7: 40, 5: 60}
    assert top_k([1, 3, 5, 7], sq, 1) == [7]
    assert top_k([1, 3, 5, 7], sq, 2) == [1, 7]
    assert top_k([1, 3, 5, 7], sq, 3) == [1, 3, 7]
    assert top_k([1, 3, 5, 7], sq, 9) == [1, 3, 5, 7]


def random_process(L, seed, hot=0.3):
    """A seeded confidence process: per step, per position, a confidence with a mix of high and low values."""
    rng = random.Random(seed)

    def predict(masked, rows):
        a, sq = {}, {}
        for i in rows:
            u = rng.random()
            c = rng.uniform(0.86, 0.999) if u < hot else (rng.uniform(0.1, 0.85) if u < 0.6 else rng.uniform(1e-4, 0.1))
            a[i] = rng.randrange(0, 50000)
            sq[i] = sq_of(c)
        return a, sq
    return predict


def drive_step_machine(L, predict, p):
    st = SlowFastState.fresh(L, p)
    y = [None] * L
    trace = []
    while not st.done:
        rows = rows_needed(st)
        assert rows, "an active sequence must need at least one row"
        a, sq = predict(list(st.masked), rows)
        before = list(st.masked)
        rec = slowfast_step(st, a, sq, p)
        for i, t in zip(rec.positions, rec.tokens):
            assert before[i] and not st.masked[i]
            y[i] = t
        # never re-masked
        assert all(before[i] or not st.masked[i] for i in range(L))
        # everything left of s_cycle is decoded
        assert not any(st.masked[: st.s_cycle])
        trace.append(rec)
    return y, trace


@pytest.mark.parametrize("seed", range(40))
def test_invariants_and_step_machine_equals_loop(seed):
    rng = random.Random(1000 + seed)
    L = rng.choice([1, 2, 3, 7, 16, 33, 64, 100])
    p = SlowFastParams(k_max=rng.choice([1, 2, 3, 8]), w_hist=rng.choice([1, 2, 3]),
                       sigma2_stable=rng.choice([0.2, 1.0, 30.0]), k_slow=rng.choice([1, 2, 4]),
                       k_fast=rng.choice([1, 3]), max_steps=rng.choice([0, 0, L // 2 + 1, 2 * L]),
                       min_high_count=rng.choice([1, 1, 3]))
    N = p.max_steps if p.max_steps > 0 else L
    y1, t1 = slowfast_loop(L, random_process(L, seed), p)
    y2, t2 = drive_step_machine(L, random_process(L, seed), p)
    assert [r.key() for r in t1] == [r.key() for r in t2]
    assert y1 == y2
    assert all(v is not None for v in y1)                      # no mask left
    assert 1 <= len(t1) <= N                                   # terminates within N steps
    seen = [i for r in t1 for i in r.positions]
    assert sorted(seen) == list(range(L))                      # each position decoded exactly once
    assert all(len(r.positions) >= 1 for r in t1)              # every step makes progress


def test_reduces_to_low_confidence_remasking():
    """tau_min < 0 makes the span the whole window, tau_high > 1 disables parallel unmasking, K_max = W = 1:
    every step then unmasks the single most confident masked token, which is LLaDA's low-confidence
    remasking with N = L (n_un grows by one per step)."""
    L = 24
    p = SlowFastParams(tau_min_conf=-1.0, tau_high_conf=2.0, sigma2_stable=math.inf, k_max=1, w_hist=1)
    order = []
    rng = random.Random(7)
    table = {}

    def predict(masked, rows):
        a, sq = {}, {}
        for i in rows:
            table[i] = rng.uniform(0.01, 0.99)
            a[i], sq[i] = i, sq_of(table[i])
        # the textbook rule, stated independently: most confident masked position
        cands = [i for i in range(L) if masked[i]]
        order.append(max(cands, key=lambda i: (table.get(i, -1.0) if i in rows else -1.0, -i)))
        return a, sq

    y, trace = slowfast_loop(L, predict, p)
    assert len(trace) == L
    assert [r.positions for r in trace[:-1]] == [[o] for o in order[:-1]]


def test_two_separated_blocks_are_both_accelerated():
    """Appendix case study scenario: two high-confidence blocks separated by an uncertain gap.  Both blocks
    must be decoded by parallel (fast) steps, and the whole sequence in far fewer than L steps."""
    L = 32
    hot = set(range(0, 8)) | set(range(16, 24))

    def predict(masked, rows):
        return {i: i for i in rows}, {i: sq_of(0.97 if i in hot else 0.02) for i in rows}

    y, trace = slowfast_loop(L, predict, SlowFastParams())
    # the end point jumps over the gap to the far block (e_cand = 23 twice -> span [0,24)), and one fast
    # step unmasks every confident token of both blocks at once; the gap then falls back to top-1 steps
    par = [r for r in trace if r.phase == FAST and len(r.positions) >= 4]
    assert len(par) == 1 and set(par[0].positions) == hot - {0, 1} and (par[0].s, par[0].hi) == (0, 24)
    assert [r.positions for r in trace[:2]] == [[0], [1]] and trace[1].stable == 1
    assert len(trace) < L - 6


def test_empty_and_single():
    y, t = slowfast_loop(0, lambda m, r: ({}, {}), SlowFastParams())
    assert y == [] and t == []
    y, t = slowfast_loop(1, lambda m, r: ({0: 9}, {0: sq_of(0.5)}), SlowFastParams())
    assert y == [9] and len(t) == 1 and t[0].positions == [0]
