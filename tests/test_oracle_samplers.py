"""Pins for the oracle's LLaDA sampling strategies (Section 3.1: random, low-confidence and semi-autoregressive remasking):
the generator against its published known-answer vectors, the unmask counts against the closed form of the noise schedule,
the literal "n_un highest confidences over ALL positions, decoded ones at confidence 1" against the restated rule, blocks
strictly left to right, and the step machine against the whole-loop statement."""
import random
from fractions import Fraction

import pytest

from oracle import samplers as SM
from oracle.scheduler import QBITS, SlowFastParams, slowfast_loop


def sq_of(conf: float) -> int:
    return max(1 << QBITS, int(round((1 << QBITS) / conf)))


def random_process(L, seed):
    """predict callback with fresh random confidences in (0, 1) at every call; token at position i is 100 + i."""
    rng = random.Random(seed)
    calls = []

    def predict(masked, rows):
        calls.append(list(rows))
        return {i: 100 + i for i in rows}, {i: sq_of(rng.uniform(0.01, 0.99)) for i in rows}
    return predict, calls


def test_philox_known_answers():
    """The three known-answer vectors published with the generator (Random123 distribution, philox4x32 with 10 rounds)."""
    assert SM.philox4x32_10((0, 0, 0, 0), (0, 0)) == (0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8)
    assert SM.philox4x32_10((0xFFFFFFFF,) * 4, (0xFFFFFFFF,) * 2) == (0x408F276D, 0x41C83B0E, 0xA20BC7C6, 0x6D5451FD)
    assert SM.philox4x32_10((0x243F6A88, 0x85A308D3, 0x13198A2E, 0x03707344), (0xA4093822, 0x299F31D0)) == \
        (0xD16CFE09, 0x94FDCCEB, 0x5001E420, 0x24126EA1)


def test_philox_is_a_bijection_on_a_small_slice_and_depends_on_every_input():
    base = SM.philox4x32_10((1, 2, 3, 4), (5, 6))
    seen = {base}
    for w in range(4):
        c = [1, 2, 3, 4]; c[w] ^= 1
        seen.add(SM.philox4x32_10(c, (5, 6)))
    seen.add(SM.philox4x32_10((1, 2, 3, 4), (4, 6)))
    seen.add(SM.philox4x32_10((1, 2, 3, 4), (5, 7)))
    assert len(seen) == 7
    assert len({SM.philox4x32_10((i, 0, 0, 0), (9, 9)) for i in range(2000)}) == 2000


@pytest.mark.parametrize("L,N", [(16, 16), (16, 4), (10, 4), (7, 3), (12, 24), (1, 1), (5, 1)])
def test_low_confidence_unmask_counts_follow_the_noise_schedule(L, N):
    predict, _ = random_process(L, L * 100 + N)
    y, trace = SM.low_confidence_remasking(L, N, predict)
    unmasked = 0
    for rec in trace:
        k = N - rec.step
        unmasked += len(rec.positions)
        assert unmasked == int(Fraction(L) * (1 - Fraction(k - 1, N)) // 1)       # floor(L (1 - t_{k-1}))
    assert len(trace) <= N and all(t == 100 + i for i, t in enumerate(y))


def test_low_confidence_equals_the_literal_rule_over_all_positions():
    """The paper's wording: rank ALL positions by confidence, decoded ones at 1, keep the n_un best.  Brute force on floats."""
    L, N = 12, 5
    rng = random.Random(3)
    confs = {}

    def predict(masked, rows):
        c = {i: rng.uniform(0.05, 0.95) for i in rows}
        confs[len(confs)] = c
        return {i: i for i in rows}, {i: sq_of(c[i]) for i in rows}

    y, trace = SM.low_confidence_remasking(L, N, predict)
    decoded = set()
    for rec in trace:
        k = N - rec.step
        c_all = {i: (1.0 if i in decoded else confs[rec.step][i]) for i in range(L)}
        n_un = (L * (N - k + 1)) // N
        keep = set(sorted(range(L), key=lambda i: (-c_all[i], i))[:n_un])
        assert decoded <= keep                              # decoded positions rank first
        assert sorted(keep - decoded) == rec.positions
        decoded |= keep


def test_low_confidence_with_one_token_per_step_is_the_slowfast_special_case():
    """SlowFast that never leaves the exploratory stage (K_max beyond the budget, a variance threshold nothing meets) unmasks
    the single most confident masked position per step — low-confidence remasking with N = L — computed here by the two
    independent functions on the same confidence process."""
    L = 20
    p1, _ = random_process(L, 77)
    p2, _ = random_process(L, 77)
    y1, t1 = SM.low_confidence_remasking(L, L, p1)
    y2, t2 = slowfast_loop(L, p2, SlowFastParams(k_max=10 ** 6, sigma2_stable=0.0, k_slow=1))
    assert y1 == y2 and [r.positions for r in t1] == [r.positions for r in t2]


def test_random_remasking_expected_counts_and_last_step():
    L, N = 64, 8
    totals = [0.0] * N
    runs = 300
    for seed in range(runs):
        predict, _ = random_process(L, seed)
        y, trace = SM.random_remasking(L, N, predict, seed=seed * 7919 + 1)
        assert all(t is not None for t in y)                # the step k = 1 unmasks whatever is left
        left = L
        for rec in trace:
            left -= len(rec.positions)
            totals[rec.step] += left
        for s in range(len(trace), N):                      # stopped early: nothing masked from there on
            totals[s] += 0
    for s in range(N):
        k = N - s
        expect = L * (k - 1) / N                            # E[masked after step k] = L t_{k-1}
        assert abs(totals[s] / runs - expect) <= 0.08 * L / N + 0.5, (s, totals[s] / runs, expect)


def test_random_draw_is_the_integer_threshold_on_the_first_output_word():
    for k in (1, 2, 3, 7, 256):
        for pos in range(50):
            u = SM.philox4x32_10((pos, 4, 2, 0), (0xDEADBEEF, 0x12345))[0]
            assert SM.random_unmask(0x12345DEADBEEF, 2, 4, pos, k) == (u < -(-(1 << 32) // k))
    assert all(SM.random_unmask(5, 0, s, i, 1) for s in range(3) for i in range(40))      # k = 1: probability 1


def test_a_draw_is_accepted_by_exactly_ceil_2_32_over_k_values():
    """Random remasking unmasks with probability 1 - s/t = 1/k at countdown k (Section 3.1 with the linear schedule): the
    accepted draws are u = 0 .. ceil(2^32 / k) - 1, also where k divides 2^32 and the boundary value is an integer."""
    for k in (1, 2, 3, 4, 7, 256, 1000, 65536):
        n_accept = -(-(1 << 32) // k)
        assert SM.draw_accepts(n_accept - 1, k)
        assert n_accept == (1 << 32) or not SM.draw_accepts(n_accept, k)
        assert SM.draw_accepts(0, k)
    assert not SM.draw_accepts((1 << 31), 2) and SM.draw_accepts((1 << 31) - 1, 2)


@pytest.mark.parametrize("strategy", [SM.LOW_CONFIDENCE, SM.RANDOM])
def test_semi_autoregressive_blocks_run_left_to_right(strategy):
    L, N, bl = 22, 12, 8                                    # blocks [0,8) [8,16) [16,22); 4 steps each
    predict, calls = random_process(L, 5)
    y, trace = SM.semi_autoregressive(L, N, bl, strategy, predict, seed=11)
    assert all(t is not None for t in y)
    done = set()
    for rec in trace:
        lo, hi = rec.block * bl, min(L, (rec.block + 1) * bl)
        assert all(lo <= i < hi for i in rec.positions)
        assert all(i in done for i in range(lo))            # every earlier block is complete
        done |= set(rec.positions)
        assert rec.block == rec.step // 4 and rec.k_block == 4 - rec.step % 4
    assert all(all(i // bl == rows[0] // bl for i in rows) for rows in calls if rows)   # only the current block's rows are read
    with pytest.raises(ValueError):
        SM.semi_autoregressive(L, 10, bl, strategy, predict)


def test_one_block_is_the_plain_strategy():
    L, N = 14, 7
    a, _ = random_process(L, 9); b, _ = random_process(L, 9)
    assert SM.semi_autoregressive(L, N, 100, SM.LOW_CONFIDENCE, a)[1] == SM.low_confidence_remasking(L, N, b)[1]


@pytest.mark.parametrize("strategy,L,N,bl", [(SM.LOW_CONFIDENCE, 24, 12, 0), (SM.LOW_CONFIDENCE, 24, 12, 8), (SM.RANDOM, 24, 24, 0),
                                             (SM.RANDOM, 30, 9, 10), (SM.LOW_CONFIDENCE, 9, 18, 0)])
def test_step_machine_equals_the_loop(strategy, L, N, bl):
    for seed in range(10):
        pa, _ = random_process(L, seed)
        pb, _ = random_process(L, seed)
        y, trace = SM.semi_autoregressive(L, N, bl if bl else L, strategy, pa, seed=seed + 3, seq=2)
        p = SM.VanillaParams(strategy=strategy, max_steps=N, block_len=bl, seed=seed + 3)
        st = SM.VanillaState.fresh(L, p)
        got = []
        y2 = [None] * L
        while not st.done:
            rows = SM.vanilla_rows_needed(st)
            a, sq = pb(list(st.masked), rows) if rows else ({}, {})
            rec = SM.vanilla_step(st, a, sq, p, seq=2)
            for i, t in zip(rec.positions, rec.tokens):
                y2[i] = t
            got.append(rec.key())
        assert got == [r.key() for r in trace] and y2 == y
