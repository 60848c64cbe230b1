"""Pins for the oracle's row statistics (greedy token, Section 3.1 Eq. 3; confidence, Section 3.1):
brute force on tiny rows, closed forms, invariances, and the bound that ties the canonical fixed-point
denominator S_q to the plain double-precision softmax."""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import rowstats as RS

Q = RS.QBITS


def brute(row):
    """max-prob and first argmax by the definition, with exact-ish arithmetic (math.fsum of math.exp)."""
    vals = [float(v) for v in row]
    finite = [v for v in vals if not math.isnan(v)]
    m = max(finite)
    a = next(i for i, v in enumerate(vals) if v == m)
    den = math.fsum(math.exp(v - m) for v in vals if not math.isnan(v))
    return a, 1.0 / den


def bf16_round(x):
    """fp32 -> nearest-even bf16 bit patterns (numpy only)."""
    u = np.asarray(x, np.float32).view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    return r


def widen(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32)


def test_bruteforce_tiny_rows():
    rng = np.random.default_rng(0)
    rows = []
    for V in (1, 2, 3, 8, 17, 64):
        for scale in (0.1, 3.0, 30.0):
            rows.append(rng.normal(0, scale, V).astype(np.float32))
    rows.append(np.array([5, 5, 5, 5], np.float32))                 # all tied -> id 0
    rows.append(np.array([1, 7, 7, 3], np.float32))                 # tie -> first
    rows.append(np.array([-3e38, 3e38, 0, 1], np.float32))          # huge spread
    rows.append(np.array([-np.inf, 2.0, -np.inf, 1.0], np.float32))  # -inf entries contribute nothing
    rows.append(np.array([0.0, -0.0, -1.0], np.float32))            # +0 == -0 -> first
    rows.append(np.array([-0.0, 0.0, -1.0], np.float32))
    rows.append(np.array([-80.0, -80.5, -300.0], np.float32))       # all negative
    for row in rows:
        st = RS.row_stats(row[None, :])
        a, c = brute(row)
        assert int(st["argmax"][0]) == a
        assert st["conf_exact"][0] == pytest.approx(c, rel=1e-12)
        V = len(row)
        cq = (1 << Q) / float(st["sq"][0])
        assert abs(cq - c) <= c * 1.2e-5 + V * 2.0 ** -Q


def test_uniform_row_is_exact():
    # every term is the maximum: P = 3 exactly, e_v = 2^28 exactly, so S_q = V * 2^28 and c = 1/V
    for V in (1, 5, 4096, 126464):
        st = RS.row_stats(np.full((1, V), -2.75, np.float32))
        assert int(st["sq"][0]) == V << Q
        assert int(st["argmax"][0]) == 0
        assert st["conf_exact"][0] == pytest.approx(1.0 / V, rel=1e-12)


def test_power_of_two_gaps_closed_form():
    # x_v - m = -j*ln2 is not representable, but a row {0, -K} with K huge contributes exactly nothing:
    st = RS.row_stats(np.array([[0.0] + [-100.0] * 1000], np.float32))
    assert int(st["sq"][0]) == 1 << Q                                 # terms below 2^-28 truncate to zero
    # one winner with margin d over V-1 equal losers: c = 1 / (1 + (V-1) e^-d)
    for V, d in ((10, 1.0), (1000, 5.0), (126464, 9.0), (126464, 14.0)):
        row = np.full(V, 0.0, np.float32); row[V // 3] = d
        st = RS.row_stats(row[None, :])
        c = 1.0 / (1.0 + (V - 1) * math.exp(-d))
        assert st["conf_exact"][0] == pytest.approx(c, rel=1e-10)
        assert (1 << Q) / float(st["sq"][0]) == pytest.approx(c, rel=2e-5, abs=V * 2.0 ** -Q)
        assert int(st["argmax"][0]) == V // 3


def test_small_terms_truncate_to_the_integer_the_mathematics_fixes():
    """A row {0, d}: S_q = 2^28 + trunc(2^28 e^d up to the recipe's 1e-5 relative error).  Where 2^28 e^d sits well inside an
    integer interval the truncation is fixed by the mathematics alone: the terms just above 1 (the last shift that keeps a
    bit), the first ones that vanish, and a ladder of small integers in between."""
    ln2 = math.log(2.0)
    checked = 0
    for j in range(-3, 14):                                           # 2^28 e^d = 2^j * e^f
        for f in (0.05, 0.2, 0.3):
            d = np.float32(-(28 - j) * ln2 + f)
            val = (1 << Q) * math.exp(float(d))                       # on the fp32 value actually handed over
            if abs(val - round(val)) < 1e-4 * val + 0.02:             # too close to an integer to be fixed within 1e-5
                continue
            st = RS.row_stats(np.array([[0.0, d]], np.float32))
            assert int(st["sq"][0]) == (1 << Q) + int(math.floor(val)), (j, f, val)
            checked += 1
    assert checked >= 40
    # the three regimes by name: one unit left, nothing left, and exactly nothing far below
    assert int(RS.row_stats(np.array([[0.0, -28 * ln2 + 0.2]], np.float32))["sq"][0]) == (1 << Q) + 1
    assert int(RS.row_stats(np.array([[0.0, -29 * ln2 + 0.2]], np.float32))["sq"][0]) == (1 << Q)
    assert int(RS.row_stats(np.array([[5.0, 5.0 - 28 * ln2 - 0.2]], np.float32))["sq"][0]) == (1 << Q)


def test_canonical_sum_is_permutation_invariant_and_translation_stable():
    rng = np.random.default_rng(3)
    row = rng.normal(0, 4, 5000).astype(np.float32)
    st0 = RS.row_stats(row[None, :])
    for _ in range(5):
        perm = rng.permutation(row.size)
        st = RS.row_stats(row[perm][None, :])
        assert int(st["sq"][0]) == int(st0["sq"][0])                  # integer sum: order-independent
        assert perm[int(st["argmax"][0])] == int(st0["argmax"][0])
    shifted = RS.row_stats((row + np.float32(8.0))[None, :])          # softmax is shift-invariant
    assert (1 << Q) / float(shifted["sq"][0]) == pytest.approx((1 << Q) / float(st0["sq"][0]), rel=3e-5)


def test_sq_tracks_exact_softmax_on_workload_like_rows():
    rng = np.random.default_rng(1)
    V = 126464
    x = rng.normal(0, 4, (6, V)).astype(np.float32)
    for r, margin in enumerate((0.0, 0.5, 3.0, 6.0, 9.0, 12.0)):
        x[r, 1000 * r + 7] = x[r].max() + margin
    bits = bf16_round(x)
    st = RS.row_stats(bits)
    xf = widen(bits)
    for r in range(x.shape[0]):
        a, c = brute(xf[r])
        assert int(st["argmax"][r]) == a
        assert st["conf_exact"][r] == pytest.approx(c, rel=1e-9)
        cq = (1 << Q) / float(st["sq"][r])
        # polynomial (3.4e-6) + range reduction and mantissa rounding, relative; truncation V * 2^-28 absolute on the sum
        assert abs(cq - c) <= c * 1e-5 + c * c * V * 2.0 ** -Q
    # the bf16 entry point and the fp32 entry point agree on widened values
    st32 = RS.row_stats(np.ascontiguousarray(xf))
    assert np.array_equal(st32["sq"], st["sq"]) and np.array_equal(st32["argmax"], st["argmax"])


def test_threshold_decisions_match_exact_confidence_away_from_the_boundary():
    rng = np.random.default_rng(5)
    V = 4096
    x = rng.normal(0, 2.5, (400, V)).astype(np.float32)
    x[np.arange(400), rng.integers(0, V, 400)] += rng.uniform(0, 22, 400).astype(np.float32)
    st = RS.row_stats(x)
    for tau in (0.1, 0.85):
        dec = RS.exceeds(st["sq"], tau)
        far = np.abs(st["conf_exact"] - tau) > 1e-3
        assert np.array_equal(dec[far], (st["conf_exact"] > tau)[far])
    assert 0.05 < np.mean(RS.exceeds(st["sq"], 0.85)) < 0.95        # the test exercises both outcomes


def test_planted_sign_and_index_mistakes_would_be_caught():
    # a transposed comparison (argmin), a dropped max-subtraction or exp(+x) all change these values
    row = np.array([[0.0, 1.0, 2.0, 3.0]], np.float32)
    st = RS.row_stats(row)
    e = [math.exp(v - 3.0) for v in (0.0, 1.0, 2.0, 3.0)]
    assert int(st["argmax"][0]) == 3
    assert st["conf_exact"][0] == pytest.approx(1.0 / sum(e), rel=1e-14)
    assert float(st["vmax"][0]) == 3.0
    assert abs(int(st["sq"][0]) / 2.0 ** Q - sum(e)) < 1e-5
