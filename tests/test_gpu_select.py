"""GPU parity: one step of the SlowFast rule (row statistics + selection) against the oracle's step machine,
bit for bit, driven with seeded synthetic logits whose confidences fire every branch."""
import numpy as np
import pytest
import torch

from oracle import rowstats as RS
from oracle.scheduler import FAST, SLOW, SlowFastState, rows_needed, slowfast_step
from paper_2506_10848_b200 import binding as sfs
from paper_2506_10848_b200 import workloads as W

from helpers import oracle_state_as_ints, params_pair, state_to_dict, write_state

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def synthetic_step_logits(n_rows, V, gen, dtype):
    """Rows with a planted winner whose margin makes confidences spread over (0, 1)."""
    x = torch.randn((n_rows, V), generator=gen) * 1.5
    col = torch.randint(0, V, (n_rows,), generator=gen)
    margin = torch.rand((n_rows,), generator=gen) * 14.0
    x[torch.arange(n_rows), col] = x.max(dim=1).values + margin
    return x.to(dtype)


def run_lockstep(B, P, L, V, pkw, seed, dtype=torch.bfloat16, supply_all_rows=False):
    po, pg = params_pair(**pkw)
    S = P + L
    gen = torch.Generator().manual_seed(seed)
    session = sfs.sfs_select_session_create(V, B, S)
    try:
        tokens = torch.full((B, S), V - 1, dtype=torch.int32, device=DEV)
        mask = torch.zeros((B, S), dtype=torch.uint8, device=DEV); mask[:, P:] = 1
        state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
        sfs.sfs_state_init(state, B, L, pg)
        sel_count = torch.zeros(B, dtype=torch.int32, device=DEV)
        sel_pos = torch.zeros((B, L), dtype=torch.int32, device=DEV)
        sel_tok = torch.zeros((B, L), dtype=torch.int32, device=DEV)
        next_rows = torch.zeros(B * L, dtype=torch.int32, device=DEV)
        next_n = torch.zeros(1, dtype=torch.int32, device=DEV)
        trace = torch.zeros((B, sfs.TRACE_INTS), dtype=torch.int32, device=DEV)
        ost = [SlowFastState.fresh(L, po) for _ in range(B)]
        oy = [[None] * L for _ in range(B)]
        steps = 0
        while not all(s.done for s in ost):
            need = [(b, i) for b in range(B) for i in rows_needed(ost[b])]
            if steps > 0:                                   # the library's own row list for this step
                n = int(next_n.item())
                assert next_rows[:n].tolist() == [b * S + P + i for (b, i) in need]
            rows_list = need
            if supply_all_rows:                             # extra rows must be ignored
                rows_list = [(b, i) for b in range(B) for i in range(L) if ost[b].masked[i] and not ost[b].done]
            n_rows = len(rows_list)
            logits = synthetic_step_logits(n_rows, V, gen, dtype)
            rows = torch.tensor([b * S + P + i for (b, i) in rows_list], dtype=torch.int32, device=DEV)
            n_dev = torch.tensor([n_rows], dtype=torch.int32, device=DEV)
            dl = logits.to(DEV)
            sfs.sfs_select(session, dl, sfs.LOGITS_BF16 if dtype == torch.bfloat16 else sfs.LOGITS_F32, V, rows, n_dev,
                           n_rows, tokens, mask, B, S, P, state, pg, sel_count, sel_pos, sel_tok, next_rows, next_n, trace)
            torch.cuda.synchronize()
            st = RS.row_stats(W.bf16_bits(logits) if dtype == torch.bfloat16 else logits.numpy())
            for b in range(B):
                if ost[b].done:
                    assert int(sel_count[b]) == 0
                    continue
                idx = {i: j for j, (bb, i) in enumerate(rows_list) if bb == b}
                a = {i: int(st["argmax"][j]) for i, j in idx.items()}
                sq = {i: int(st["sq"][j]) for i, j in idx.items()}
                rec = slowfast_step(ost[b], a, sq, po)
                for i, t in zip(rec.positions, rec.tokens):
                    oy[b][i] = t
                n = int(sel_count[b])
                assert sel_pos[b, :n].tolist() == rec.positions
                assert sel_tok[b, :n].tolist() == rec.tokens
                tr = trace[b].tolist()
                assert tr[:6] == [rec.phase, rec.s, rec.hi, rec.e_cand, rec.stable, len(rec.positions)]
                got = state_to_dict(state[b])
                want = oracle_state_as_ints(ost[b], po.w_hist)
                if ost[b].done:                                   # phase / span of a finished sequence carry no meaning
                    want = {k: want[k] for k in ("n_masked", "done", "k_remaining")}
                for k_, v_ in want.items():
                    assert got[k_] == v_, (k_, got, want)
                assert got["status"] == 0
            steps += 1
            assert steps <= (po.max_steps or L) + 1
        tk = tokens.cpu()
        mk = mask.cpu()
        for b in range(B):
            assert tk[b, P:].tolist() == oy[b]
            assert int(mk[b].sum()) == 0
        return steps
    finally:
        sfs.sfs_session_destroy(session)


@pytest.mark.parametrize("seed", range(6))
def test_lockstep_default_params(seed):
    steps = run_lockstep(B=3, P=5, L=48, V=512, pkw={}, seed=seed)
    assert steps < 48                                       # parallel unmasking happened


@pytest.mark.parametrize("seed,pkw", [
    (10, dict(k_max=3, w_hist=3, sigma2_stable=30.0, k_slow=2, k_fast=3)),
    (11, dict(k_max=1, w_hist=1, k_slow=4, min_high_count=3)),
    (12, dict(max_steps=9, k_slow=1)),                       # the step budget runs out: forced last step
    (13, dict(tau_min_conf=-1.0, tau_high_conf=2.0, sigma2_stable=float("inf"), k_max=1, w_hist=1)),
    (14, dict(w_hist=8, k_max=12, sigma2_stable=400.0)),
    (15, dict(k_max=3, w_hist=2, sigma2_stable=0.0)),        # no variance is below 0: every cycle ends by the K_max fallback
    (16, dict(k_max=2, w_hist=5)),                           # the history cannot fill before K_max
])
def test_lockstep_other_params(seed, pkw):
    run_lockstep(B=2, P=3, L=40, V=256, pkw=pkw, seed=seed)


def test_lockstep_fp32_logits_extra_rows_and_ragged_sizes():
    run_lockstep(B=1, P=0, L=1, V=8, pkw={}, seed=20, dtype=torch.float32)
    run_lockstep(B=4, P=7, L=33, V=1000, pkw={}, seed=21, dtype=torch.float32, supply_all_rows=True)
    run_lockstep(B=2, P=1, L=300, V=512, pkw=dict(k_slow=3), seed=22, supply_all_rows=True)


def test_missing_row_is_reported_not_guessed():
    po, pg = params_pair()
    B, P, L, V = 1, 2, 8, 64
    S = P + L
    session = sfs.sfs_select_session_create(V, B, S)
    try:
        tokens = torch.full((B, S), V - 1, dtype=torch.int32, device=DEV)
        mask = torch.zeros((B, S), dtype=torch.uint8, device=DEV); mask[:, P:] = 1
        state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
        sfs.sfs_state_init(state, B, L, pg)
        logits = torch.randn((L - 1, V)).to(torch.bfloat16).to(DEV)      # the row of position L-1 is withheld
        rows = torch.arange(P, P + L - 1, dtype=torch.int32, device=DEV)
        sel_count = torch.zeros(B, dtype=torch.int32, device=DEV)
        sfs.sfs_select(session, logits, sfs.LOGITS_BF16, V, rows, None, L - 1, tokens, mask, B, S, P, state, pg, sel_count)
        torch.cuda.synchronize()
        assert state_to_dict(state[0])["status"] == sfs.ERR_MISSING_ROW
        assert int(sel_count[0]) == 0 and int(mask.sum()) == L
    finally:
        sfs.sfs_session_destroy(session)


def test_epilogue_microbenchmark_one_slow_one_fast_step():
    """bf16 logits [256, 126464] with planted winners; one exploratory and one accelerated step from a given
    span [lo, hi), compared with the oracle."""
    V, L, P, B = 126464, 256, 0, 1
    po, pg = params_pair()
    x = W.planted_logits(L, V, seed=1, device="cpu")
    st = RS.row_stats(W.bf16_bits(x))
    frac = [float(np.mean(RS.exceeds(st["sq"], t))) for t in (0.1, 0.85, 0.9)]
    print("fraction of rows above 0.1 / 0.85 / 0.9:", frac)
    lo, hi = W.span(L, seed=1)
    dl = x.to(DEV)
    session = sfs.sfs_select_session_create(V, B, L)
    try:
        for phase in (SLOW, FAST):
            tokens = torch.full((B, L), V - 1, dtype=torch.int32, device=DEV)
            mask = torch.ones((B, L), dtype=torch.uint8, device=DEV); mask[:, :lo] = 0
            state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
            sfs.sfs_state_init(state, B, L, pg)
            write_state(state, 0, phase=phase, s_cycle=lo, hi=hi if phase == FAST else 0, n_masked=L - lo,
                        k_remaining=L - lo, hist_len=1 if phase == SLOW else 0, hist0=L - 1, step_count=1 if phase == SLOW else 0)
            ost = SlowFastState(L=L, k=L - lo, phase=phase, s_cycle=lo, hi=hi if phase == FAST else 0,
                                step_count=1 if phase == SLOW else 0, H=[L - 1] if phase == SLOW else [],
                                masked=[i >= lo for i in range(L)])
            need = rows_needed(ost)
            rows = torch.tensor(need, dtype=torch.int32, device=DEV)
            sub = dl[need].contiguous()
            sel_count = torch.zeros(B, dtype=torch.int32, device=DEV)
            sel_pos = torch.zeros((B, L), dtype=torch.int32, device=DEV)
            sel_tok = torch.zeros((B, L), dtype=torch.int32, device=DEV)
            sfs.sfs_select(session, sub, sfs.LOGITS_BF16, V, rows, None, len(need), tokens, mask, B, L, P, state, pg,
                           sel_count, sel_pos, sel_tok)
            torch.cuda.synchronize()
            rec = slowfast_step(ost, {i: int(st["argmax"][i]) for i in need}, {i: int(st["sq"][i]) for i in need}, po)
            n = int(sel_count[0])
            assert sel_pos[0, :n].tolist() == rec.positions and sel_tok[0, :n].tolist() == rec.tokens
            got = state_to_dict(state[0])
            for k_, v_ in oracle_state_as_ints(ost, po.w_hist).items():
                assert got[k_] == v_, (k_, got)
            if phase == FAST:
                assert n > 1                               # several in-span rows exceed tau_high: parallel unmasking
    finally:
        sfs.sfs_session_destroy(session)


def _one_step_inputs(B, P, L, V, pg, gen):
    S = P + L
    tokens = torch.full((B, S), V - 1, dtype=torch.int32, device=DEV)
    mask = torch.zeros((B, S), dtype=torch.uint8, device=DEV); mask[:, P:] = 1
    state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
    sfs.sfs_state_init(state, B, L, pg)
    rows = torch.tensor([b * S + P + i for b in range(B) for i in range(L)], dtype=torch.int32, device=DEV)
    logits = synthetic_step_logits(B * L, V, gen, torch.bfloat16).to(DEV)
    return tokens, mask, state, rows, logits


def test_row_index_outside_the_token_grid_is_skipped_and_reported():
    """A row list may carry a stale or foreign index: the statistics of such a row are dropped (never written outside the
    scratch), the device status word reports it, and the sequence whose row is now missing stops with MISSING_ROW."""
    B, P, L, V = 2, 4, 24, 512
    S = P + L
    po, pg = params_pair()
    session = sfs.sfs_select_session_create(V, B, S)
    try:
        tokens, mask, state, rows, logits = _one_step_inputs(B, P, L, V, pg, torch.Generator().manual_seed(5))
        bad = rows.clone()
        bad[3] = B * S + 1000                               # sequence 0's row 3: beyond the grid
        bad[L + 7] = -9                                     # sequence 1's row 7: negative
        before = tokens.clone()
        sfs.sfs_select(session, logits, sfs.LOGITS_BF16, V, bad, None, B * L, tokens, mask, B, S, P, state, pg)
        with pytest.raises(sfs.SfsError) as e:
            sfs.sfs_check_device_status()
        assert e.value.status == sfs.ERR_INVALID_ARG
        sfs.sfs_check_device_status()                       # sticky word is cleared by the read
        for b in range(B):
            assert state_to_dict(state[b])["status"] == sfs.ERR_MISSING_ROW
        assert torch.equal(tokens, before) and int(mask[:, P:].sum()) == B * L
    finally:
        sfs.sfs_session_destroy(session)


def test_statistics_of_a_finished_sequence_do_not_survive_into_the_next_generation():
    """Rows supplied for a sequence that is already done are consumed like any others: when the scratch is reused with a
    fresh state, a needed row that the caller omits is reported as missing instead of being read from the old call."""
    B, P, L, V = 1, 0, 16, 512
    S = P + L
    po, pg = params_pair(max_steps=1)                       # one permitted step: it decodes everything, the sequence is done
    gen = torch.Generator().manual_seed(6)
    session = sfs.sfs_select_session_create(V, B, S)
    try:
        tokens, mask, state, rows, logits = _one_step_inputs(B, P, L, V, pg, gen)
        sfs.sfs_select(session, logits, sfs.LOGITS_BF16, V, rows, None, L, tokens, mask, B, S, P, state, pg)
        assert state_to_dict(state[0])["done"] == 1
        # statistics for the finished sequence arrive once more (a caller running a batch does this for finished members)
        sfs.sfs_select(session, logits, sfs.LOGITS_BF16, V, rows, None, L, tokens, mask, B, S, P, state, pg)
        # new generation on the same scratch; row 5 is left out
        _, pg2 = params_pair()
        tokens, mask, state, rows, logits = _one_step_inputs(B, P, L, V, pg2, gen)
        keep = [i for i in range(L) if i != 5]
        sfs.sfs_select(session, logits[keep].contiguous(), sfs.LOGITS_BF16, V, rows[keep].contiguous(), None, L - 1, tokens, mask, B, S, P, state, pg2)
        sfs.sfs_check_device_status()
        assert state_to_dict(state[0])["status"] == sfs.ERR_MISSING_ROW and int(mask.sum()) == L
    finally:
        sfs.sfs_session_destroy(session)


@pytest.mark.parametrize("case", ["near_ties", "threshold_edges", "all_confident", "near_ties_k2"])
def test_full_vocabulary_steps_where_the_cheap_pass_cannot_decide(case):
    """Long bf16 rows take the two-pass row statistics.  These inputs are built so that the enclosures of the cheap pass
    leave the step's questions open — top-1 candidates closer than the enclosure width, confidences within 1e-5 of a
    threshold, many rows with S_q = 2^28 exactly — and the decisions must still be the oracle's, slow and fast step."""
    V, L, P, B = 126464, 48, 0, 1
    po, pg = params_pair(k_slow=2, k_fast=3) if case == "near_ties_k2" else params_pair()     # k > 1: every candidate is recomputed
    if case.startswith("near_ties"):
        conf = torch.full((L,), 0.05, dtype=torch.float64)
        conf[10] = 0.30000; conf[20] = 0.30001; conf[30] = 0.29999; conf[31] = 0.30000        # best four within 3e-5 relative
    elif case == "threshold_edges":
        conf = torch.linspace(0.02, 0.95, L, dtype=torch.float64)
        conf[5] = 0.1 + 1e-6; conf[6] = 0.1 - 1e-6; conf[7] = 0.85 + 1e-6; conf[8] = 0.85 - 1e-6; conf[40] = 0.1000001
    else:
        conf = torch.full((L,), 1.0 - 1e-12, dtype=torch.float64)
    logits = W.logits_for_confidences(conf, V, seed=3)
    stats = RS.row_stats(W.bf16_bits(logits))
    session = sfs.sfs_select_session_create(V, B, L)
    try:
        for phase, span in ((SLOW, None), (FAST, (4, 44))):
            tokens = torch.full((B, L), V - 1, dtype=torch.int32, device=DEV)
            mask = torch.ones((B, L), dtype=torch.uint8, device=DEV)
            state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
            sfs.sfs_state_init(state, B, L, pg)
            ost = SlowFastState.fresh(L, po)
            if phase == FAST:
                write_state(state, 0, phase=1, s_cycle=span[0], hi=span[1])
                ost.phase, ost.s_cycle, ost.hi = FAST, span[0], span[1]
            rows = torch.arange(L, dtype=torch.int32, device=DEV)
            sel_count = torch.zeros(B, dtype=torch.int32, device=DEV)
            sel_pos = torch.zeros((B, L), dtype=torch.int32, device=DEV); sel_tok = torch.zeros((B, L), dtype=torch.int32, device=DEV)
            trace = torch.zeros((B, sfs.TRACE_INTS), dtype=torch.int32, device=DEV)
            sfs.sfs_select(session, logits.to(DEV), sfs.LOGITS_BF16, V, rows, None, L, tokens, mask, B, L, P, state, pg,
                           sel_count, sel_pos, sel_tok, trace=trace)
            torch.cuda.synchronize()
            rec = slowfast_step(ost, {i: int(stats["argmax"][i]) for i in range(L)}, {i: int(stats["sq"][i]) for i in range(L)}, po)
            n = int(sel_count[0])
            assert sel_pos[0, :n].tolist() == rec.positions and sel_tok[0, :n].tolist() == rec.tokens, (case, phase)
            assert trace[0].tolist()[:6] == [rec.phase, rec.s, rec.hi, rec.e_cand, rec.stable, len(rec.positions)], (case, phase)
        sfs.sfs_check_device_status()
    finally:
        sfs.sfs_session_destroy(session)


@pytest.mark.parametrize("V", [512, 126464])
def test_thresholds_are_strict_where_the_confidence_equals_them(V):
    """Rows with n equal maxima and nothing else within reach have S_q = n 2^28 exactly, i.e. c = 1/n.  With tau_min = 1/4
    and tau_high = 1/2 (both exact in float32) the rows at c = 1/4 and c = 1/2 sit on the thresholds: the comparisons are
    strict, on short rows (one-pass statistics) and on full-vocabulary rows (the cheap pass cannot decide them)."""
    L, P, B = 16, 0, 1
    n_max = [1, 2, 3, 4, 5, 2, 4, 1, 3, 4, 2, 6, 4, 2, 1, 4]
    logits = torch.full((L, V), -200.0, dtype=torch.float32)
    g = torch.Generator().manual_seed(V)
    for i, n in enumerate(n_max):
        logits[i, torch.randperm(V, generator=g)[:n]] = 1.5
    logits = logits.to(torch.bfloat16)
    stats = RS.row_stats(W.bf16_bits(logits))
    assert [int(s) for s in stats["sq"]] == [n << 28 for n in n_max]
    po, pg = params_pair(tau_min_conf=0.25, tau_high_conf=0.5)
    session = sfs.sfs_select_session_create(V, B, L)
    try:
        for phase, span in ((SLOW, None), (FAST, (1, 15))):
            tokens = torch.full((B, L), V - 1, dtype=torch.int32, device=DEV)
            mask = torch.ones((B, L), dtype=torch.uint8, device=DEV)
            state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
            sfs.sfs_state_init(state, B, L, pg)
            ost = SlowFastState.fresh(L, po)
            if phase == FAST:
                write_state(state, 0, phase=1, s_cycle=span[0], hi=span[1])
                ost.phase, ost.s_cycle, ost.hi = FAST, span[0], span[1]
            rows = torch.arange(L, dtype=torch.int32, device=DEV)
            sel_count = torch.zeros(B, dtype=torch.int32, device=DEV)
            sel_pos = torch.zeros((B, L), dtype=torch.int32, device=DEV); sel_tok = torch.zeros((B, L), dtype=torch.int32, device=DEV)
            trace = torch.zeros((B, sfs.TRACE_INTS), dtype=torch.int32, device=DEV)
            sfs.sfs_select(session, logits.to(DEV), sfs.LOGITS_BF16, V, rows, None, L, tokens, mask, B, L, P, state, pg,
                           sel_count, sel_pos, sel_tok, trace=trace)
            torch.cuda.synchronize()
            rec = slowfast_step(ost, {i: int(stats["argmax"][i]) for i in range(L)}, {i: int(stats["sq"][i]) for i in range(L)}, po)
            n = int(sel_count[0])
            assert sel_pos[0, :n].tolist() == rec.positions and sel_tok[0, :n].tolist() == rec.tokens, phase
            assert trace[0].tolist()[:6] == [rec.phase, rec.s, rec.hi, rec.e_cand, rec.stable, len(rec.positions)], phase
            if phase == SLOW:
                assert rec.e_cand == 14                           # position 15 (c = 1/4) does not reach tau_min, 14 (c = 1) does
            else:
                assert rec.positions == [7, 14]                   # c = 1 only: the rows at c = 1/2 stay masked
        sfs.sfs_check_device_status()
    finally:
        sfs.sfs_session_destroy(session)


@pytest.mark.parametrize("min_high,expect", [(2, [3, 9]), (3, [3])])
def test_fast_step_with_exactly_the_minimum_number_of_confident_rows(min_high, expect):
    """An accelerated step whose span holds exactly two rows above tau_high: with a minimum of two the confident set is
    taken as it is, with a minimum of three the step falls back to the k_fast most confident rows (here one: of the two
    rows at c = 1 the one at the smaller position)."""
    V, L, P, B = 512, 16, 0, 1
    logits = torch.full((L, V), -200.0, dtype=torch.float32)
    g = torch.Generator().manual_seed(7)
    for i in range(L):
        logits[i, torch.randperm(V, generator=g)[: (1 if i in (3, 9) else 3)]] = 0.5      # c = 1 at rows 3 and 9, 1/3 elsewhere
    logits = logits.to(torch.bfloat16)
    stats = RS.row_stats(W.bf16_bits(logits))
    po, pg = params_pair(tau_high_conf=0.5, min_high_count=min_high, k_fast=1)
    session = sfs.sfs_select_session_create(V, B, L)
    try:
        tokens = torch.full((B, L), V - 1, dtype=torch.int32, device=DEV)
        mask = torch.ones((B, L), dtype=torch.uint8, device=DEV)
        state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
        sfs.sfs_state_init(state, B, L, pg)
        write_state(state, 0, phase=1, s_cycle=0, hi=L)
        ost = SlowFastState.fresh(L, po)
        ost.phase, ost.s_cycle, ost.hi = FAST, 0, L
        rows = torch.arange(L, dtype=torch.int32, device=DEV)
        sel_count = torch.zeros(B, dtype=torch.int32, device=DEV)
        sel_pos = torch.zeros((B, L), dtype=torch.int32, device=DEV); sel_tok = torch.zeros((B, L), dtype=torch.int32, device=DEV)
        sfs.sfs_select(session, logits.to(DEV), sfs.LOGITS_BF16, V, rows, None, L, tokens, mask, B, L, P, state, pg,
                       sel_count, sel_pos, sel_tok)
        torch.cuda.synchronize()
        sfs.sfs_check_device_status()
        rec = slowfast_step(ost, {i: int(stats["argmax"][i]) for i in range(L)}, {i: int(stats["sq"][i]) for i in range(L)}, po)
        n = int(sel_count[0])
        assert sel_pos[0, :n].tolist() == rec.positions == expect
        assert sel_tok[0, :n].tolist() == rec.tokens
    finally:
        sfs.sfs_session_destroy(session)
