"""GPU parity of the feature cache: cached steps against the oracle's cached forward pass under the SAME schedule
(the oracle is handed the row sets the GPU chose), the row choice itself against the oracle's rule on the GPU's own
similarity values (an integer decision: both sides decide on identical numbers), the similarities against the
oracle's within tolerance, and the cache-off equivalences."""
import math

import numpy as np
import pytest
import torch

from oracle import cache as C
from oracle import forward as F
from paper_2506_10848_b200 import binding as sfs
from paper_2506_10848_b200 import workloads as W

from test_gpu_forward import MAX_ABS, REL_L2, max_abs_bar, tiny_setup

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def state_tensor(B, phase=0, s_cycle=0, hi=0):
    st = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32)
    st[:, sfs.STATE_FIELDS.index("phase")] = phase
    st[:, sfs.STATE_FIELDS.index("s_cycle")] = s_cycle
    st[:, sfs.STATE_FIELDS.index("hi")] = hi
    return st.to(DEV)


def check_logits(got, ref, scale):
    err = np.abs(got - ref)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert rel <= REL_L2, rel
    assert err.max() <= max_abs_bar(scale), err.max()


# (1, 512, 128, ..): a long sequence (five key tiles) and few recomputed rows: a compact query tile against many cached key
# tiles; (1, 9, 55, ..): an odd prompt length (the response starts at an odd token index)
@pytest.mark.parametrize("B,P,L,kp,kr,rho", [(1, 32, 64, 100, 3, 0.25), (2, 24, 40, 4, 2, 0.3), (1, 8, 56, 5, 100, 0.1),
                                             (1, 512, 128, 100, 4, 0.25), (1, 9, 55, 100, 3, 0.2),
                                             (1, 8, 1112, 100, 3, 0.1)])      # more response positions than the choice kernel has threads
def test_cached_steps_match_oracle_under_the_same_schedule(B, P, L, kp, kr, rho):
    shape, model, cfg, w64 = tiny_setup(seed=3)
    S = P + L
    nl = shape.n_layers
    session = sfs.sfs_session_create(model, B, S)
    sfs.sfs_cache_enable(session, kp, kr, rho)
    g = np.random.default_rng(B * 100 + L)
    tok = np.full((B, S), shape.mask_id, dtype=np.int32)
    tok[:, :P] = g.integers(0, shape.vocab - 2, size=(B, P))
    caches = [C.FeatureCache(cfg, S) for _ in range(B)]
    logits = torch.zeros((B * S, shape.vocab), dtype=torch.float32, device=DEV)
    sets = torch.full((nl * B * S,), -1, dtype=torch.int32, device=DEV)
    sims = torch.zeros((nl * B * L,), dtype=torch.float32, device=DEV)
    n_adapt = C.adaptive_count(rho, L)
    for step in range(7):
        if step > 0:                                           # unmask a few positions, as the sampler would
            for b in range(B):
                for i in g.choice(L, size=2, replace=False):
                    tok[b, P + i] = int(g.integers(0, shape.vocab - 2))
        fast = step in (2, 5)
        span = (L // 4, L // 4 + 9) if fast else None
        st = state_tensor(B, 1, span[0], span[1]) if fast else state_tensor(B)
        d_tok = torch.from_numpy(tok).to(DEV)
        sets.fill_(-1)
        n_sel = sfs.sfs_forward_cached(session, d_tok, B, S, P, st, None, None, B * S, logits, sfs.LOGITS_F32, sets=sets, sims=sims)
        sfs.sfs_check_device_status()
        rp, rr = step % kp == 0, step % kr == 0
        assert n_sel == (S if (rp and rr) else (P if rp else 0) + (L if rr else n_adapt))
        got = logits.cpu().double().numpy().reshape(B, S, -1)
        gsets = sets.cpu().numpy()[: nl * B * n_sel].reshape(nl, B, n_sel)
        gsims = sims.cpu().numpy().reshape(nl, B, L)
        for b in range(B):
            rec = {}
            forced = lambda l, s_, c_, b=b: sorted(set(int(r) - b * S - P for r in gsets[l, b] if int(r) - b * S >= P))
            ref = C.cached_forward(cfg, w64, tok[b], P, caches[b], kp, kr, rho, span=span, select=forced, record=rec)
            # response rows on every step; prompt rows are defined only on steps that refresh the prompt
            check_logits(got[b][P:], ref[P:], shape.logit_scale)
            if rp:
                check_logits(got[b][:P], ref[:P], shape.logit_scale)
            for l in range(nl):
                # the GPU's sets are exactly the rows of the rule: segment refreshes plus the adaptive choice
                assert sorted(set(int(r) - b * S for r in gsets[l, b])) == rec["sets"][l], (step, l)
                if not rr and n_adapt > 0:
                    cand = list(range(L)) if span is None else list(range(span[0], span[1]))
                    # integer decision on identical numbers: the oracle's rule applied to the GPU's similarities
                    mine = C.least_similar(gsims[l, b][cand], cand, min(n_adapt, len(cand)))
                    chosen = sorted(set(int(r) - b * S - P for r in gsets[l, b] if int(r) - b * S >= P))
                    assert chosen == mine, (step, l)
                    # and the similarities themselves agree with the oracle's (bf16 values on the GPU side)
                    assert np.abs(gsims[l, b][cand] - rec["sims"][l]).max() <= 2e-2, (step, l)
    sfs.sfs_session_destroy(session)
    model.close()


def test_refresh_every_step_equals_the_uncached_forward_and_unchanged_tokens_do_not_drift():
    shape, model, cfg, w64 = tiny_setup(seed=4)
    B, P, L = 1, 16, 48
    S = P + L
    session = sfs.sfs_session_create(model, B, S)
    g = np.random.default_rng(9)
    tok = np.full((B, S), shape.mask_id, dtype=np.int32)
    tok[:, :P] = g.integers(0, shape.vocab - 2, size=(B, P))
    d_tok = torch.from_numpy(tok).to(DEV)
    plain = torch.zeros((S, shape.vocab), dtype=torch.float32, device=DEV)
    sfs.sfs_forward(session, d_tok, B, S, None, None, S, plain, sfs.LOGITS_F32)
    cached = torch.zeros_like(plain)
    sfs.sfs_cache_enable(session, 1, 1, 0.25)
    for _ in range(2):
        sfs.sfs_forward_cached(session, d_tok, B, S, P, None, None, None, S, cached, sfs.LOGITS_F32)
        # same kernels except that the residual projections store their increments: fp32 rounding order only
        assert (cached - plain).abs().max().item() <= 2e-3 * shape.logit_scale
    # any schedule reproduces the same logits while the tokens do not change (cached features are exact then)
    sfs.sfs_cache_enable(session, 100, 3, 0.2)
    for step in range(5):
        sfs.sfs_forward_cached(session, d_tok, B, S, P, None, None, None, S, cached, sfs.LOGITS_F32)
        first = 0 if step == 0 else P                          # prompt rows: only on the step that refreshes the prompt
        assert (cached[first:] - plain[first:]).abs().max().item() <= 4e-3 * shape.logit_scale, step
    sfs.sfs_check_device_status()
    sfs.sfs_session_destroy(session)
    model.close()


def test_generation_with_cache_finishes_and_decodes_every_position_once():
    shape, model, cfg, w64 = tiny_setup(seed=0, logit_scale=60.0)
    B, P, L = 2, 32, 64
    S = P + L
    session = sfs.sfs_session_create(model, B, S)
    sfs.sfs_cache_enable(session, 100, 4, 0.25)
    prompt = W.prompt_ids(B, P, shape.vocab - 2, seed=0).to(DEV)
    out = torch.zeros((B, S), dtype=torch.int32, device=DEV)
    state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
    trace = torch.zeros((L + 4, B, sfs.TRACE_INTS), dtype=torch.int32, device=DEV)
    sfs.sfs_generate(session, prompt, B, P, L, sfs.Params.default(), out, state, trace, L + 4)
    st = state.cpu().numpy()
    assert np.all(st[:, sfs.STATE_FIELDS.index("done")] == 1) and np.all(st[:, sfs.STATE_FIELDS.index("n_masked")] == 0)
    assert np.array_equal(out[:, :P].cpu().numpy(), prompt.cpu().numpy())
    n_sel = trace[:, :, 5].cpu().numpy()
    assert np.all(n_sel.sum(axis=0) == L)                                # every position unmasked exactly once
    sfs.sfs_session_destroy(session)
    model.close()


def replay_cached_generation(shape, model, cfg, w_or, B, P, L, kp, kr, rho, max_steps, logits_ok, cache_dtype=np.float64, seed=0):
    """Teacher-forced cached generation: the device loop runs with the cache on, one step at a time, dumping its logits, row
    list and per-layer recomputed sets.  Per step and sequence the oracle's cached forward pass is run on the oracle's own
    token state under the sets the GPU chose (logits within tolerance; the sets themselves must be the oracle's rule applied
    to the GPU's similarities), then the oracle's row statistics and scheduler, fed the GPU's logits, must reproduce the
    GPU's decisions and tokens exactly.  Returns the number of steps replayed and the tokens unmasked per sequence."""
    from oracle import rowstats as RS
    from oracle.scheduler import FAST, SlowFastParams, SlowFastState, rows_needed, slowfast_step
    S, nl = P + L, shape.n_layers
    po = SlowFastParams()
    pg = sfs.Params.default()
    prompt = W.prompt_ids(B, P, shape.vocab - 2, seed=seed)
    n_adapt = C.adaptive_count(rho, L)
    session = sfs.sfs_session_create(model, B, S)
    try:
        sfs.sfs_cache_enable(session, kp, kr, rho)
        trace = torch.zeros((max_steps, B, sfs.TRACE_INTS), dtype=torch.int32, device=DEV)
        dump = torch.zeros((B * L, shape.vocab), dtype=torch.bfloat16, device=DEV)
        rows_d = torch.zeros(B * L, dtype=torch.int32, device=DEV)
        nrows_d = torch.zeros(1, dtype=torch.int32, device=DEV)
        sets = torch.full((nl * B * S,), -1, dtype=torch.int32, device=DEV)
        sims = torch.zeros((nl * B * L,), dtype=torch.float32, device=DEV)
        sfs.sfs_cache_dump(session, sets, sims)
        sfs.sfs_generate_begin(session, prompt.to(DEV), B, P, L, pg)
        st = [SlowFastState.fresh(L, po) for _ in range(B)]
        tok = [prompt[b].tolist() + [shape.mask_id] * L for b in range(B)]
        caches = [C.FeatureCache(cfg, S, dtype=cache_dtype) for _ in range(B)]
        n_unmasked = [0] * B
        step = 0
        while step < max_steps and not all(s_.done for s_ in st):
            sets.fill_(-1)
            sfs.sfs_generate_steps(session, 1, trace, max_steps, dump, rows_d, nrows_d)
            torch.cuda.synchronize()
            rp, rr = step % kp == 0, step % kr == 0
            n_sel = S if (rp and rr) else (P if rp else 0) + (L if rr else n_adapt)
            gsets = sets.cpu().numpy()[: nl * B * n_sel].reshape(nl, B, n_sel)
            gsims = sims.cpu().numpy().reshape(nl, B, L)
            need = [(b, i) for b in range(B) for i in rows_needed(st[b])]
            n = int(nrows_d.item())
            assert rows_d[:n].tolist() == [b * S + P + i for (b, i) in need], step
            lg = dump[:n].cpu()
            got = lg.float().numpy().astype(np.float64)
            stats = RS.row_stats(W.bf16_bits(lg))
            for b in range(B):
                if st[b].done:
                    continue
                fast = st[b].phase == FAST
                span = (st[b].s_cycle, st[b].hi) if fast else None
                forced = lambda l, s_, c_, b=b: sorted(set(int(r) - b * S - P for r in gsets[l][b] if int(r) - b * S >= P))
                rec_c = {}
                idx = {i: j for j, (bb, i) in enumerate(need) if bb == b}
                mine = sorted(idx)
                ref = C.cached_forward(cfg, w_or, np.asarray(tok[b]), P, caches[b], kp, kr, rho, span=span, rows=[P + i for i in mine],
                                       select=forced, record=rec_c).astype(np.float64)
                logits_ok(step, b, got[[idx[i] for i in mine]], ref)
                for l in range(nl):
                    assert sorted(set(int(r) - b * S for r in gsets[l][b])) == rec_c["sets"][l], (step, b, l)
                    if not rr and n_adapt > 0:
                        cand = list(range(L)) if not fast else list(range(span[0], span[1]))
                        assert forced(l, None, None) == C.least_similar(gsims[l][b][cand], cand, min(n_adapt, len(cand))), (step, b, l)
                rec = slowfast_step(st[b], {i: int(stats["argmax"][j]) for i, j in idx.items()}, {i: int(stats["sq"][j]) for i, j in idx.items()}, po)
                for i, t in zip(rec.positions, rec.tokens):
                    tok[b][P + i] = t
                n_unmasked[b] += len(rec.positions)
                assert trace[step, b].tolist()[:6] == [rec.phase, rec.s, rec.hi, rec.e_cand, rec.stable, len(rec.positions)], (step, b, rec)
            step += 1
        out = torch.zeros((B, S), dtype=torch.int32, device=DEV)
        state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
        sfs.sfs_generate_end(session, out, state)
        sfs.sfs_check_device_status()
        o = out.cpu().tolist()
        for b in range(B):
            assert o[b] == tok[b], b                       # tokens written so far, masked positions still hold the mask id
            assert int(state[b, sfs.STATE_FIELDS.index("n_masked")]) == L - n_unmasked[b]
        return step, n_unmasked
    finally:
        sfs.sfs_cache_dump(session, None, None)
        sfs.sfs_cache_enable(session, 1, 1, 0.0, off=True)
        sfs.sfs_session_destroy(session)


@pytest.mark.parametrize("B,kp,kr,rho", [(2, 100, 4, 0.25), (1, 6, 3, 0.5)])
def test_cached_generation_is_reproduced_by_the_oracle_step_by_step(B, kp, kr, rho):
    """The whole cached decode loop on the tiny model (logit scale 60: slow and fast steps, spans, parallel unmasking)."""
    shape, model, cfg, w64 = tiny_setup(seed=0, logit_scale=60.0)
    P, L = 32, 64

    def logits_ok(step, b, got, ref):
        err = np.abs(got - ref)
        rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
        assert rel <= REL_L2, (step, b, rel)
        assert np.all(err <= max_abs_bar(shape.logit_scale) + 2.0 ** -8 * np.abs(ref)), (step, b, err.max())   # + rounding of the stored bf16 logit

    try:
        steps, n_unmasked = replay_cached_generation(shape, model, cfg, w64, B, P, L, kp, kr, rho, L, logits_ok)
        assert n_unmasked == [L] * B and steps < L                 # finished, with parallel unmasking on the way
    finally:
        model.close()


def test_cached_steps_at_widths_that_fill_no_tile():
    """Three heads of 128, d_ff 1000, vocabulary 5000, 23 + 49 tokens: the few-row projections, gathers and scatters of the
    partial steps with ragged tiles everywhere.  The tokens do not change, so the cached features stay exact and every step's
    response logits must equal the uncached forward pass (oracle and GPU)."""
    shape = W.Shape(n_layers=2, d_model=384, n_heads=3, head_dim=128, d_ff=1000, vocab=5000, mask_id=4999, rms_eps=1e-5,
                    rope_theta=10000.0, logit_scale=8.0)
    w = W.model_weights(shape, seed=6, gain_std=0.2)
    wd = {k: (v.to(DEV) if k != "layers" else [{kk: vv.to(DEV) for kk, vv in lw.items()} for lw in v]) for k, v in w.items()}
    model = sfs.Model(shape, wd)
    cfg = F.ModelConfig(**shape.asdict())
    w64 = W.weights_to_numpy(w, np.float64)
    B, P, L = 1, 23, 49
    S = P + L
    tok = torch.cat([W.prompt_ids(B, P, shape.vocab - 2, seed=2), torch.full((B, L), shape.mask_id, dtype=torch.int32)], dim=1)
    d_tok = tok.to(DEV)
    session = sfs.sfs_session_create(model, B, S)
    try:
        ref = F.forward(cfg, w64, tok.numpy(), rows=[(0, t) for t in range(S)], dtype=np.float64)
        plain = torch.zeros((B * S, shape.vocab), dtype=torch.float32, device=DEV)
        sfs.sfs_forward(session, d_tok, B, S, None, None, B * S, plain, sfs.LOGITS_F32)
        plain = plain.cpu().double().numpy()
        scale = np.abs(ref).max()
        sfs.sfs_cache_enable(session, 100, 3, 0.3)
        logits = torch.zeros((B * S, shape.vocab), dtype=torch.float32, device=DEV)
        for step in range(6):
            fast = step in (2, 4)
            st = state_tensor(B, 1, 10, 31) if fast else state_tensor(B)
            n_sel = sfs.sfs_forward_cached(session, d_tok, B, S, P, st, None, None, B * S, logits, sfs.LOGITS_F32)
            sfs.sfs_check_device_status()
            assert n_sel == (S if step == 0 else (L if step % 3 == 0 else C.adaptive_count(0.3, L)))
            got = logits.cpu().double().numpy()
            lo = 0 if step == 0 else P                       # prompt rows are defined on the step that refreshes the prompt
            rel = np.linalg.norm(got[lo:] - ref[lo:]) / np.linalg.norm(ref[lo:])
            rel_plain = np.linalg.norm(got[lo:] - plain[lo:]) / np.linalg.norm(plain[lo:])
            assert rel <= REL_L2, (step, rel)
            # the same features through other tile shapes and sum orders: far inside the rounding noise of either path
            assert rel_plain <= 3e-3 and np.abs(got[lo:] - plain[lo:]).max() <= 2e-2 * scale, (step, rel_plain)
    finally:
        sfs.sfs_session_destroy(session)
        model.close()
