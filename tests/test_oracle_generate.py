"""The oracle's full denoising loop on the tiny workload: invariants of Section 3.1 (known tokens are
preserved; the sequence ends without masks) and agreement between `generate` and the teacher-forced `replay`."""
import numpy as np

from oracle import forward as F
from oracle import generate as G
from oracle.scheduler import SlowFastParams
from paper_2506_10848_b200 import workloads as W


def test_tiny_full_loop_invariants_and_replay():
    shape = W.TINY
    cfg = F.ModelConfig(**shape.asdict())
    w = W.weights_to_numpy(W.model_weights(shape, seed=0), np.float64)
    prompt = W.prompt_ids(1, 32, 4094, seed=0)[0].tolist()
    L = 64
    p = SlowFastParams()
    captured = {}
    y, trace = G.generate(cfg, w, prompt, L, p, dtype=np.float64,
                          logits_hook=lambda step, rows, lg: captured.__setitem__(step, (list(rows), lg.copy())))
    assert y[:32] == prompt and len(y) == 96
    assert 1 <= len(trace) <= L
    seen = sorted(i for r in trace for i in r.positions)
    assert seen == list(range(L))
    assert all(0 <= t < shape.vocab for t in y)
    # teacher-forced replay with the captured logits reproduces the trace exactly
    def feed(step, rows):
        r, lg = captured[step]
        assert r == rows
        return lg
    y2, trace2 = G.replay(L, p, feed)
    assert [r.key() for r in trace2] == [r.key() for r in trace]
    assert y2 == y[32:]


def _tiny():
    shape = W.TINY
    cfg = F.ModelConfig(**shape.asdict())
    w = W.weights_to_numpy(W.model_weights(shape, seed=0), np.float64)
    prompt = W.prompt_ids(1, 32, 4094, seed=0)[0].tolist()
    return shape, cfg, w, prompt


def test_generate_feeds_the_scheduler_the_logits_of_the_response_rows():
    """Pins the row mapping of `generate`: the logits of step k's row i are the predictor's output at sequence
    position P + i for the tokens as they stood before step k (rebuilt here from the trace alone)."""
    shape, cfg, w, prompt = _tiny()
    P, L = len(prompt), 24
    captured = {}
    y, trace = G.generate(cfg, w, prompt, L, SlowFastParams(), dtype=np.float64,
                          logits_hook=lambda step, rows, lg: captured.__setitem__(step, (list(rows), lg.copy())))
    tok = list(prompt) + [cfg.mask_id] * L
    for k, rec in enumerate(trace):
        full = F.forward(cfg, w, np.asarray([tok]), dtype=np.float64)
        rows, lg = captured[k]
        want = np.asarray(full).reshape(P + L, -1)[[P + i for i in rows]].astype(np.float32)
        assert np.array_equal(lg, want), k
        # a shifted mapping (row i read at position i, or at P + i - 1) would not reproduce these logits
        wrong = np.asarray(full).reshape(P + L, -1)[[P + i - 1 for i in rows]].astype(np.float32)
        assert not np.array_equal(lg, wrong)
        for i, t in zip(rec.positions, rec.tokens):
            tok[P + i] = t
    assert tok == y


def test_cached_generation_with_everything_refreshed_is_the_uncached_generation():
    shape, cfg, w, prompt = _tiny()
    L = 24
    p = SlowFastParams()
    lg_a, lg_b = {}, {}
    ya, ta = G.generate(cfg, w, prompt, L, p, logits_hook=lambda s, r, lg: lg_a.__setitem__(s, lg.copy()))
    yb, tb = G.generate_cached(cfg, w, prompt, L, p, 1, 1, 0.25, logits_hook=lambda s, r, lg: lg_b.__setitem__(s, lg.copy()))
    assert ya == yb and [r.key() for r in ta] == [r.key() for r in tb]
    assert all(np.allclose(lg_a[s], lg_b[s], rtol=1e-6, atol=1e-6) for s in lg_a)
    # rho = 1 with the prompt refreshed every step recomputes every row as well
    yc, tc = G.generate_cached(cfg, w, prompt, L, p, 1, 1000, 1.0)
    assert yc == ya and [r.key() for r in tc] == [r.key() for r in ta]


def test_cached_generation_schedule_span_and_restart():
    """The cache counter restarts with the generation (step 0 recomputes every row); accelerated steps restrict the
    adaptive candidates to the span; the sequence still ends without masks and every position is decoded once."""
    dct = W.TINY.asdict(); dct["logit_scale"] = 60.0                     # both thresholds fire: slow and fast steps occur
    shape = W.Shape(**dct)
    cfg = F.ModelConfig(**shape.asdict())
    w = W.weights_to_numpy(W.model_weights(shape, seed=0), np.float64)
    prompt = W.prompt_ids(1, 32, 4094, seed=0)[0].tolist()
    P, L, kp, kr, rho = 32, 32, 100, 4, 0.25
    recs = {}
    y, trace = G.generate_cached(cfg, w, prompt, L, SlowFastParams(), kp, kr, rho, record_hook=lambda s, r: recs.__setitem__(s, r))
    assert sorted(i for r in trace for i in r.positions) == list(range(L)) and y[:P] == prompt
    assert recs[0]["sets"][0] == list(range(P + L))
    n_adapt = 8
    saw_fast = False
    for s, r in enumerate(trace):
        sets = recs[s]["sets"][0]
        if s % kr == 0:
            assert set(P + i for i in range(L)) <= set(sets)
        else:
            assert all(q >= P for q in sets) and len(sets) <= n_adapt
            if r.phase == 1:
                saw_fast = True
                assert all(r.s <= q - P < r.hi for q in sets), (s, sets, r.s, r.hi)
                assert len(sets) == min(n_adapt, r.hi - r.s)
            else:
                assert len(sets) == n_adapt
    assert saw_fast
    y2, trace2 = G.generate_cached(cfg, w, prompt, L, SlowFastParams(), kp, kr, rho)
    assert y2 == y and [r.key() for r in trace2] == [r.key() for r in trace]


def test_cached_generation_hands_the_span_of_an_accelerated_step_to_the_cache(monkeypatch):
    """What the cache is told per step: the span [s_cycle, hi) when the step is an accelerated one, nothing otherwise
    (the spans of the run above can cover the whole response, where the restriction is invisible in the sets)."""
    dct = W.TINY.asdict(); dct["logit_scale"] = 60.0
    shape = W.Shape(**dct)
    cfg = F.ModelConfig(**shape.asdict())
    w = W.weights_to_numpy(W.model_weights(shape, seed=0), np.float64)
    prompt = W.prompt_ids(1, 32, 4094, seed=0)[0].tolist()
    seen = []
    real = G.C.cached_forward

    def spy(*a, **k):
        seen.append((k.get("span"), list(k.get("rows"))))
        return real(*a, **k)

    monkeypatch.setattr(G.C, "cached_forward", spy)
    y, trace = G.generate_cached(cfg, w, prompt, 32, SlowFastParams(), 100, 4, 0.25)
    assert len(seen) == len(trace) and any(r.phase == 1 for r in trace)
    for r, (span, rows) in zip(trace, seen):
        assert span == ((r.s, r.hi) if r.phase == 1 else None), (r.step, span)
        assert all(32 <= q < 64 for q in rows)                        # logits rows are sequence positions of the response
