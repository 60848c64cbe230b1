"""Pins of the cached forward pass of the oracle (oracle/cache.py) against what the cache rule fixes by itself:
the uncached forward pass (oracle/forward.py, pinned on its own) whenever nothing is reused or nothing changed, a
closed form when nothing is recomputed, and brute force for the least-similar selection."""
import itertools
import math

import numpy as np
import pytest

from oracle import cache as C
from oracle import forward as F
from paper_2506_10848_b200 import workloads as W

SHAPE = W.Shape(n_layers=3, d_model=64, n_heads=2, head_dim=32, d_ff=96, vocab=128, mask_id=127,
                rms_eps=1e-5, rope_theta=10000.0, logit_scale=2.0)
CFG = F.ModelConfig(**SHAPE.asdict())
WTS = W.weights_to_numpy(W.model_weights(SHAPE, seed=5, std=0.2, gain_std=0.3), np.float64)   # every norm its own gains
P, L = 6, 10
S = P + L


def toks(seed, masked=L):
    g = np.random.default_rng(seed)
    t = g.integers(0, 126, size=S)
    t[S - masked:] = CFG.mask_id
    return t


def test_everything_refreshed_is_the_uncached_forward():
    t0 = toks(1)
    cache = C.FeatureCache(CFG, S)
    for step in range(3):                                   # K_p = K_r = 1: every step recomputes every row
        t = t0.copy(); t[P:P + step] = step + 3
        got = C.cached_forward(CFG, WTS, t, P, cache, 1, 1, 0.25)
        ref = F.forward(CFG, WTS, t[None, :])
        assert np.allclose(got, ref, rtol=1e-11, atol=1e-11)


@pytest.mark.parametrize("kp,kr,rho", [(100, 5, 0.25), (3, 2, 0.0), (7, 7, 1.0)])
def test_unchanged_tokens_reproduce_the_uncached_logits_under_any_schedule(kp, kr, rho):
    """If no token changes, every cached feature equals what would be recomputed, so the schedule cannot matter."""
    t = toks(2, masked=4)
    ref = F.forward(CFG, WTS, t[None, :])
    cache = C.FeatureCache(CFG, S)
    for step in range(9):
        got = C.cached_forward(CFG, WTS, t, P, cache, kp, kr, rho, span=(2, 7) if step % 2 else None)
        assert np.allclose(got, ref, rtol=1e-10, atol=1e-10), step


def test_nothing_recomputed_moves_only_the_changed_embedding():
    """rho = 0 on a non-refresh step: the residual stream is the fresh embedding plus cached increments, so the final
    hidden state of the changed position moves by exactly E[new] - E[old] and no other position moves."""
    t = toks(3)
    cache = C.FeatureCache(CFG, S)
    C.cached_forward(CFG, WTS, t, P, cache, 100, 100, 0.0)             # t = 0: fills the cache
    t2 = t.copy(); t2[P + 4] = 17
    x_old = np.asarray(WTS["tok_emb"])[t] + sum(cache.A) + sum(cache.Fo)
    got = C.cached_forward(CFG, WTS, t2, P, cache, 100, 100, 0.0)
    x_new = x_old.copy(); x_new[P + 4] += WTS["tok_emb"][17] - WTS["tok_emb"][CFG.mask_id]
    ref = (F.rms_norm(x_new, WTS["final_norm"], CFG.rms_eps) @ WTS["lm_head"].T) * CFG.logit_scale
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-12)
    others = [i for i in range(S) if i != P + 4]
    assert np.allclose(got[others], (F.rms_norm(x_old, WTS["final_norm"], CFG.rms_eps) @ WTS["lm_head"].T * CFG.logit_scale)[others])


def test_forcing_all_candidates_equals_rho_one_and_prompt_rows_stay_cached():
    t = toks(4)
    a, b = C.FeatureCache(CFG, S), C.FeatureCache(CFG, S)
    for cch in (a, b):
        C.cached_forward(CFG, WTS, t, P, cch, 100, 100, 1.0)
    t2 = t.copy(); t2[P] = 9; t2[P + 1] = 11
    ra, rb = {}, {}
    la = C.cached_forward(CFG, WTS, t2, P, a, 100, 100, 1.0, record=ra)
    lb = C.cached_forward(CFG, WTS, t2, P, b, 100, 100, 0.1, select=lambda l, s, c: list(c), record=rb)
    assert np.array_equal(la, lb)
    assert all(ra["sets"][l] == [P + i for i in range(L)] for l in range(CFG.n_layers))   # no prompt row recomputed
    # the prompt's cached keys are the ones of step 0 although prompt rows attend to the (changed) response
    full = F.forward(CFG, WTS, t2[None, :])
    assert not np.allclose(la[:P], full[:P], rtol=1e-6, atol=1e-6)


def test_schedule_counter_and_fast_step_candidates():
    t = toks(5)
    cache = C.FeatureCache(CFG, S)
    seen = []
    for step in range(7):
        rec = {}
        tt = t.copy(); tt[P:P + step] = 5 + step
        C.cached_forward(CFG, WTS, tt, P, cache, 6, 3, 0.3, span=(3, 6) if step in (1, 4) else None, record=rec)
        seen.append(rec["sets"][0])
    k = C.adaptive_count(0.3, L)
    assert k == 3 and C.adaptive_count(0.25, 10) == 3 and C.adaptive_count(0.5, 10) == 5      # ceil(3.0), ceil(2.5), ceil(5.0)
    assert C.adaptive_count(0.1, 10) == 1 and C.adaptive_count(0.0, 10) == 0 and C.adaptive_count(1.0, 10) == 10
    assert C.adaptive_count(0.25, 512) == 128 and C.adaptive_count(0.3, 7) == 3
    allr = [P + i for i in range(L)]
    assert seen[0] == list(range(S)) and seen[6] == list(range(S))       # t = 0, 6: both intervals fire
    assert seen[3] == allr                                               # t = 3: response interval only
    assert len(seen[2]) == k and len(seen[5]) == k and set(seen[2]) <= set(allr)
    assert len(seen[1]) == min(k, 3) and set(seen[1]) <= {P + 3, P + 4, P + 5}   # fast step: candidates = the span
    assert cache.t == 7


def test_least_similar_matches_brute_force_and_picks_the_planted_row():
    g = np.random.default_rng(0)
    for _ in range(50):
        n = int(g.integers(1, 7)); k = int(g.integers(0, n + 1))
        cand = sorted(g.choice(20, size=n, replace=False).tolist())
        sims = np.round(g.normal(size=n), 1)                              # rounding plants ties
        got = C.least_similar(sims, cand, k)
        best = min(itertools.combinations(range(n), k), key=lambda c: sorted((sims[j], cand[j]) for j in c))
        assert got == sorted(cand[j] for j in best)
    a = g.normal(size=(5, 8)); b = a.copy(); b[3] = -a[3]; b[1] = 2 * a[1]
    s = C.cosine_similarity(a, b)
    assert np.allclose(s, [1, 1, 1, -1, 1]) and C.least_similar(s, [0, 1, 2, 3, 4], 1) == [3]
    assert C.cosine_similarity(np.zeros((1, 4)), np.ones((1, 4)))[0] == 0.0


def test_changed_token_is_the_least_similar_value_in_the_first_layer():
    t = toks(6)
    cache = C.FeatureCache(CFG, S)
    C.cached_forward(CFG, WTS, t, P, cache, 100, 100, 0.1)
    t2 = t.copy(); t2[P + 7] = 33
    rec = {}
    C.cached_forward(CFG, WTS, t2, P, cache, 100, 100, 0.1, record=rec)
    assert rec["sets"][0] == [P + 7]                                      # k = ceil(0.1 * 10) = 1
    assert np.allclose(np.delete(rec["sims"][0], 7), 1.0)                 # layer 0 sees only the embeddings
