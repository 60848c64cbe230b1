"""ORACLE (test infrastructure): the mask predictor with dLLM-Cache-style feature caching, plain numpy.

The paper only says that its sampler "integrates" an adaptive feature cache that reuses the prompt's and the
response's intermediate features across denoising steps and refreshes them at a long and a short interval
(Section 2.2; the (K_p, K_r) pairs of Table 4).  The mechanism is therefore a reading, stated once here:

  Per layer l the cache holds, for every position of the sequence, the rotated key K_l, the value V_l, the
  attention branch's residual increment A_l = attention(...) Wo^T and the MLP branch's increment F_l.
  Step counter t starts at 0.  refresh_p = (t mod K_p == 0), refresh_r = (t mod K_r == 0).
  x_0 = E[tok] is always computed for every position (a newly unmasked token changes its embedding).
  In layer l the set R_l of recomputed positions is
        prompt positions, if refresh_p;  plus
        all response positions, if refresh_r;  otherwise the adaptive set: with h = RMSNorm(x) and
        v_i = h_i Wv^T for the candidate response positions C, the k = min(ceil(rho * L), |C|) candidates (the product taken in double) whose
        cosine similarity  <v_i, V_l[i]> / (|v_i| |V_l[i]|)  to their cached value is smallest (ties: lower
        position first).  C is every response position in a slow step and the span [s_cycle, hi) in a fast
        step (out-of-span positions keep their cached features while the span is decoded).
  For i in R_l:  K_l[i], V_l[i] are overwritten from the fresh h_i; the attention of query i runs over ALL cached
  keys / values of its sequence (with the rows of R_l already overwritten); A_l[i] = a_i Wo^T is overwritten.
  Then  x += A_l  for every position (cached rows reuse their old increment);  for i in R_l the MLP is evaluated on
  RMSNorm(x_i) and F_l[i] overwritten;  x += F_l  for every position.
  With R_l = everything this is the uncached forward pass, operation for operation.

`select` may be supplied to force the adaptive sets (e.g. the sets another implementation chose): the cached
outputs of two implementations are compared under the same schedule.
"""
import math
from typing import Callable, Dict, List, Optional, Sequence

import numpy as np

from . import forward as F


class FeatureCache:
    def __init__(self, cfg: F.ModelConfig, S: int, dtype=np.float64):
        z = lambda: [np.zeros((S, cfg.d_model), dtype) for _ in range(cfg.n_layers)]
        self.K, self.V, self.A, self.Fo = z(), z(), z(), z()
        self.t = 0
        self.dtype = dtype


def cosine_similarity(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """Row-wise <a, b> / (|a| |b|); 0 where a norm vanishes."""
    num = np.sum(a * b, axis=-1)
    den = np.sqrt(np.sum(a * a, axis=-1)) * np.sqrt(np.sum(b * b, axis=-1))
    return np.where(den > 0, num / np.where(den > 0, den, 1), 0.0)


def least_similar(sims: np.ndarray, candidates: Sequence[int], k: int) -> List[int]:
    """The k candidates with the smallest similarity, ties to the lower position; returned ascending."""
    order = sorted(range(len(candidates)), key=lambda j: (float(sims[j]), candidates[j]))
    return sorted(candidates[j] for j in order[:k])


def adaptive_count(rho: float, L: int) -> int:
    """ceil(rho * L), one IEEE double multiply."""
    return int(math.ceil(float(rho) * float(L)))


def cached_forward(cfg: F.ModelConfig, w: Dict, tokens: Sequence[int], P: int, cache: FeatureCache,
                   k_prompt: int, k_response: int, rho: float, span: Optional[Sequence[int]] = None,
                   rows: Optional[Sequence[int]] = None,
                   select: Optional[Callable[[int, np.ndarray, List[int]], List[int]]] = None,
                   record: Optional[Dict] = None) -> np.ndarray:
    """One denoising step's forward pass of ONE sequence under the cache rule above; advances cache.t.

    tokens: ids [S]; P: prompt length; span: (lo, hi) response positions of a fast step, None in a slow step;
    rows: sequence positions whose logits are wanted (default all).  `select(l, sims, candidates)` overrides the
    adaptive choice (response positions in, response positions out).  `record`, if a dict, receives per layer the
    recomputed positions ("sets") and the similarities ("sims").  Returns logits [len(rows), V].
    """
    dtype = cache.dtype
    cast = lambda a: np.asarray(a, dtype=dtype)
    tokens = np.asarray(tokens)
    S = tokens.shape[0]
    L = S - P
    H, dh = cfg.n_heads, cfg.head_dim
    refresh_p = (cache.t % k_prompt) == 0
    refresh_r = (cache.t % k_response) == 0
    cand = list(range(L)) if span is None else list(range(span[0], span[1]))
    k_adapt = min(adaptive_count(rho, L), len(cand))
    x = cast(w["tok_emb"])[tokens]                                   # [S, d]
    pos_all = np.arange(S)
    for l in range(cfg.n_layers):
        lw = w["layers"][l]
        h = F.rms_norm(x, cast(lw["attn_norm"]), cfg.rms_eps)
        R: List[int] = list(range(P)) if refresh_p else []
        if refresh_r:
            R += [P + i for i in range(L)]
        elif k_adapt > 0:
            crow = np.asarray([P + i for i in cand])
            v_new = h[crow] @ cast(lw["wv"]).T
            sims = cosine_similarity(v_new, cache.V[l][crow])
            chosen = select(l, sims, cand) if select is not None else least_similar(sims, cand, k_adapt)
            R += [P + i for i in chosen]
            if record is not None:
                record.setdefault("sims", {})[l] = sims.copy()
        R = sorted(set(R))
        if record is not None:
            record.setdefault("sets", {})[l] = list(R)
        if R:
            Ri = np.asarray(R)
            hr = h[Ri]
            q = F.rope((hr @ cast(lw["wq"]).T).reshape(len(R), H, dh), pos_all[Ri], cfg.rope_theta)
            kk = F.rope((hr @ cast(lw["wk"]).T).reshape(len(R), H, dh), pos_all[Ri], cfg.rope_theta)
            cache.K[l][Ri] = kk.reshape(len(R), H * dh)
            cache.V[l][Ri] = hr @ cast(lw["wv"]).T
            # queries of R against every cached key / value of the sequence
            Kc = cache.K[l].reshape(S, H, dh)
            Vc = cache.V[l].reshape(S, H, dh)
            s = np.einsum("qhd,khd->hqk", q, Kc) / dtype(np.sqrt(dh))
            s = s - s.max(axis=-1, keepdims=True)
            p = np.exp(s)
            p = p / p.sum(axis=-1, keepdims=True)
            a = np.einsum("hqk,khd->qhd", p, Vc).reshape(len(R), H * dh)
            cache.A[l][Ri] = a @ cast(lw["wo"]).T
        x = x + cache.A[l]
        if R:
            h2 = F.rms_norm(x[Ri], cast(lw["mlp_norm"]), cfg.rms_eps)
            hid = F.silu(h2 @ cast(lw["w_gate"]).T) * (h2 @ cast(lw["w_up"]).T)
            cache.Fo[l][Ri] = hid @ cast(lw["w_down"]).T
        x = x + cache.Fo[l]
    cache.t += 1
    if rows is None:
        rows = list(range(S))
    sel = x[np.asarray(rows, dtype=np.int64)] if len(rows) else np.zeros((0, cfg.d_model), dtype)
    hf = F.rms_norm(sel, cast(w["final_norm"]), cfg.rms_eps)
    return (hf @ cast(w["lm_head"]).T) * dtype(cfg.logit_scale)
