"""ORACLE (test infrastructure): the mask predictor p_theta as a plain numpy forward pass.

The paper (Section 3.1, Eq. 2) only requires a bidirectional predictor P_theta(r_0 | c, y^(k)); the
architecture is the LLaDA-style one the workload definitions give: pre-norm blocks without a causal mask,

    x0 = E[tok]
    per layer:  h = RMSNorm(x; g_attn);  q, k, v = h Wq^T, h Wk^T, h Wv^T  (no bias)
                RoPE on q, k with the absolute position 0..S-1 over prompt || response,
                    pairing (j, j + dh/2), angle = pos * theta^(-2j/dh)
                a = softmax(q k^T / sqrt(dh)) v   over ALL S positions of the same sequence
                x += a Wo^T
                h = RMSNorm(x; g_mlp);  x += (silu(h Wg^T) * (h Wu^T)) Wd^T
    logits = logit_scale * RMSNorm(x; g_final) W_lm^T

All arithmetic is done in `dtype` (float64 by default, float32 to keep large shapes affordable); the only
library primitives used are numpy's matmul, exp and sqrt.  No blocking, no fusion.
"""
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import numpy as np


@dataclass
class ModelConfig:
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    mask_id: int
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    logit_scale: float = 1.0


def rms_norm(x, g, eps):
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + x.dtype.type(eps)) * g


def rope(x, positions, theta):
    """x: [S, H, dh]; rotate pairs (j, j + dh/2) by positions * theta^(-2j/dh)."""
    dh = x.shape[-1]
    half = dh // 2
    j = np.arange(half, dtype=np.float64)
    inv_freq = theta ** (-2.0 * j / dh)
    ang = positions.astype(np.float64)[:, None] * inv_freq[None, :]          # [S, half], exact in double
    cos = np.cos(ang).astype(x.dtype)[:, None, :]
    sin = np.sin(ang).astype(x.dtype)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1)


def attention(q, k, v):
    """q, k, v: [S, H, dh] of one sequence; bidirectional (no mask)."""
    dh = q.shape[-1]
    s = np.einsum("qhd,khd->hqk", q, k) / q.dtype.type(np.sqrt(dh))
    s = s - s.max(axis=-1, keepdims=True)
    p = np.exp(s)
    p = p / p.sum(axis=-1, keepdims=True)
    return np.einsum("hqk,khd->qhd", p, v)


def silu(x):
    return x / (1.0 + np.exp(-x))


def forward(cfg: ModelConfig, w: Dict, tokens: np.ndarray, rows: Optional[Sequence[Sequence[int]]] = None,
            dtype=np.float64, collect: Optional[Dict] = None) -> np.ndarray:
    """tokens: int [B, S] (masked positions hold cfg.mask_id).  rows: list of (b, pos) whose logits are
    wanted, default every position.  Returns logits [R, V] in `dtype`.

    `collect`, if a dict, receives intermediate activations by name (for kernel-level parity tests).
    """
    tokens = np.asarray(tokens)
    B, S = tokens.shape
    H, dh, d = cfg.n_heads, cfg.head_dim, cfg.d_model
    cast = lambda a: np.asarray(a, dtype=dtype)
    pos = np.arange(S)
    x = cast(w["tok_emb"])[tokens]                                   # [B, S, d]
    if collect is not None:
        collect["embed"] = x.copy()
    for l in range(cfg.n_layers):
        lw = w["layers"][l]
        h = rms_norm(x, cast(lw["attn_norm"]), cfg.rms_eps)
        q = h @ cast(lw["wq"]).T
        k = h @ cast(lw["wk"]).T
        v = h @ cast(lw["wv"]).T
        a = np.empty_like(q)
        for b in range(B):
            qb = rope(q[b].reshape(S, H, dh), pos, cfg.rope_theta)
            kb = rope(k[b].reshape(S, H, dh), pos, cfg.rope_theta)
            a[b] = attention(qb, kb, v[b].reshape(S, H, dh)).reshape(S, H * dh)
            if collect is not None and b == 0:
                collect.setdefault("q_rope", {})[l] = qb.reshape(S, H * dh).copy()
                collect.setdefault("k_rope", {})[l] = kb.reshape(S, H * dh).copy()
        if collect is not None:
            collect.setdefault("attn_norm", {})[l] = h.copy()
            collect.setdefault("v", {})[l] = v.copy()
            collect.setdefault("attn", {})[l] = a.copy()
        x = x + a @ cast(lw["wo"]).T
        h = rms_norm(x, cast(lw["mlp_norm"]), cfg.rms_eps)
        g = h @ cast(lw["w_gate"]).T
        u = h @ cast(lw["w_up"]).T
        hid = silu(g) * u
        x = x + hid @ cast(lw["w_down"]).T
        if collect is not None:
            collect.setdefault("hidden", {})[l] = hid.copy()
            collect.setdefault("x", {})[l] = x.copy()
    if rows is None:
        rows = [(b, t) for b in range(B) for t in range(S)]
    sel = np.stack([x[b, t] for (b, t) in rows]) if len(rows) else np.zeros((0, d), dtype)
    hf = rms_norm(sel, cast(w["final_norm"]), cfg.rms_eps)
    if collect is not None:
        collect["final_h"] = hf.copy()
    logits = (hf @ cast(w["lm_head"]).T) * dtype(cfg.logit_scale)
    return logits
