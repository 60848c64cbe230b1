"""Pins for the oracle's mask-predictor forward (Section 3.1, Eq. 2; architecture from the workload
definitions): closed forms, invariances and library routines on the special cases they cover."""
import numpy as np
import pytest
import torch

from oracle import forward as F


def tiny_cfg(**kw):
    base = dict(n_layers=2, d_model=32, n_heads=2, head_dim=16, d_ff=48, vocab=97, mask_id=96,
                rms_eps=1e-5, rope_theta=10000.0, logit_scale=2.0)
    base.update(kw)
    return F.ModelConfig(**base)


def rand_weights(cfg, seed=0, std=0.3):
    rng = np.random.default_rng(seed)
    d, ff, V = cfg.d_model, cfg.d_ff, cfg.vocab
    n = lambda *s: rng.normal(0, std, s)
    return {"tok_emb": n(V, d), "final_norm": 1 + 0.1 * n(d), "lm_head": n(V, d),
            "layers": [{"attn_norm": 1 + 0.1 * n(d), "wq": n(d, d), "wk": n(d, d), "wv": n(d, d), "wo": n(d, d),
                        "mlp_norm": 1 + 0.1 * n(d), "w_gate": n(ff, d), "w_up": n(ff, d), "w_down": n(d, ff)}
                       for _ in range(cfg.n_layers)]}


def test_rmsnorm_closed_forms():
    g = np.array([1.0, 2.0, -1.0, 0.5])
    x = np.full((3, 4), 7.0)
    assert np.allclose(F.rms_norm(x, g, 0.0), np.broadcast_to(g, (3, 4)))          # constant row -> gain
    x = np.array([[3.0, 4.0, 0.0, 0.0]])
    assert np.allclose(F.rms_norm(x, np.ones(4), 0.0), x / 2.5)                     # rms of (3,4,0,0) = 2.5
    t = torch.tensor(np.random.default_rng(0).normal(size=(5, 16)))
    ref = torch.nn.functional.rms_norm(t, (16,), torch.ones(16, dtype=t.dtype), 1e-5).numpy()
    assert np.allclose(F.rms_norm(t.numpy(), np.ones(16), 1e-5), ref, atol=1e-12)


def test_rope_properties():
    rng = np.random.default_rng(1)
    S, H, dh = 9, 2, 16
    q, k = rng.normal(size=(S, H, dh)), rng.normal(size=(S, H, dh))
    pos = np.arange(S)
    rq = F.rope(q, pos, 10000.0)
    assert np.allclose(rq[0], q[0])                                                  # position 0: identity
    assert np.allclose(np.linalg.norm(rq, axis=-1), np.linalg.norm(q, axis=-1))      # a rotation
    # relative-position property: <R_m q, R_n k> depends on m - n only
    qq = np.broadcast_to(q[:1], (S, H, dh)); kk = np.broadcast_to(k[:1], (S, H, dh))
    a = np.einsum("shd,thd->hst", F.rope(qq, pos, 10000.0), F.rope(kk, pos, 10000.0))
    b = np.einsum("shd,thd->hst", F.rope(qq, pos + 5, 10000.0), F.rope(kk, pos + 5, 10000.0))
    assert np.allclose(a, b)
    # first pair (j = 0, partner dh/2) rotates by exactly `pos` radians, counter-clockwise
    e = np.zeros((S, 1, dh)); e[:, 0, 0] = 1.0
    r = F.rope(e, pos, 10000.0)
    assert np.allclose(r[:, 0, 0], np.cos(pos)) and np.allclose(r[:, 0, dh // 2], np.sin(pos))
    # last pair rotates by pos * theta^(-(dh-2)/dh)
    e = np.zeros((S, 1, dh)); e[:, 0, dh // 2 - 1] = 1.0
    r = F.rope(e, pos, 10000.0)
    assert np.allclose(r[:, 0, dh - 1], np.sin(pos * 10000.0 ** (-(dh - 2) / dh)))


def test_attention_against_library_and_limits():
    rng = np.random.default_rng(2)
    S, H, dh = 11, 3, 8
    q, k, v = (rng.normal(size=(S, H, dh)) for _ in range(3))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(q).permute(1, 0, 2)[None], torch.tensor(k).permute(1, 0, 2)[None],
        torch.tensor(v).permute(1, 0, 2)[None], is_causal=False)[0].permute(1, 0, 2).numpy()
    assert np.allclose(F.attention(q, k, v), ref, atol=1e-12)
    assert np.allclose(F.attention(np.zeros_like(q), k, v), np.broadcast_to(v.mean(0), (S, H, dh)))  # q = 0 -> mean of v
    big = np.zeros_like(k); big[4] = 50.0                                            # key 4 dominates
    assert np.allclose(F.attention(np.ones_like(q), big, v), np.broadcast_to(v[4], (S, H, dh)), atol=1e-9)


def test_silu():
    x = np.linspace(-6, 6, 25)
    assert np.allclose(F.silu(x), torch.nn.functional.silu(torch.tensor(x)).numpy(), atol=1e-14)


def test_forward_closed_form_when_blocks_are_silent():
    cfg = tiny_cfg()
    w = rand_weights(cfg)
    for lw in w["layers"]:
        lw["wo"][:] = 0.0
        lw["w_down"][:] = 0.0
    tok = np.array([[3, 96, 5, 96, 96, 1]])
    logits = F.forward(cfg, w, tok)
    e = w["tok_emb"][tok[0]]
    h = e / np.sqrt((e * e).mean(-1, keepdims=True) + cfg.rms_eps) * w["final_norm"]
    assert np.allclose(logits, cfg.logit_scale * h @ w["lm_head"].T, atol=1e-12)


def test_forward_is_bidirectional_batch_independent_and_row_selectable():
    cfg = tiny_cfg()
    w = rand_weights(cfg, 3)
    rng = np.random.default_rng(4)
    tok = rng.integers(0, 96, (2, 7))
    base = F.forward(cfg, w, tok).reshape(2, 7, -1)
    t2 = tok.copy(); t2[0, 6] = (t2[0, 6] + 1) % 96                                 # change the LAST token of sequence 0
    pert = F.forward(cfg, w, t2).reshape(2, 7, -1)
    assert np.abs(pert[0, 0] - base[0, 0]).max() > 1e-6                              # position 0 sees it: no causal mask
    assert np.array_equal(pert[1], base[1])                                          # other sequence untouched
    rows = [(1, 2), (0, 5)]
    sel = F.forward(cfg, w, tok, rows=rows)
    assert np.allclose(sel[0], base[1, 2]) and np.allclose(sel[1], base[0, 5])
    # the same sequence alone gives the same logits (attention never crosses sequences)
    alone = F.forward(cfg, w, tok[1:2]).reshape(7, -1)
    assert np.allclose(alone, base[1], atol=1e-12)
    cfg2 = tiny_cfg(logit_scale=6.0)
    assert np.allclose(F.forward(cfg2, w, tok).reshape(2, 7, -1), 3.0 * base)


def test_single_layer_against_an_independent_torch_composition():
    """One block assembled from torch library routines (linear, SDPA, rms_norm, silu) with rotary applied
    through complex multiplication — a different route to the same rotation."""
    cfg = tiny_cfg(n_layers=1)
    w = rand_weights(cfg, 5)
    tok = np.array([[7, 96, 96, 11, 2]])
    S, H, dh, d = 5, cfg.n_heads, cfg.head_dim, cfg.d_model
    T = lambda a: torch.tensor(a, dtype=torch.float64)
    lw = w["layers"][0]
    x = T(w["tok_emb"])[torch.tensor(tok[0])]
    nrm = lambda t, g: torch.nn.functional.rms_norm(t, (d,), T(g), cfg.rms_eps)
    h = nrm(x, lw["attn_norm"])
    q = torch.nn.functional.linear(h, T(lw["wq"])).view(S, H, dh)
    k = torch.nn.functional.linear(h, T(lw["wk"])).view(S, H, dh)
    v = torch.nn.functional.linear(h, T(lw["wv"])).view(S, H, dh)
    ang = torch.arange(S, dtype=torch.float64)[:, None] * cfg.rope_theta ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh)
    rot = torch.polar(torch.ones_like(ang), ang)[:, None, :]
    cplx = lambda t: torch.complex(t[..., : dh // 2], t[..., dh // 2:])
    back = lambda c: torch.cat([c.real, c.imag], -1)
    q, k = back(cplx(q) * rot), back(cplx(k) * rot)
    a = torch.nn.functional.scaled_dot_product_attention(q.permute(1, 0, 2)[None], k.permute(1, 0, 2)[None],
                                                         v.permute(1, 0, 2)[None])[0].permute(1, 0, 2).reshape(S, d)
    x = x + torch.nn.functional.linear(a, T(lw["wo"]))
    h = nrm(x, lw["mlp_norm"])
    hid = torch.nn.functional.silu(torch.nn.functional.linear(h, T(lw["w_gate"]))) * torch.nn.functional.linear(h, T(lw["w_up"]))
    x = x + torch.nn.functional.linear(hid, T(lw["w_down"]))
    ref = (cfg.logit_scale * torch.nn.functional.linear(nrm(x, w["final_norm"]), T(w["lm_head"]))).numpy()
    assert np.allclose(F.forward(cfg, w, tok), ref, atol=1e-10)
