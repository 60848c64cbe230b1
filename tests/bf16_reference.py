"""A test-side model of WHERE the bf16 pipeline rounds (not an oracle, and not part of the library): the mask
predictor's forward pass in fp32 with a round-to-nearest-even to bf16 at the points where a bf16 pipeline stores a
GEMM operand — the normalised input of each branch, q / k after the projection and again after the rotation, v, the
softmax probabilities, the attention output, the SwiGLU output and the final normalised rows.  The residual stream,
every accumulation and the logits stay fp32.

The parity tests use it to separate two things the fp32 oracle cannot tell apart at depth 32: the rounding noise that
any bf16 pipeline has (the oracle-to-this distance) and an arithmetic error of the kernels (the GPU-to-this distance,
which must be far smaller)."""
import numpy as np
import torch


def _r(t):
    return t.to(torch.bfloat16).to(torch.float32)


def _rms(x, g, eps):
    inv = torch.rsqrt((x * x).mean(dim=-1, keepdim=True) + eps)
    return x * inv * g


def _rope(x, pos, theta):
    """x [S, H, dh] fp32: pairs (j, j + dh/2) rotate by pos * theta^(-2j/dh); the table is evaluated in double."""
    dh = x.shape[-1]
    half = dh // 2
    j = torch.arange(half, dtype=torch.float64)
    ang = pos.to(torch.float64)[:, None] * theta ** (-2.0 * j / dh)[None, :]
    cos, sin = torch.cos(ang).float()[:, None, :], torch.sin(ang).float()[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1)


def forward_bf16_points(cfg, w, tokens, rows):
    """cfg: any object with the shape fields; w: dict of torch tensors (bf16 or fp32; w["layers"][l] may be produced
    lazily); tokens: int [S] of ONE sequence; rows: positions whose logits are wanted.  Returns fp32 numpy [len(rows), V]."""
    f32 = lambda t: t.detach().to("cpu").to(torch.float32)
    tok = torch.as_tensor(np.asarray(tokens), dtype=torch.long)
    S = tok.shape[0]
    H, dh = cfg.n_heads, cfg.head_dim
    pos = torch.arange(S)
    x = f32(w["tok_emb"])[tok]
    for l in range(cfg.n_layers):
        lw = w["layers"][l]
        h = _r(_rms(x, f32(lw["attn_norm"]), cfg.rms_eps))
        q = _r(_rope(_r(h @ f32(lw["wq"]).T).reshape(S, H, dh), pos, cfg.rope_theta))
        k = _r(_rope(_r(h @ f32(lw["wk"]).T).reshape(S, H, dh), pos, cfg.rope_theta))
        v = _r(h @ f32(lw["wv"]).T).reshape(S, H, dh)
        s = torch.einsum("qhd,khd->hqk", q, k) / float(np.sqrt(dh))
        p = torch.exp(s - s.max(dim=-1, keepdim=True).values)
        a = torch.einsum("hqk,khd->qhd", _r(p), v) / p.sum(dim=-1).transpose(0, 1)[:, :, None]   # rounded numerator, exact denominator
        a = _r(a.reshape(S, H * dh))
        x = x + a @ f32(lw["wo"]).T
        h = _r(_rms(x, f32(lw["mlp_norm"]), cfg.rms_eps))
        g, u = h @ f32(lw["w_gate"]).T, h @ f32(lw["w_up"]).T
        hid = _r(g / (1.0 + torch.exp(-g)) * u)
        x = x + hid @ f32(lw["w_down"]).T
    hf = _r(_rms(x[torch.as_tensor(list(rows), dtype=torch.long)], f32(w["final_norm"]), cfg.rms_eps))
    return ((hf @ f32(w["lm_head"]).T) * float(cfg.logit_scale)).numpy()
