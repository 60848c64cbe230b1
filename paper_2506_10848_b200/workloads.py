"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

Holds no arithmetic of the method: only random draws with the shapes and value distributions of the
workloads (model shapes, prompt ids, planted-winner logits).  Each tensor has its own generator seeded
from (seed, name), so any subset of a model can be produced without producing the rest.
"""
import zlib
from dataclasses import dataclass, asdict
from typing import Dict, Optional

import torch


@dataclass(frozen=True)
class Shape:
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    mask_id: int
    rms_eps: float
    rope_theta: float
    logit_scale: float

    def asdict(self):
        return asdict(self)


TINY = Shape(n_layers=2, d_model=256, n_heads=4, head_dim=64, d_ff=688, vocab=4096, mask_id=4095,
             rms_eps=1e-5, rope_theta=10000.0, logit_scale=8.0)
LLADA_8B = Shape(n_layers=32, d_model=4096, n_heads=32, head_dim=128, d_ff=12288, vocab=126464,
                 mask_id=126463, rms_eps=1e-5, rope_theta=500000.0, logit_scale=1.0)


def with_layers(shape: Shape, n_layers: int) -> Shape:
    d = shape.asdict()
    d["n_layers"] = n_layers
    return Shape(**d)


def _gen(seed: int, name: str, device: str) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + zlib.crc32(name.encode())) & 0x7FFFFFFFFFFF)
    return g


def normal_bf16(shape, std: float, seed: int, name: str, device: str = "cpu") -> torch.Tensor:
    """N(0, std^2) drawn in fp32 and rounded to bf16 (both implementations use the rounded values)."""
    g = _gen(seed, name, device)
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    step = 1 << 26
    for lo in range(0, flat.numel(), step):           # chunked: the fp32 temporary stays small
        n = min(step, flat.numel() - lo)
        flat[lo:lo + n] = (torch.randn(n, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)
    return out


def model_weights(shape: Shape, seed: int, device: str = "cpu", std: float = 0.02, gain_std: float = 0.0) -> Dict:
    """Random-init weights: matrices N(0, std^2) as bf16; RMSNorm gains 1, or 1 + N(0, gain_std^2) (each norm its own draw:
    what the parity tests use, so that a gain that is dropped or taken from the wrong norm shows)."""
    d, ff, V = shape.d_model, shape.d_ff, shape.vocab
    count = [0]

    def ones():
        count[0] += 1
        g = torch.ones(d, dtype=torch.float32, device=device)
        if gain_std > 0.0:
            g = g + normal_bf16((d,), gain_std, seed, f"gain{count[0]}", device).to(torch.float32)
        return g.to(torch.bfloat16)

    w = {
        "tok_emb": normal_bf16((V, d), std, seed, "tok_emb", device),
        "final_norm": ones(),
        "lm_head": normal_bf16((V, d), std, seed, "lm_head", device),
        "layers": [],
    }
    for l in range(shape.n_layers):
        w["layers"].append({
            "attn_norm": ones(),
            "wq": normal_bf16((d, d), std, seed, f"l{l}.wq", device),
            "wk": normal_bf16((d, d), std, seed, f"l{l}.wk", device),
            "wv": normal_bf16((d, d), std, seed, f"l{l}.wv", device),
            "wo": normal_bf16((d, d), std, seed, f"l{l}.wo", device),
            "mlp_norm": ones(),
            "w_gate": normal_bf16((ff, d), std, seed, f"l{l}.w_gate", device),
            "w_up": normal_bf16((ff, d), std, seed, f"l{l}.w_up", device),
            "w_down": normal_bf16((d, ff), std, seed, f"l{l}.w_down", device),
        })
    return w


def weights_to_numpy(w: Dict, dtype) -> Dict:
    """bf16 torch weights -> numpy arrays of `dtype` (values unchanged: bf16 widens exactly)."""
    conv = lambda t: t.detach().to("cpu").to(torch.float32).numpy().astype(dtype)
    out = {k: conv(v) for k, v in w.items() if k != "layers"}
    out["layers"] = [{k: conv(v) for k, v in lw.items()} for lw in w["layers"]]
    return out


def prompt_ids(batch: int, length: int, vocab_hi: int, seed: int, device: str = "cpu") -> torch.Tensor:
    """Uniform random ids in [0, vocab_hi), int32 [batch, length]."""
    g = _gen(seed, "prompt", "cpu")
    return torch.randint(0, vocab_hi, (batch, length), generator=g, dtype=torch.int32).to(device)


def planted_logits(rows: int, vocab: int, seed: int, noise_std: float = 4.0, margin_hi: float = 12.0,
                   device: str = "cpu") -> torch.Tensor:
    """Epilogue microbenchmark logits: N(0, noise_std^2) noise, and in every row one planted winner equal
    to the row's noise maximum plus a margin drawn from U(0, margin_hi).  bf16 [rows, vocab]."""
    g = _gen(seed, "planted_logits", device)
    x = torch.randn((rows, vocab), generator=g, device=device, dtype=torch.float32) * noise_std
    col = torch.randint(0, vocab, (rows,), generator=g, device=device)
    margin = torch.rand((rows,), generator=g, device=device, dtype=torch.float32) * margin_hi
    x[torch.arange(rows, device=device), col] = x.max(dim=1).values + margin
    return x.to(torch.bfloat16)


def history_ids(current: torch.Tensor, window: int, vocab: int, seed: int, agree: float = 0.7) -> torch.Tensor:
    """Previous `window` steps' predicted ids [window, R]: each entry equals `current` with probability
    `agree`, otherwise a uniform random id."""
    g = _gen(seed, "history_ids", "cpu")
    R = current.numel()
    keep = torch.rand((window, R), generator=g) < agree
    rnd = torch.randint(0, vocab, (window, R), generator=g, dtype=torch.int32)
    return torch.where(keep, current.to("cpu").to(torch.int32)[None, :], rnd)


def span(L: int, seed: int):
    """A span [lo, hi) with 0 <= lo < hi <= L drawn uniformly."""
    g = _gen(seed, "span", "cpu")
    a, b = sorted(torch.randint(0, L + 1, (2,), generator=g).tolist())
    if a == b:
        a, b = (a - 1, b) if a > 0 else (a, b + 1)
    return a, b


def bf16_bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 array of its bit patterns (what the oracle's bf16 entry takes)."""
    return t.detach().to("cpu").contiguous().view(torch.int16).numpy().view("uint16")


def frontier_confidences(masked, step: int, seed: int, reach: float = 12.0, noise: float = 0.06, seq: int = 0) -> torch.Tensor:
    """A synthetic confidence process with the shape the paper describes for trained models: positions just behind the
    decoded frontier are predicted with high confidence, confidence decays with the distance from it, and it jitters
    from step to step.  masked: sequence of bools; returns float64 [L] in (0.001, 0.999) (1.0 at decoded positions)."""
    L = len(masked)
    g = _gen(seed, f"frontier.{seq}.{step}", "cpu")
    jitter = (torch.rand(L, generator=g, dtype=torch.float64) * 2 - 1) * noise
    c = torch.ones(L, dtype=torch.float64)
    open_ = [i for i in range(L) if masked[i]]
    if open_:
        front = open_[0]
        for rank, i in enumerate(open_):
            d = 0.5 * (i - front) + 0.5 * rank             # distance from the frontier, decoded gaps count half
            c[i] = min(0.999, max(0.001, 0.97 * float(torch.exp(torch.tensor(-d / reach, dtype=torch.float64))) + float(jitter[i])))
    return c


def logits_for_confidences(conf: torch.Tensor, vocab: int, seed: int, step: int = 0) -> torch.Tensor:
    """bf16 logits [len(conf), vocab] whose softmax maximum is (up to bf16 rounding of the one non-zero logit) conf[i]:
    all entries 0 except one winner per row at log(c (V-1) / (1-c)), at a seeded column."""
    n = conf.numel()
    g = _gen(seed, f"conf_logits.{step}", "cpu")
    col = torch.randint(0, vocab, (n,), generator=g)
    x = torch.zeros((n, vocab), dtype=torch.float32)
    c = conf.to(torch.float64).clamp(1.0 / vocab + 1e-6, 1 - 1e-9)
    x[torch.arange(n), col] = torch.log(c * (vocab - 1) / (1 - c)).to(torch.float32)
    return x.to(torch.bfloat16)
