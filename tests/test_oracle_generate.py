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
