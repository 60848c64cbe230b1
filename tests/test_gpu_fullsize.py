"""GPU parity at the full LLaDA-8B shape, in the launch configurations the benchmark times.

* batch 1, prompt 256 + 256 masked: logits of sampled rows against the oracle's forward pass evaluated in fp32 with the
  same bf16-rounded weights (the oracle pulls one layer at a time from the device, so the host never holds the model);
* batch 8, prompt 512 + 256 masked: every sequence of the batch is independent (a sequence run alone gives the same
  logits up to the rounding order of other tile shapes), and a few steps of the device loop keep the per-sequence
  invariants (one token per step and sequence here, nothing re-masked).
"""
import numpy as np
import pytest
import torch

from oracle import forward as F
from paper_2506_10848_b200 import binding as sfs
from paper_2506_10848_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
# Tolerance at depth 32.  Weights are the same bf16 values on both sides, so the whole error is the rounding of the GEMM
# operands that are activations (normalised input, q / k / v, softmax probabilities, attention output, SwiGLU output: each
# 2^-9 relative, ~1.1e-3 rms).  It enters the fp32 residual stream once per branch and layer and grows like sqrt(depth):
# 3.5e-3 relative L2 on the 2-layer model, 1.8e-2 measured here.  The bar is 4.4e-3 * sqrt(n_layers) relative L2 and 6.5
# standard deviations of that noise for the largest of the ~760k compared logits; the 1e-2 / 3e-2 figures quoted for
# bf16 hold for the shallow model only.
def tolerances(n_layers, ref):
    rel = 4.4e-3 * np.sqrt(n_layers)
    return rel, 6.5 * rel * float(np.sqrt(np.mean(ref * ref)))


class LazyLayers:
    """w["layers"] for the oracle: layer l is converted to numpy when asked for, and dropped afterwards."""

    def __init__(self, layers):
        self.layers = layers

    def __getitem__(self, l):
        return {k: v.detach().to("cpu").to(torch.float32).numpy() for k, v in self.layers[l].items()}

    def __len__(self):
        return len(self.layers)


@pytest.fixture(scope="module")
def model8b():
    shape = W.LLADA_8B
    w = W.model_weights(shape, seed=2, device=DEV)
    model = sfs.Model(shape, w)
    yield shape, w, model
    model.close()


def test_logits_of_sampled_rows_match_the_oracle_at_the_8b_shape(model8b):
    shape, w, model = model8b
    B, P, L = 1, 256, 256
    S = P + L
    tok = torch.cat([W.prompt_ids(B, P, shape.vocab - 2, seed=2), torch.full((B, L), shape.mask_id, dtype=torch.int32)], dim=1)
    rows = [(0, P), (0, P + 1), (0, P + 100), (0, P + 177), (0, S - 1), (0, 3)]
    session = sfs.sfs_session_create(model, B, S)
    try:
        d_rows = torch.tensor([b * S + t for (b, t) in rows], dtype=torch.int32, device=DEV)
        lg = torch.zeros((len(rows), shape.vocab), dtype=torch.float32, device=DEV)
        sfs.sfs_forward(session, tok.to(DEV), B, S, d_rows, None, len(rows), lg, sfs.LOGITS_F32)
        sfs.sfs_check_device_status()
        got = lg.cpu().double().numpy()
    finally:
        sfs.sfs_session_destroy(session)
    conv = lambda t: t.detach().to("cpu").to(torch.float32).numpy()
    w_or = {"tok_emb": conv(w["tok_emb"]), "final_norm": conv(w["final_norm"]), "lm_head": conv(w["lm_head"]), "layers": LazyLayers(w["layers"])}
    cfg = F.ModelConfig(**shape.asdict())
    ref = F.forward(cfg, w_or, tok.numpy(), rows=rows, dtype=np.float32).astype(np.float64)
    max_abs = np.abs(got - ref).max()
    rel_l2 = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    print(f"8B forward, {len(rows)} sampled rows: max_abs={max_abs:.4g} rel_l2={rel_l2:.4g} (|logit| max {np.abs(ref).max():.3g})")
    tol_rel, tol_abs = tolerances(shape.n_layers, ref)
    assert rel_l2 <= tol_rel and max_abs <= tol_abs, (rel_l2, tol_rel, max_abs, tol_abs)
    # the oracle's greedy token is (nearly) the GPU's: its GPU logit is within the error bar of the GPU's maximum
    for j in range(len(rows)):
        assert got[j].max() - got[j, int(ref[j].argmax())] <= 2 * tol_abs


def test_batch_of_eight_is_eight_independent_sequences(model8b):
    shape, w, model = model8b
    B, P, L = 8, 512, 256
    S = P + L
    prompt = W.prompt_ids(B, P, shape.vocab - 2, seed=4)
    tok = torch.cat([prompt, torch.full((B, L), shape.mask_id, dtype=torch.int32)], dim=1)
    pick = [(0, P), (3, P + 7), (3, S - 1), (7, P + 128), (7, 11)]
    session = sfs.sfs_session_create(model, B, S)
    try:
        d_rows = torch.tensor([b * S + t for (b, t) in pick], dtype=torch.int32, device=DEV)
        lg8 = torch.zeros((len(pick), shape.vocab), dtype=torch.float32, device=DEV)
        sfs.sfs_forward(session, tok.to(DEV), B, S, d_rows, None, len(pick), lg8, sfs.LOGITS_F32)
        alone = {}
        for b in sorted({b for b, _ in pick}):
            rows_b = [t for (bb, t) in pick if bb == b]
            lg1 = torch.zeros((len(rows_b), shape.vocab), dtype=torch.float32, device=DEV)
            sfs.sfs_forward(session, tok[b:b + 1].to(DEV), 1, S, torch.tensor(rows_b, dtype=torch.int32, device=DEV), None, len(rows_b), lg1,
                            sfs.LOGITS_F32)
            for j, t in enumerate(rows_b):
                alone[(b, t)] = lg1[j].clone()
        sfs.sfs_check_device_status()
        # Other tile shapes sum in another order; the first bf16 rounding that flips decorrelates the two runs, so they
        # differ like two draws of the rounding noise: the same bar as against the oracle (times sqrt 2).
        for j, key in enumerate(pick):
            a, b = lg8[j].double().cpu().numpy(), alone[key].double().cpu().numpy()
            tol_rel, tol_abs = tolerances(shape.n_layers, b)
            assert np.linalg.norm(a - b) / np.linalg.norm(b) <= 1.5 * tol_rel and np.abs(a - b).max() <= 1.5 * tol_abs, key
        # a few steps of the device loop over the whole batch
        out = torch.zeros((B, S), dtype=torch.int32, device=DEV)
        state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
        trace = torch.zeros((6, B, sfs.TRACE_INTS), dtype=torch.int32, device=DEV)
        sfs.sfs_generate_begin(session, prompt.to(DEV), B, P, L, sfs.Params.default())
        sfs.sfs_generate_steps(session, 6, trace, 6)
        n_active, n_steps = sfs.sfs_generate_end(session, out, state)
        st = state.cpu().numpy()
        f = sfs.STATE_FIELDS.index
        assert n_steps == 6 and n_active == B
        assert np.all(st[:, f("steps_done")] == 6) and np.all(st[:, f("status")] == 0)
        unmasked = trace[:, :, 5].cpu().numpy().sum(axis=0)
        assert np.all(unmasked >= 6) and np.all(st[:, f("n_masked")] == L - unmasked)
        o = out.cpu()
        assert torch.equal(o[:, :P], prompt)
        assert np.all((o[:, P:] != shape.mask_id).sum(dim=1).numpy() >= unmasked - 1)   # (an argmax may be the mask id itself)
    finally:
        sfs.sfs_session_destroy(session)
