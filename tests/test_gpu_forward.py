"""GPU parity: attention, the full forward pass and the whole generation loop against the oracle."""
import numpy as np
import pytest
import torch

from oracle import forward as F
from oracle import generate as G
from oracle import rowstats as RS
from oracle.scheduler import SlowFastParams
from paper_2506_10848_b200 import binding as sfs
from paper_2506_10848_b200 import workloads as W

from bf16_reference import forward_bf16_points
from helpers import params_pair, state_to_dict

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

# Tolerance of bf16-path logits against the oracle: relative L2 <= 1e-2 and max-abs <= 3e-2, the latter for
# logits of natural scale.  Every GEMM operand is rounded to bf16 (2^-9 relative), which puts a floor of about
# 3.5e-3 relative L2 on a 2-layer model; the absolute error grows linearly with logit_scale, so the max-abs
# bar is 3e-2 * max(1, logit_scale / 4) (the tiny workload multiplies its logits by 8).
MAX_ABS, REL_L2 = 3e-2, 1e-2


def max_abs_bar(logit_scale):
    return MAX_ABS * max(1.0, logit_scale / 4.0)


@pytest.mark.parametrize("B,S,H,dh", [(1, 96, 4, 64), (2, 136, 2, 128), (1, 512, 2, 128), (3, 264, 1, 64), (2, 768, 2, 128), (1, 1536, 1, 128),
                                      (1, 1024, 2, 64), (1, 648, 1, 64), (1, 1160, 3, 128)])
def test_attention_matches_oracle(B, S, H, dh):
    # up to 12 key tiles per query tile, ragged last tiles (96, 136, 264, 648, 1160), both head dimensions
    g = torch.Generator().manual_seed(S + dh)
    d = H * dh
    q = torch.randn((B * S, d), generator=g).to(torch.bfloat16)
    k = torch.randn((B * S, d), generator=g).to(torch.bfloat16)
    v = torch.randn((B * S, d), generator=g).to(torch.bfloat16)
    qk = torch.cat([q, k], dim=1).contiguous().to(DEV)
    vt = v.t().contiguous().to(DEV)
    out = torch.zeros((B * S, d), dtype=torch.bfloat16, device=DEV)
    sfs.sfs_attention(qk, vt, out, B, S, H, dh)
    sfs.sfs_check_device_status()
    got = out.cpu().double().numpy()
    for b in range(B):
        sl = slice(b * S, (b + 1) * S)
        ref = F.attention(q[sl].double().numpy().reshape(S, H, dh), k[sl].double().numpy().reshape(S, H, dh),
                          v[sl].double().numpy().reshape(S, H, dh)).reshape(S, d)
        err = np.abs(got[sl] - ref).max()
        assert err <= 2e-2, (b, err)                         # P and the output are rounded to bf16 (2^-9 relative)


def tiny_setup(seed=0, logit_scale=None):
    shape = W.TINY
    if logit_scale is not None:
        dct = shape.asdict(); dct["logit_scale"] = logit_scale
        shape = W.Shape(**dct)
    w = W.model_weights(shape, seed=seed, gain_std=0.2)       # every norm its own gains
    wd = {k: (v.to(DEV) if k != "layers" else [{kk: vv.to(DEV) for kk, vv in lw.items()} for lw in v]) for k, v in w.items()}
    model = sfs.Model(shape, wd)
    cfg = F.ModelConfig(**shape.asdict())
    w64 = W.weights_to_numpy(w, np.float64)
    return shape, model, cfg, w64


def test_forward_logits_tiny_within_tolerance():
    shape, model, cfg, w64 = tiny_setup()
    B, P, L = 2, 32, 64
    S = P + L
    tok = torch.cat([W.prompt_ids(B, P, 4094, seed=0), torch.full((B, L), shape.mask_id, dtype=torch.int32)], dim=1)
    session = sfs.sfs_session_create(model, B, S)
    try:
        rows = [(b, P + i) for b in range(B) for i in range(0, L, 3)] + [(0, 0), (1, 5)]
        d_rows = torch.tensor([b * S + t for (b, t) in rows], dtype=torch.int32, device=DEV)
        n = len(rows)
        lg32 = torch.zeros((n, shape.vocab), dtype=torch.float32, device=DEV)
        sfs.sfs_forward(session, tok.to(DEV), B, S, d_rows, None, n, lg32, sfs.LOGITS_F32)
        lgb = torch.zeros((n, shape.vocab), dtype=torch.bfloat16, device=DEV)
        n_dev = torch.tensor([n - 3], dtype=torch.int32, device=DEV)      # device-side row count
        sfs.sfs_forward(session, tok.to(DEV), B, S, d_rows, n_dev, n, lgb, sfs.LOGITS_BF16)
        sfs.sfs_check_device_status()
        ref = F.forward(cfg, w64, tok.numpy(), rows=rows, dtype=np.float64)
        got = lg32.cpu().double().numpy()
        max_abs = np.abs(got - ref).max()
        rel_l2 = np.linalg.norm(got - ref) / np.linalg.norm(ref)
        print(f"tiny forward: max_abs={max_abs:.4g} rel_l2={rel_l2:.4g} (|logit| max {np.abs(ref).max():.3g})")
        assert rel_l2 <= REL_L2 and max_abs <= max_abs_bar(shape.logit_scale)
        assert np.abs(got - ref).max() / shape.logit_scale <= MAX_ABS     # 3e-2 on the unscaled logits
        # bf16 output = round-to-nearest-even of the fp32 output; rows beyond the device count stay untouched
        assert torch.equal(lgb[: n - 3], lg32[: n - 3].to(torch.bfloat16))
        assert float(lgb[n - 3:].abs().max()) == 0.0
    finally:
        sfs.sfs_session_destroy(session)
        model.close()


def test_forward_logits_with_peaked_attention():
    """Random-init projections give nearly uniform attention, where an error in the rotary embedding or in the score scale
    moves the logits only at second order.  Here W_q and W_k are eight times larger: the softmax is peaked, positions matter
    at first order, and so does the rounding of q and k — the bar is the distance of the rounding-only model of a bf16
    pipeline from the same oracle, plus 15 %."""
    shape = W.TINY
    w = W.model_weights(shape, seed=8, gain_std=0.2)
    for lw in w["layers"]:
        lw["wq"] = (lw["wq"].float() * 8.0).to(torch.bfloat16)
        lw["wk"] = (lw["wk"].float() * 8.0).to(torch.bfloat16)
    wd = {k: (v.to(DEV) if k != "layers" else [{kk: vv.to(DEV) for kk, vv in lw.items()} for lw in v]) for k, v in w.items()}
    model = sfs.Model(shape, wd)
    cfg = F.ModelConfig(**shape.asdict())
    w64 = W.weights_to_numpy(w, np.float64)
    B, P, L = 2, 40, 160
    S = P + L
    tok = torch.cat([W.prompt_ids(B, P, 4094, seed=3), torch.full((B, L), shape.mask_id, dtype=torch.int32)], dim=1)
    tok[:, P + 5:P + 60:3] = W.prompt_ids(B, 19, 4094, seed=4)        # a partly decoded response: rows differ by more than position
    session = sfs.sfs_session_create(model, B, S)
    try:
        rows = [(b, t) for b in range(B) for t in range(0, S, 7)]
        d_rows = torch.tensor([b * S + t for (b, t) in rows], dtype=torch.int32, device=DEV)
        lg = torch.zeros((len(rows), shape.vocab), dtype=torch.float32, device=DEV)
        sfs.sfs_forward(session, tok.to(DEV), B, S, d_rows, None, len(rows), lg, sfs.LOGITS_F32)
        sfs.sfs_check_device_status()
        ref = F.forward(cfg, w64, tok.numpy(), rows=rows, dtype=np.float64)
        got = lg.cpu().double().numpy()
        emu = np.concatenate([forward_bf16_points(cfg, w, tok[b].numpy(), [t for (bb, t) in rows if bb == b]) for b in range(B)])
        rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
        rel_model = np.linalg.norm(emu - ref) / np.linalg.norm(ref)
        print(f"peaked attention: GPU vs oracle rel_l2={rel:.4g}, rounding-only model vs oracle {rel_model:.4g}")
        assert rel <= 1.15 * rel_model and rel <= 3e-2, (rel, rel_model)
        assert np.abs(got - ref).max() <= 1.4 * np.abs(emu - ref).max()
    finally:
        sfs.sfs_session_destroy(session)
        model.close()


@pytest.mark.parametrize("dims", [dict(d_model=384, n_heads=3, head_dim=128, d_ff=1000, vocab=5000),
                                  dict(d_model=640, n_heads=10, head_dim=64, d_ff=1736, vocab=8200)])
def test_forward_logits_at_widths_that_fill_no_tile(dims):
    """Widths that are multiples of 8 and of nothing larger where the library allows it (d_ff, vocab), three or ten heads, a
    sequence of 72 or 200 tokens: ragged tiles in every projection (rows, columns and the K of the down projection), ragged
    key tiles, and a vocabulary that ends inside a column tile."""
    shape = W.Shape(n_layers=2, mask_id=dims["vocab"] - 1, rms_eps=1e-5, rope_theta=10000.0, logit_scale=8.0, **dims)
    w = W.model_weights(shape, seed=5, gain_std=0.2)
    wd = {k: (v.to(DEV) if k != "layers" else [{kk: vv.to(DEV) for kk, vv in lw.items()} for lw in v]) for k, v in w.items()}
    model = sfs.Model(shape, wd)
    cfg = F.ModelConfig(**shape.asdict())
    w64 = W.weights_to_numpy(w, np.float64)
    try:
        for (B, P, L) in ((2, 31, 41), (1, 9, 191)):
            S = P + L
            tok = torch.cat([W.prompt_ids(B, P, shape.vocab - 2, seed=1), torch.full((B, L), shape.mask_id, dtype=torch.int32)], dim=1)
            session = sfs.sfs_session_create(model, B, S)
            rows = [(b, t) for b in range(B) for t in range(0, S, 5)]
            d_rows = torch.tensor([b * S + t for (b, t) in rows], dtype=torch.int32, device=DEV)
            lg = torch.zeros((len(rows), shape.vocab), dtype=torch.float32, device=DEV)
            sfs.sfs_forward(session, tok.to(DEV), B, S, d_rows, None, len(rows), lg, sfs.LOGITS_F32)
            sfs.sfs_check_device_status()
            ref = F.forward(cfg, w64, tok.numpy(), rows=rows, dtype=np.float64)
            got = lg.cpu().double().numpy()
            rel_l2 = np.linalg.norm(got - ref) / np.linalg.norm(ref)
            # these logits are larger than the tiny model's (rms 4), so the absolute bar is the one of the rounding-only model
            # of a bf16 pipeline (fp32 arithmetic, bf16 at the stored operands) against the same oracle, plus 30 %
            emu = np.concatenate([forward_bf16_points(cfg, w, tok[b].numpy(), [t for (bb, t) in rows if bb == b]) for b in range(B)])
            rel_model, abs_model = np.linalg.norm(emu - ref) / np.linalg.norm(ref), np.abs(emu - ref).max()
            assert rel_l2 <= REL_L2 and rel_l2 <= 1.10 * rel_model, (B, S, rel_l2, rel_model)
            assert np.abs(got - ref).max() <= 1.3 * abs_model, (B, S, np.abs(got - ref).max(), abs_model)
            # and the whole loop runs to the end on this shape: every position decoded once, prompt untouched
            out = torch.zeros((B, S), dtype=torch.int32, device=DEV)
            state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
            sfs.sfs_generate(session, tok[:, :P].contiguous().to(DEV), B, P, L, sfs.Params.default(), out, state)
            sfs.sfs_check_device_status()
            o = out.cpu()
            assert torch.equal(o[:, :P], tok[:, :P]) and int((o[:, P:] == shape.mask_id).sum()) == 0
            for b in range(B):
                st = state_to_dict(state[b])
                assert st["done"] == 1 and st["n_masked"] == 0 and st["status"] == 0
            sfs.sfs_session_destroy(session)
    finally:
        model.close()


@pytest.mark.parametrize("logit_scale,B,P,L,pkw", [
    (8.0, 1, 32, 64, {}), (60.0, 3, 32, 64, {}),
    (60.0, 1, 0, 8, {}),                         # no prompt at all
    (60.0, 2, 7, 1, {}),                         # a single position to decode
    (60.0, 1, 5, 19, {"max_steps": 3}),          # the step budget runs out long before the positions do
    (8.0, 2, 3, 13, {"max_steps": 4, "k_slow": 2, "k_fast": 3}),
])
def test_generate_tiny_teacher_forced(logit_scale, B, P, L, pkw):
    """Whole loop on the device; then the oracle's selection is fed the GPU's own logits step by step and
    must reproduce the GPU's trace and tokens exactly.  logit_scale 60 makes confidences cross both
    thresholds, so parallel unmasking and span logic are exercised with a real model in the loop.  The
    degenerate shapes: empty prompt, one position, a budget of steps far below the number of positions."""
    shape, model, cfg, w64 = tiny_setup(logit_scale=logit_scale)
    S = P + L
    po, pg = params_pair(**pkw)
    prompt = W.prompt_ids(B, P, 4094, seed=0)
    session = sfs.sfs_session_create(model, B, S)
    try:
        out = torch.zeros((B, S), dtype=torch.int32, device=DEV)
        state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
        trace = torch.zeros((L, B, sfs.TRACE_INTS), dtype=torch.int32, device=DEV)
        sfs.sfs_generate(session, prompt.to(DEV), B, P, L, pg, out, state, trace, L)
        torch.cuda.synchronize()
        steps_gpu = [state_to_dict(state[b])["steps_done"] for b in range(B)]

        # replay step by step, dumping the logits of every step
        sfs.sfs_generate_begin(session, prompt.to(DEV), B, P, L, pg)
        dump = torch.zeros((B * L, shape.vocab), dtype=torch.bfloat16, device=DEV)
        rows_d = torch.zeros(B * L, dtype=torch.int32, device=DEV)
        nrows_d = torch.zeros(1, dtype=torch.int32, device=DEV)
        from oracle.scheduler import SlowFastState, rows_needed, slowfast_step
        ost = [SlowFastState.fresh(L, po) for _ in range(B)]
        oy = [[None] * L for _ in range(B)]
        step = 0
        first_logits = None
        while not all(s.done for s in ost):
            sfs.sfs_generate_steps(session, 1, None, 0, dump, rows_d, nrows_d)
            torch.cuda.synchronize()
            n = int(nrows_d.item())
            need = [(b, i) for b in range(B) for i in rows_needed(ost[b])]
            assert rows_d[:n].tolist() == [b * S + P + i for (b, i) in need]
            lg = dump[:n].cpu()
            if step == 0:
                first_logits = lg.float().numpy().copy()
            st = RS.row_stats(W.bf16_bits(lg))
            for b in range(B):
                if ost[b].done:
                    continue
                idx = {i: j for j, (bb, i) in enumerate(need) if bb == b}
                rec = slowfast_step(ost[b], {i: int(st["argmax"][j]) for i, j in idx.items()},
                                    {i: int(st["sq"][j]) for i, j in idx.items()}, po)
                for i, t in zip(rec.positions, rec.tokens):
                    oy[b][i] = t
                tr = trace[step, b].tolist()
                assert tr[:6] == [rec.phase, rec.s, rec.hi, rec.e_cand, rec.stable, len(rec.positions)], (step, b, tr, rec)
            step += 1
        n_active, n_steps = sfs.sfs_generate_end(session)
        assert n_active == 0
        tk = out.cpu()
        for b in range(B):
            assert tk[b, :P].tolist() == prompt[b].tolist()
            assert tk[b, P:].tolist() == oy[b]
            assert steps_gpu[b] == ost[b].steps_done
        print("steps per sequence:", steps_gpu)
        if logit_scale > 30 and L >= 32 and not pkw:
            assert min(steps_gpu) < L                      # thresholds fired: fewer steps than tokens

        # first-step logits against the oracle's own forward (the response is fully masked at step 0)
        tok0 = torch.cat([prompt, torch.full((B, L), shape.mask_id, dtype=torch.int32)], dim=1).numpy()
        ref = F.forward(cfg, w64, tok0, rows=[(b, P + i) for b in range(B) for i in range(L)], dtype=np.float64)
        err = np.abs(first_logits - ref)
        tol = max_abs_bar(logit_scale) + 2.0 ** -8 * np.abs(ref)   # + the bf16 rounding of the stored logit
        assert np.all(err <= tol), float(err.max())
    finally:
        sfs.sfs_session_destroy(session)
        model.close()
