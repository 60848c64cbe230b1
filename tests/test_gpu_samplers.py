"""GPU parity of the LLaDA sampling strategies (Section 3.1) on the selection engine: low-confidence remasking, random
remasking (Philox draws) and their semi-autoregressive block form, bit for bit against the oracle's step machine on seeded
synthetic logits; then the strategies through the whole device loop on the tiny model, teacher-forced."""
import numpy as np
import pytest
import torch

from oracle import rowstats as RS
from oracle import samplers as SM
from paper_2506_10848_b200 import binding as sfs
from paper_2506_10848_b200 import workloads as W

from helpers import state_to_dict
from test_gpu_select import synthetic_step_logits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def pair(strategy, max_steps, block_len, seed):
    po = SM.VanillaParams(strategy=strategy, max_steps=max_steps, block_len=block_len, seed=seed)
    pg = sfs.Params.default(sampler=strategy, max_steps=max_steps, block_len=block_len, seed=seed)
    return po, pg


@pytest.mark.parametrize("strategy,B,P,L,N,bl,seed", [
    (SM.LOW_CONFIDENCE, 1, 0, 64, 0, 0, 0),            # N = L: one token per step
    (SM.LOW_CONFIDENCE, 3, 5, 40, 10, 0, 0),           # several tokens per step
    (SM.LOW_CONFIDENCE, 2, 3, 48, 24, 16, 0),          # semi-autoregressive, three blocks
    (SM.LOW_CONFIDENCE, 1, 2, 9, 18, 0, 0),            # more steps than positions: steps that unmask nothing
    (SM.LOW_CONFIDENCE, 2, 0, 50, 12, 9, 0),           # ragged last block (6 blocks: 9 x 5 + 5)
    (SM.RANDOM, 3, 4, 64, 16, 0, 0x1234567890ABCDEF),
    (SM.RANDOM, 2, 0, 60, 12, 20, 7),                  # blocks, blocks may finish early
    (SM.RANDOM, 1, 8, 300, 0, 0, 99),
])
def test_vanilla_samplers_lockstep_with_the_oracle(strategy, B, P, L, N, bl, seed):
    V = 1024
    S = P + L
    po, pg = pair(strategy, N, bl, seed)
    gen = torch.Generator().manual_seed(L * 31 + N)
    session = sfs.sfs_select_session_create(V, B, S)
    try:
        tokens = torch.full((B, S), V - 1, dtype=torch.int32, device=DEV)
        mask = torch.zeros((B, S), dtype=torch.uint8, device=DEV); mask[:, P:] = 1
        state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
        sfs.sfs_state_init(state, B, L, pg)
        sel_count = torch.zeros(B, dtype=torch.int32, device=DEV)
        sel_pos = torch.zeros((B, L), dtype=torch.int32, device=DEV)
        sel_tok = torch.zeros((B, L), dtype=torch.int32, device=DEV)
        next_rows = torch.zeros(B * L, dtype=torch.int32, device=DEV)
        next_n = torch.zeros(1, dtype=torch.int32, device=DEV)
        trace = torch.zeros((B, sfs.TRACE_INTS), dtype=torch.int32, device=DEV)
        ost = [SM.VanillaState.fresh(L, po) for _ in range(B)]
        oy = [[V - 1] * L for _ in range(B)]
        steps = 0
        while not all(s.done for s in ost):
            need = [(b, i) for b in range(B) for i in SM.vanilla_rows_needed(ost[b])]
            if steps > 0:
                n = int(next_n.item())
                assert next_rows[:n].tolist() == [b * S + P + i for (b, i) in need], steps
            n_rows = len(need)
            logits = synthetic_step_logits(max(n_rows, 1), V, gen, torch.bfloat16)
            rows = torch.tensor([b * S + P + i for (b, i) in need] or [0], dtype=torch.int32, device=DEV)
            n_dev = torch.tensor([n_rows], dtype=torch.int32, device=DEV)
            sfs.sfs_select(session, logits.to(DEV), sfs.LOGITS_BF16, V, rows, n_dev, max(n_rows, 1), tokens, mask, B, S, P, state, pg,
                           sel_count, sel_pos, sel_tok, next_rows, next_n, trace)
            torch.cuda.synchronize()
            st = RS.row_stats(W.bf16_bits(logits))
            for b in range(B):
                if ost[b].done:
                    assert int(sel_count[b]) == 0
                    continue
                idx = {i: j for j, (bb, i) in enumerate(need) if bb == b}
                rec = SM.vanilla_step(ost[b], {i: int(st["argmax"][j]) for i, j in idx.items()}, {i: int(st["sq"][j]) for i, j in idx.items()}, po, seq=b)
                for i, t in zip(rec.positions, rec.tokens):
                    oy[b][i] = t
                n = int(sel_count[b])
                assert sel_pos[b, :n].tolist() == rec.positions and sel_tok[b, :n].tolist() == rec.tokens, (steps, b)
                lo, hi = rec.block * ost[b].block_len, min(L, (rec.block + 1) * ost[b].block_len)
                assert trace[b].tolist()[:6] == [rec.block, lo, hi, rec.k_block, 0, len(rec.positions)], (steps, b)
                got = state_to_dict(state[b])
                assert got["steps_done"] == ost[b].steps_done and got["n_masked"] == sum(ost[b].masked) and got["done"] == int(ost[b].done)
                assert got["status"] == 0
            steps += 1
        assert tokens[:, P:].cpu().tolist() == oy and int(mask.sum()) == 0
        sfs.sfs_check_device_status()
    finally:
        sfs.sfs_session_destroy(session)


def test_invalid_sampler_settings_are_rejected():
    st = torch.zeros((1, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
    with pytest.raises(sfs.SfsError):
        sfs.sfs_state_init(st, 1, 64, sfs.Params.default(sampler=3))
    with pytest.raises(sfs.SfsError):                       # 4 blocks, 10 steps
        sfs.sfs_state_init(st, 1, 64, sfs.Params.default(sampler=1, block_len=16, max_steps=10))
    sfs.sfs_state_init(st, 1, 64, sfs.Params.default(sampler=1, block_len=16, max_steps=12))


@pytest.mark.parametrize("strategy,N,bl", [(SM.LOW_CONFIDENCE, 16, 0), (SM.LOW_CONFIDENCE, 32, 16), (SM.RANDOM, 16, 32)])
def test_vanilla_generation_on_the_tiny_model_is_reproduced_by_the_oracle(strategy, N, bl):
    """The device loop (forward, LM head, row statistics, selection) under a LLaDA strategy; the oracle's step machine, fed the
    GPU's logits of every step, gives the same rows, selections and tokens."""
    from test_gpu_forward import tiny_setup
    shape, model, cfg, w64 = tiny_setup(logit_scale=8.0)
    B, P, L = 2, 32, 64
    S = P + L
    po, pg = pair(strategy, N, bl, 2024)
    prompt = W.prompt_ids(B, P, 4094, seed=0)
    session = sfs.sfs_session_create(model, B, S)
    try:
        trace = torch.zeros((N, B, sfs.TRACE_INTS), dtype=torch.int32, device=DEV)
        dump = torch.zeros((B * L, shape.vocab), dtype=torch.bfloat16, device=DEV)
        rows_d = torch.zeros(B * L, dtype=torch.int32, device=DEV)
        nrows_d = torch.zeros(1, dtype=torch.int32, device=DEV)
        sfs.sfs_generate_begin(session, prompt.to(DEV), B, P, L, pg)
        ost = [SM.VanillaState.fresh(L, po) for _ in range(B)]
        oy = [[shape.mask_id] * L for _ in range(B)]
        step = 0
        while not all(s.done for s in ost):
            sfs.sfs_generate_steps(session, 1, trace, N, dump, rows_d, nrows_d)
            torch.cuda.synchronize()
            n = int(nrows_d.item())
            got_rows = rows_d[:n].tolist()
            need = [(b, i) for b in range(B) for i in SM.vanilla_rows_needed(ost[b])]
            if step > 0:
                assert got_rows == [b * S + P + i for (b, i) in need], step
            else:                                           # the first step is handed every response row; the extra ones are ignored
                assert set(b * S + P + i for (b, i) in need) <= set(got_rows)
            where = {r: j for j, r in enumerate(got_rows)}
            stats = RS.row_stats(W.bf16_bits(dump[:n].cpu()))
            for b in range(B):
                if ost[b].done:
                    continue
                idx = {i: where[b * S + P + i] for i in SM.vanilla_rows_needed(ost[b])}
                rec = SM.vanilla_step(ost[b], {i: int(stats["argmax"][j]) for i, j in idx.items()}, {i: int(stats["sq"][j]) for i, j in idx.items()}, po, seq=b)
                for i, t in zip(rec.positions, rec.tokens):
                    oy[b][i] = t
                assert trace[step, b].tolist()[3:6] == [rec.k_block, 0, len(rec.positions)], (step, b)
            step += 1
        out = torch.zeros((B, S), dtype=torch.int32, device=DEV)
        state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
        n_active, _ = sfs.sfs_generate_end(session, out, state)
        sfs.sfs_check_device_status()
        assert n_active == 0 and out[:, P:].cpu().tolist() == oy and torch.equal(out[:, :P].cpu(), prompt)
        assert step <= N
    finally:
        sfs.sfs_session_destroy(session)
        model.close()


@pytest.mark.parametrize("strategy,N,bl", [(SM.LOW_CONFIDENCE, 0, 0), (SM.LOW_CONFIDENCE, 8, 12), (SM.RANDOM, 6, 0)])
def test_vanilla_samplers_on_full_vocabulary_rows(strategy, N, bl):
    """Long bf16 rows go through the two-pass row statistics, whose second pass must know what each strategy asks of a row
    (low-confidence: the ranking, top-1 or top-k; random: nothing).  Confidences are planted close together so that the
    ranking is decided by the canonical values."""
    V, B, P, L = 126464, 2, 0, 24
    S = P + L
    po, pg = pair(strategy, N, bl, 77)
    session = sfs.sfs_select_session_create(V, B, S)
    try:
        tokens = torch.full((B, S), V - 1, dtype=torch.int32, device=DEV)
        mask = torch.ones((B, S), dtype=torch.uint8, device=DEV)
        state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV)
        sfs.sfs_state_init(state, B, L, pg)
        sel_count = torch.zeros(B, dtype=torch.int32, device=DEV)
        sel_pos = torch.zeros((B, L), dtype=torch.int32, device=DEV); sel_tok = torch.zeros((B, L), dtype=torch.int32, device=DEV)
        ost = [SM.VanillaState.fresh(L, po) for _ in range(B)]
        g = torch.Generator().manual_seed(5)
        step = 0
        while not all(s_.done for s_ in ost):
            need = [(b, i) for b in range(B) for i in SM.vanilla_rows_needed(ost[b])]
            conf = 0.3 + 2e-5 * torch.randint(0, 4, (max(len(need), 1),), generator=g).double()      # near-ties
            logits = W.logits_for_confidences(conf, V, seed=9, step=step)
            rows = torch.tensor([b * S + P + i for (b, i) in need] or [0], dtype=torch.int32, device=DEV)
            n_dev = torch.tensor([len(need)], dtype=torch.int32, device=DEV)
            sfs.sfs_select(session, logits.to(DEV), sfs.LOGITS_BF16, V, rows, n_dev, max(len(need), 1), tokens, mask, B, S, P, state, pg,
                           sel_count, sel_pos, sel_tok)
            torch.cuda.synchronize()
            st = RS.row_stats(W.bf16_bits(logits))
            for b in range(B):
                if ost[b].done:
                    continue
                idx = {i: j for j, (bb, i) in enumerate(need) if bb == b}
                rec = SM.vanilla_step(ost[b], {i: int(st["argmax"][j]) for i, j in idx.items()}, {i: int(st["sq"][j]) for i, j in idx.items()}, po, seq=b)
                n = int(sel_count[b])
                assert sel_pos[b, :n].tolist() == rec.positions and sel_tok[b, :n].tolist() == rec.tokens, (step, b)
            step += 1
        assert int(mask.sum()) == 0
        sfs.sfs_check_device_status()
    finally:
        sfs.sfs_session_destroy(session)
