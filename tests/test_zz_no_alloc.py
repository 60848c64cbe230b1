"""sfs_select_static - the selection step for callers that may not allocate device memory (graph capture or
replay, allocation-free serving loops, GPUs whose memory another runtime owns).  It must give exactly what
sfs_select gives, call after call, although all calls share one built-in scratch array.  This file is
collected last on purpose: if it fails, every other test has already run."""
import pytest
import torch

from paper_2506_10848_b200 import binding as sfs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def fresh(B, P, L, V, pg):
    S = P + L
    d = dict(tokens=torch.full((B, S), V - 1, dtype=torch.int32, device=DEV),
             mask=torch.zeros((B, S), dtype=torch.uint8, device=DEV),
             state=torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=DEV),
             sel_count=torch.zeros(B, dtype=torch.int32, device=DEV),
             sel_pos=torch.zeros((B, L), dtype=torch.int32, device=DEV),
             sel_tok=torch.zeros((B, L), dtype=torch.int32, device=DEV),
             next_rows=torch.zeros(B * L, dtype=torch.int32, device=DEV),
             next_n=torch.zeros(1, dtype=torch.int32, device=DEV),
             trace=torch.zeros((B, sfs.TRACE_INTS), dtype=torch.int32, device=DEV))
    d["mask"][:, P:] = 1
    sfs.sfs_state_init(d["state"], B, L, pg)
    return d


def test_static_entry_matches_session_entry_on_consecutive_calls():
    B, P, L, V = 3, 4, 40, 1024
    S = P + L
    pg = sfs.Params.default(k_slow=2)
    gen = torch.Generator().manual_seed(123)
    session = sfs.sfs_select_session_create(V, B, S)
    try:
        a, b = fresh(B, P, L, V, pg), fresh(B, P, L, V, pg)
        n_rows, rows = B * L, torch.tensor([q * S + P + i for q in range(B) for i in range(L)], dtype=torch.int32, device=DEV)
        for call in range(4):                               # several calls in a row on the shared array
            x = torch.randn((n_rows, V), generator=gen) * 1.5
            x[torch.arange(n_rows), torch.randint(0, V, (n_rows,), generator=gen)] += torch.rand(n_rows, generator=gen) * 14
            logits = x.to(torch.bfloat16).to(DEV)
            n_dev = torch.tensor([n_rows], dtype=torch.int32, device=DEV)
            sfs.sfs_select(session, logits, sfs.LOGITS_BF16, V, rows, n_dev, n_rows, a["tokens"], a["mask"], B, S, P, a["state"], pg,
                           a["sel_count"], a["sel_pos"], a["sel_tok"], a["next_rows"], a["next_n"], a["trace"])
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            sfs.sfs_select_static(V, logits, sfs.LOGITS_BF16, V, rows, n_dev, n_rows, b["tokens"], b["mask"], B, S, P, b["state"], pg,
                                  b["sel_count"], b["sel_pos"], b["sel_tok"], b["next_rows"], b["next_n"], b["trace"])
            torch.cuda.synchronize()
            if call > 0:                                    # (the very first call may load the kernels' code)
                assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the amount of free device memory"
            for key in ("tokens", "mask", "state", "sel_count", "next_n", "trace"):
                assert torch.equal(a[key], b[key]), (call, key)
            for q in range(B):
                n = int(a["sel_count"][q])
                assert n >= 1
                assert torch.equal(a["sel_pos"][q, :n], b["sel_pos"][q, :n]) and torch.equal(a["sel_tok"][q, :n], b["sel_tok"][q, :n])
            n = int(a["next_n"])
            assert torch.equal(a["next_rows"][:n], b["next_rows"][:n])
            rows, n_rows = a["next_rows"][:n].clone(), n      # the next call reads the rows this one asked for
            if n_rows == 0:
                break
    finally:
        sfs.sfs_session_destroy(session)


def test_static_entry_rejects_sizes_beyond_its_array():
    pg = sfs.Params.default()
    t = torch.zeros(8, dtype=torch.int32, device=DEV)
    with pytest.raises(sfs.SfsError) as e:
        sfs.sfs_select_static(64, t, sfs.LOGITS_BF16, 64, t, None, 1, t, t, 1, sfs.STATIC_MAX_POSITIONS + 8, 0, t, pg)
    assert e.value.status == sfs.ERR_UNSUPPORTED and "built-in scratch" in str(e.value)
    with pytest.raises(sfs.SfsError) as e:
        sfs.sfs_select_static(64, t, sfs.LOGITS_BF16, 64, t, None, 1, t, t, sfs.STATIC_MAX_BATCH + 1, 8, 0, t, pg)
    assert e.value.status == sfs.ERR_UNSUPPORTED


def test_static_entry_reports_a_bad_row_index_in_the_sequence_state():
    """No session, hence no process-wide status word to read: a row index outside the token grid is skipped (nothing is
    written outside the built-in array) and shows up as state.status of the sequences of that call."""
    B, P, L, V = 1, 0, 16, 256
    pg = sfs.Params.default()
    d = fresh(B, P, L, V, pg)
    rows = torch.arange(L, dtype=torch.int32, device=DEV)
    rows[2] = sfs.STATIC_MAX_POSITIONS * 64                # far outside
    logits = (torch.randn((L, V), generator=torch.Generator().manual_seed(1)) * 2).to(torch.bfloat16).to(DEV)
    sfs.sfs_select_static(V, logits, sfs.LOGITS_BF16, V, rows, None, L, d["tokens"], d["mask"], B, L, P, d["state"], pg)
    torch.cuda.synchronize()
    status = int(d["state"][0, sfs.STATE_FIELDS.index("status")])
    assert status in (sfs.ERR_MISSING_ROW, sfs.ERR_INVALID_ARG) and int(d["mask"].sum()) == L
