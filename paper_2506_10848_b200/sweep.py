"""Hyper-parameter sweep of the SlowFast schedule on the GPU: for every setting the whole selection loop (row statistics +
transition rule, `sfs_select`) runs on logits built from the seeded frontier confidence process, and the step counts are
reported — the schedule-only counterpart of the paper's sensitivity figures (accuracy needs trained weights).

    python -m paper_2506_10848_b200.sweep [--L 256] [--seeds 4] [--vocab 512]

No forward pass is involved: the confidence process stands in for the predictor, so a setting costs L small launches."""
import argparse
import json

import torch

from . import binding as sfs
from . import workloads as W

SWEEPS = {
    "k_max": [1, 2, 4, 8, 16, 32],
    "w_hist": [1, 2, 3, 4, 6, 8],
    "sigma2_stable": [0.25, 0.5, 1.0, 2.0, 4.0, 16.0],
    "tau_min_conf": [0.02, 0.05, 0.1, 0.2, 0.4],
    "tau_high_conf": [0.5, 0.7, 0.85, 0.95, 0.99],
}


def run_schedule(L, params, seed, vocab=512, reach=12.0, noise=0.06, device="cuda:0", on_step=None):
    """One sequence through the selection loop.  Returns the final state as a dict of the sfs_state fields and the number
    of steps; `on_step(step, rows, logits_bf16_cpu, trace_row)` is called after every step (inspection / parity tests)."""
    session = sfs.sfs_select_session_create(vocab, 1, L)
    try:
        tokens = torch.full((1, L), vocab - 1, dtype=torch.int32, device=device)
        mask = torch.ones((1, L), dtype=torch.uint8, device=device)
        state = torch.zeros((1, sfs.STATE_INTS), dtype=torch.int32, device=device)
        sfs.sfs_state_init(state, 1, L, params)
        next_rows = torch.arange(L, dtype=torch.int32, device=device)
        next_n = torch.tensor([L], dtype=torch.int32, device=device)
        trace = torch.zeros((1, sfs.TRACE_INTS), dtype=torch.int32, device=device)
        steps = 0
        while True:
            n = int(next_n.item())
            if n == 0:
                break
            rows = next_rows[:n].clone()
            masked = mask[0].cpu().bool().tolist()
            conf = W.frontier_confidences(masked, steps, seed, reach, noise)
            logits = W.logits_for_confidences(conf[rows.cpu().long()], vocab, seed, steps)
            sfs.sfs_select(session, logits.to(device), sfs.LOGITS_BF16, vocab, rows, None, n, tokens, mask, 1, L, 0, state, params,
                           next_rows=next_rows, next_n_rows=next_n, trace=trace)
            if on_step is not None:
                torch.cuda.synchronize()
                on_step(steps, rows.cpu().tolist(), logits, trace[0].cpu().tolist())
            steps += 1
        st = dict(zip(sfs.STATE_FIELDS, state[0].cpu().tolist()))
        return st, steps
    finally:
        sfs.sfs_session_destroy(session)


def sweep(L=256, seeds=4, vocab=512, device="cuda:0"):
    out = {"L": L, "seeds": seeds, "vocab": vocab, "sweeps": {}}
    for name, values in SWEEPS.items():
        rows = []
        for v in values:
            acc = {"steps": 0.0, "n_slow": 0.0, "n_fast": 0.0, "n_cycles": 0.0, "n_fallback": 0.0}
            for seed in range(seeds):
                st, steps = run_schedule(L, sfs.Params.default(**{name: v}), seed, vocab, device=device)
                assert st["done"] == 1 and st["n_masked"] == 0 and st["status"] == 0
                acc["steps"] += steps
                for k in ("n_slow", "n_fast", "n_cycles", "n_fallback"):
                    acc[k] += st[k]
            row = {k: x / seeds for k, x in acc.items()}
            row["value"] = v
            row["tokens_per_step"] = L / row["steps"]
            rows.append(row)
        out["sweeps"][name] = rows
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--L", type=int, default=256)
    ap.add_argument("--seeds", type=int, default=4)
    ap.add_argument("--vocab", type=int, default=512)
    ap.add_argument("--json", action="store_true")
    a = ap.parse_args()
    res = sweep(a.L, a.seeds, a.vocab)
    if a.json:
        print(json.dumps(res))
        return
    print(f"SlowFast schedule through sfs_select on the frontier confidence process: L={a.L}, {a.seeds} seeds (low-confidence remasking, N = L: {a.L} steps)")
    for name, rows in res["sweeps"].items():
        print(f"\n{name:>14} | steps  slow  fast cycles fallback tok/step")
        for m in rows:
            print(f"{m['value']:>14} | {m['steps']:5.1f} {m['n_slow']:5.1f} {m['n_fast']:5.1f} {m['n_cycles']:6.1f} {m['n_fallback']:8.1f} {m['tokens_per_step']:8.2f}")


if __name__ == "__main__":
    main()
