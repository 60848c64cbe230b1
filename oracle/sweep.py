"""ORACLE-side tool (test infrastructure, CPU only): sensitivity of the SlowFast schedule to its hyper-parameters on a
synthetic confidence process — the in-box counterpart of the paper's sensitivity figures (stability check: K_max,
sigma^2_stable, W_hist; confidence thresholds: tau_min_conf, tau_high_conf), which were measured on benchmark accuracy
and TPS that need trained weights.  What can be measured without them is the schedule itself: denoising steps per
sequence (the paper's speed-up is a step-count ratio, every step costing one forward pass), the slow / fast split, the
number of cycles and fallbacks — against low-confidence remasking with N = L as the 1.00x row.

It also runs the alternative readings of the passages where the paper is at odds with itself (e_cycle from the last
candidate instead of the window mean; H_W kept across cycles; one accelerated step per cycle as Algorithm 1 prints it) so
that their effect on the schedule is on record.

    python -m oracle.sweep [--L 256] [--seeds 8] [--reach 12] [--noise 0.06]
"""
import argparse
import json
from dataclasses import replace
from typing import Dict, List

from . import samplers as SM
from .scheduler import FAST, QBITS, SLOW, SlowFastParams, slowfast_loop


def sq_from_confidence(c: float) -> int:
    """The canonical denominator a row with max-probability c would have (2^28 / c, at least 2^28)."""
    return max(1 << QBITS, int(round((1 << QBITS) / c)))


def frontier_predict(L: int, seed: int, reach: float, noise: float):
    """predict callback over the seeded frontier confidence process (the generator lives with the other workload recipes)."""
    from paper_2506_10848_b200 import workloads as W
    step = [0]

    def predict(masked, rows):
        c = W.frontier_confidences(masked, step[0], seed, reach, noise)
        step[0] += 1
        return {i: 1000 + i for i in rows}, {i: sq_from_confidence(float(c[i])) for i in rows}
    return predict


def run_once(L: int, p: SlowFastParams, seed: int, reach: float, noise: float) -> Dict:
    y, trace = slowfast_loop(L, frontier_predict(L, seed, reach, noise), p)
    slow = sum(1 for r in trace if r.phase == SLOW)
    return dict(steps=len(trace), slow=slow, fast=len(trace) - slow, cycles=1 + sum(1 for a, b in zip(trace, trace[1:]) if b.s != a.s),
                fallback=sum(1 for r in trace if r.phase == FAST and len(r.positions) == p.k_fast and r.e_cand == -1 and len(r.positions) < (r.hi - r.s)),
                leftover=sum(1 for t in y if t is None), tokens=sum(len(r.positions) for r in trace))


def mean_over_seeds(L: int, p: SlowFastParams, seeds: int, reach: float, noise: float) -> Dict:
    runs = [run_once(L, p, s, reach, noise) for s in range(seeds)]
    out = {k: sum(r[k] for r in runs) / len(runs) for k in runs[0]}
    out["tokens_per_step"] = out["tokens"] / max(out["steps"], 1e-9)
    return out


SWEEPS = {
    "k_max": [1, 2, 4, 8, 16, 32],
    "w_hist": [1, 2, 3, 4, 6, 8],
    "sigma2_stable": [0.25, 0.5, 1.0, 2.0, 4.0, 16.0],
    "tau_min_conf": [0.02, 0.05, 0.1, 0.2, 0.4],
    "tau_high_conf": [0.5, 0.7, 0.85, 0.95, 0.99],
}
READINGS = {
    "default (floor mean, history reset, multi-step fast)": {},
    "R2: e_cycle = last candidate": {"e_cycle_rule": "last_candidate"},
    "R5: history kept across cycles": {"reset_history": False},
    "R6: one accelerated step per cycle": {"fast_single_step": True},
}


def sweep(L: int = 256, seeds: int = 8, reach: float = 12.0, noise: float = 0.06) -> Dict:
    base = SlowFastParams()
    res = {"L": L, "seeds": seeds, "process": {"reach": reach, "noise": noise}, "sweeps": {}, "readings": {}}
    lc_steps = L                                                       # low-confidence remasking with N = L: one token per step
    pr = frontier_predict(L, 0, reach, noise)
    assert len(SM.low_confidence_remasking(L, L, pr)[1]) == lc_steps
    res["baseline_low_confidence_steps"] = lc_steps
    for name, values in SWEEPS.items():
        rows = []
        for v in values:
            m = mean_over_seeds(L, replace(base, **{name: v}), seeds, reach, noise)
            m["value"] = v
            m["step_ratio_vs_low_confidence"] = lc_steps / m["steps"]
            rows.append(m)
        res["sweeps"][name] = rows
    for name, kw in READINGS.items():
        m = mean_over_seeds(L, replace(base, **kw), seeds, reach, noise)
        m["step_ratio_vs_low_confidence"] = lc_steps / m["steps"]
        res["readings"][name] = m
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--L", type=int, default=256)
    ap.add_argument("--seeds", type=int, default=8)
    ap.add_argument("--reach", type=float, default=12.0)
    ap.add_argument("--noise", type=float, default=0.06)
    ap.add_argument("--json", action="store_true")
    a = ap.parse_args()
    res = sweep(a.L, a.seeds, a.reach, a.noise)
    if a.json:
        print(json.dumps(res))
        return
    print(f"SlowFast schedule on the frontier confidence process: L={a.L}, {a.seeds} seeds, reach={a.reach}, noise={a.noise}")
    print(f"low-confidence remasking, N = L: {res['baseline_low_confidence_steps']} steps (1.00x)")
    for name, rows in res["sweeps"].items():
        print(f"\n{name:>14} | steps  slow  fast cycles tok/step  x fewer steps")
        for m in rows:
            print(f"{m['value']:>14} | {m['steps']:5.1f} {m['slow']:5.1f} {m['fast']:5.1f} {m['cycles']:6.1f} {m['tokens_per_step']:8.2f} {m['step_ratio_vs_low_confidence']:8.2f}")
    print("\nreadings")
    for name, m in res["readings"].items():
        print(f"{name:>55} | steps {m['steps']:6.1f}  tok/step {m['tokens_per_step']:5.2f}  masks left {m['leftover']:5.1f}  x fewer steps {m['step_ratio_vs_low_confidence']:5.2f}")


if __name__ == "__main__":
    main()
