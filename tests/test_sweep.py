"""The hyper-parameter sweep harness: the oracle-side sweep (CPU) shows the trends Section 4.3 describes and the effect of the
alternative readings; the GPU-side sweep is the same schedule through sfs_select and must agree with the oracle step for step
when both read the same logits."""
import pytest

from oracle import sweep as OS
from oracle.scheduler import SlowFastParams


def test_oracle_sweep_trends_and_alternative_readings():
    L, seeds = 96, 3
    hi = [OS.mean_over_seeds(L, SlowFastParams(tau_high_conf=t), seeds, 12.0, 0.06)["steps"] for t in (0.5, 0.85, 0.99)]
    assert hi[0] < hi[1] < hi[2] <= L                       # a higher tau_high_conf decodes more cautiously
    w = [OS.mean_over_seeds(L, SlowFastParams(w_hist=v), seeds, 12.0, 0.06)["slow"] for v in (1, 2, 4)]
    assert w[0] < w[1] < w[2]                               # a longer window spends more exploratory steps
    base = OS.mean_over_seeds(L, SlowFastParams(), seeds, 12.0, 0.06)
    assert base["leftover"] == 0 and base["tokens"] == L and base["steps"] < L
    one = OS.mean_over_seeds(L, SlowFastParams(fast_single_step=True), seeds, 12.0, 0.06)
    assert one["leftover"] > 0                              # Algorithm 1 as printed leaves masks behind s_cycle
    last = OS.mean_over_seeds(L, SlowFastParams(e_cycle_rule="last_candidate"), seeds, 12.0, 0.06)
    keep = OS.mean_over_seeds(L, SlowFastParams(reset_history=False), seeds, 12.0, 0.06)
    assert last["leftover"] == 0 and keep["leftover"] == 0 and last["tokens"] == L and keep["tokens"] == L
    res = OS.sweep(L=32, seeds=1)
    assert set(res["sweeps"]) == {"k_max", "w_hist", "sigma2_stable", "tau_min_conf", "tau_high_conf"} and len(res["readings"]) == 4


@pytest.mark.gpu
@pytest.mark.parametrize("kw", [{}, {"tau_high_conf": 0.6, "k_max": 3}, {"w_hist": 4, "sigma2_stable": 4.0, "tau_min_conf": 0.3}])
def test_gpu_sweep_schedule_is_the_oracle_schedule_on_the_same_logits(kw):
    from oracle import rowstats as RS
    from oracle.scheduler import SlowFastState, rows_needed, slowfast_step
    from paper_2506_10848_b200 import binding as sfs
    from paper_2506_10848_b200 import sweep as GS
    from paper_2506_10848_b200 import workloads as W
    L = 160
    po = SlowFastParams(**kw)
    pg = sfs.Params.default(**kw)
    ost = SlowFastState.fresh(L, po)

    def on_step(step, rows, logits, trace_row):
        assert rows == rows_needed(ost), step
        st = RS.row_stats(W.bf16_bits(logits))
        rec = slowfast_step(ost, {i: int(st["argmax"][j]) for j, i in enumerate(rows)}, {i: int(st["sq"][j]) for j, i in enumerate(rows)}, po)
        assert trace_row[:6] == [rec.phase, rec.s, rec.hi, rec.e_cand, rec.stable, len(rec.positions)], step

    st, steps = GS.run_schedule(L, pg, seed=5, on_step=on_step)
    assert ost.done and steps == ost.steps_done == st["steps_done"] and st["n_masked"] == 0 and steps < L
