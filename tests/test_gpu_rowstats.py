"""GPU parity: row statistics (greedy token, canonical softmax denominator) against the oracle, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import rowstats as RS
from paper_2506_10848_b200 import binding as sfs
from paper_2506_10848_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def gpu_stats(logits, vocab, ld, dtype, n_rows_dev=None, max_rows=None):
    R = logits.shape[0] if max_rows is None else max_rows
    arg = torch.full((R,), -7, dtype=torch.int32, device=DEV)
    sq = torch.full((R,), -7, dtype=torch.int64, device=DEV)
    conf = torch.full((R,), -7.0, dtype=torch.float32, device=DEV)
    sfs.sfs_row_stats(logits, dtype, vocab, ld, n_rows_dev, R, argmax=arg, sq=sq, conf=conf)
    torch.cuda.synchronize()
    return arg.cpu().numpy(), sq.cpu().numpy().view(np.uint64), conf.cpu().numpy()


@pytest.mark.parametrize("R,V", [(1, 8), (3, 64), (5, 2048), (7, 4096), (4, 4104), (6, 16384), (3, 32768 + 64),
                                 (5, 65536 + 8), (9, 126464), (2, 131072)])
def test_bf16_fast_path_matches_oracle(R, V):
    x = W.planted_logits(R, V, seed=100 + R, device="cpu")
    if R > 2:
        x[1, :] = x[1, 0]                                   # a fully tied row
        x[2, V // 2] = x[2].max()                           # a duplicated maximum
    ref = RS.row_stats(W.bf16_bits(x))
    arg, sq, conf = gpu_stats(x.to(DEV), V, V, sfs.LOGITS_BF16)
    assert np.array_equal(arg, ref["argmax"])
    assert np.array_equal(sq, ref["sq"])
    assert np.allclose(conf, ref["conf_exact"], rtol=2e-5, atol=V * 2.0 ** -28)


@pytest.mark.parametrize("V,ld", [(1, 1), (7, 7), (1000, 1003), (4095, 4096), (126463, 126464)])
def test_generic_paths_match_oracle(V, ld):
    R = 5
    g = torch.Generator().manual_seed(V)
    full = (torch.randn((R, ld), generator=g) * 3).to(torch.float32)
    full[0, V // 2] += 9.0
    ref32 = RS.row_stats(np.ascontiguousarray(full[:, :V].numpy()))
    arg, sq, _ = gpu_stats(full.to(DEV), V, ld, sfs.LOGITS_F32)
    assert np.array_equal(arg, ref32["argmax"]) and np.array_equal(sq, ref32["sq"])
    fb = full.to(torch.bfloat16)
    refb = RS.row_stats(np.ascontiguousarray(W.bf16_bits(fb)[:, :V]))
    arg, sq, _ = gpu_stats(fb.to(DEV), V, ld, sfs.LOGITS_BF16)          # odd V / ld: the generic bf16 kernel
    assert np.array_equal(arg, refb["argmax"]) and np.array_equal(sq, refb["sq"])


def test_special_values_and_device_row_count():
    V = 4096
    x = torch.zeros((6, V), dtype=torch.float32)
    x[0] = -float("inf"); x[0, 17] = 2.0; x[0, 900] = 1.0              # -inf entries contribute nothing
    x[1, 5] = 3e38; x[1, 6] = -3e38                                      # huge spread
    x[2] = -1e4; x[2, V - 1] = -9990.0                                   # maximum in the last column
    x[3, 0] = 0.0; x[3, 1] = -0.0                                        # +0 == -0: lowest id wins
    x[4] = torch.linspace(-30, 30, V)
    x[5] = -float("inf")                                                 # nothing finite at all
    xb = x.to(torch.bfloat16)
    ref = RS.row_stats(W.bf16_bits(xb))
    n = torch.tensor([5], dtype=torch.int32, device=DEV)                 # device-side row count: row 5 is skipped
    arg, sq, _ = gpu_stats(xb.to(DEV), V, V, sfs.LOGITS_BF16, n_rows_dev=n, max_rows=6)
    assert np.array_equal(arg[:5], ref["argmax"][:5]) and np.array_equal(sq[:5], ref["sq"][:5])
    assert arg[5] == -7                                                  # untouched
    arg, sq, _ = gpu_stats(xb.to(DEV), V, V, sfs.LOGITS_BF16)
    assert np.array_equal(arg, ref["argmax"]) and np.array_equal(sq, ref["sq"])
    ref32 = RS.row_stats(np.ascontiguousarray(x.numpy()))
    arg, sq, _ = gpu_stats(x.to(DEV), V, V, sfs.LOGITS_F32)
    assert np.array_equal(arg, ref32["argmax"]) and np.array_equal(sq, ref32["sq"])


def test_epilogue_microbenchmark_shape_full_size():
    """The sampling-epilogue workload at full size: bf16 [256, 126464], planted winners."""
    x = W.planted_logits(256, 126464, seed=1, device="cpu")
    ref = RS.row_stats(W.bf16_bits(x))
    arg, sq, conf = gpu_stats(x.to(DEV), 126464, 126464, sfs.LOGITS_BF16)
    assert np.array_equal(arg, ref["argmax"])
    assert np.array_equal(sq, ref["sq"])
    assert np.allclose(conf, ref["conf_exact"], rtol=2e-5, atol=126464 * 2.0 ** -28)
    # run-to-run determinism
    arg2, sq2, _ = gpu_stats(x.to(DEV), 126464, 126464, sfs.LOGITS_BF16)
    assert np.array_equal(sq, sq2) and np.array_equal(arg, arg2)


def test_long_rows_special_values_padding_and_device_row_count():
    """Rows long enough for the streaming kernel: padded leading dimension, -inf / tied / huge entries, a maximum in
    the first and in the last column, and a device-side row count below the number of rows supplied."""
    V, ld, R = 40008, 40960, 9
    g = torch.Generator().manual_seed(7)
    x = torch.randn((R, ld), generator=g) * 4
    x[:, V:] = 1e30                                                      # padding beyond the vocabulary must be ignored
    x[0, :V] = -float("inf"); x[0, 33333] = 1.5
    x[1, :V] = 2.25                                                      # fully tied
    x[2, 0] = 50.0
    x[3, V - 1] = 50.0
    x[4, 100] = 3e38; x[4, 101] = -3e38
    x[5, :V] = -float("inf")
    x[6, 20000] = x[6, :V].max(); x[6, 39999] = x[6, 20000]              # duplicated maximum: lowest id wins
    xb = x.to(torch.bfloat16)
    ref = RS.row_stats(np.ascontiguousarray(W.bf16_bits(xb)[:, :V]))
    arg, sq, _ = gpu_stats(xb.to(DEV), V, ld, sfs.LOGITS_BF16)
    assert np.array_equal(arg, ref["argmax"]) and np.array_equal(sq, ref["sq"])
    n = torch.tensor([4], dtype=torch.int32, device=DEV)
    arg, sq, _ = gpu_stats(xb.to(DEV), V, ld, sfs.LOGITS_BF16, n_rows_dev=n, max_rows=R)
    assert np.array_equal(arg[:4], ref["argmax"][:4]) and np.array_equal(sq[:4], ref["sq"][:4])
    assert np.all(arg[4:] == -7)
    sfs.sfs_check_device_status()


def gpu_bounds(logits, vocab, ld):
    R = logits.shape[0]
    lo = torch.zeros(R, dtype=torch.int64, device=DEV); hi = torch.zeros(R, dtype=torch.int64, device=DEV)
    arg = torch.full((R,), -7, dtype=torch.int32, device=DEV)
    sfs.sfs_row_stats_bounds(logits, vocab, ld, None, R, lo, hi, arg)
    torch.cuda.synchronize()
    return lo.cpu().numpy().view(np.uint64), hi.cpu().numpy().view(np.uint64), arg.cpu().numpy()


@pytest.mark.parametrize("V,ld", [(126464, 126464), (65536, 65536 + 64), (131072, 131072)])
def test_enclosures_of_the_cheap_pass_contain_the_canonical_denominator(V, ld):
    """The enclosure [lo, hi] that the first pass of the selection's row statistics emits must contain the oracle's canonical
    S_q for every row — workload-like rows, flat rows (S_q = V 2^28), rows dominated by one logit, rows with -inf entries —
    and must be narrow (relative width 1.2e-4 plus the truncation allowance V), else the second pass would recompute
    everything.  Rows the cheap pass cannot bound (infinite or NaN sums) get an enclosure that contains everything."""
    R = 64
    x = W.planted_logits(R, V, seed=9, device="cpu").float()
    g = torch.Generator().manual_seed(V)
    x[1, :] = 0.5                                           # flat row
    x[2, :] = -3.0; x[2, 77] = 40.0                         # one logit dominates: S_q = 2^28 exactly
    x[3, ::2] = -float("inf")                               # half of the row contributes nothing
    x[4] = torch.randn(V, generator=g) * 0.3                # near-flat: S ~ V, the widest enclosures
    x[5] = torch.randn(V, generator=g) * 30.0               # very spread
    x[6, :] = -float("inf"); x[6, 5] = 1.0                  # a single finite entry
    x[7, :] = -float("inf")                                 # nothing finite: left to the canonical pass
    x[8, 11] = float("inf")                                 # an infinite maximum: left to the canonical pass
    full = torch.zeros((R, ld), dtype=torch.bfloat16)
    full[:, :V] = x.to(torch.bfloat16)
    ref = RS.row_stats(np.ascontiguousarray(W.bf16_bits(full)[:, :V]))
    lo, hi, arg = gpu_bounds(full.to(DEV), V, ld)
    sq = ref["sq"].astype(np.uint64)
    open_rows = {7, 8}
    for r in range(R):
        if r in open_rows:
            assert lo[r] <= 1 and hi[r] >= (1 << 62), r
            continue
        assert arg[r] == ref["argmax"][r], r
        assert lo[r] <= sq[r] <= hi[r], (r, int(lo[r]), int(sq[r]), int(hi[r]))
        assert float(hi[r] - lo[r]) <= 1.3e-4 * float(sq[r]) + 2.0 * V + 8, (r, int(hi[r] - lo[r]), int(sq[r]))
        assert lo[r] >= (1 << 28)
    # the approximate sum itself is far inside the enclosure: the slack is a safety factor, not a fit
    mid = (lo.astype(np.float64) + hi.astype(np.float64)) / 2
    rows = [r for r in range(R) if r not in open_rows]
    assert np.max(np.abs(mid[rows] - sq[rows].astype(np.float64)) / sq[rows].astype(np.float64)) <= 2e-5 + V / float(1 << 28)
