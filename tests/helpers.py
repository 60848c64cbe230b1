"""Shared helpers of the GPU parity tests (marshalling between torch tensors and the oracle's Python types)."""
import numpy as np
import torch

from oracle.scheduler import SlowFastParams, SlowFastState
from paper_2506_10848_b200 import binding as sfs


def params_pair(**kw):
    """The same hyper-parameters for the oracle and for the library."""
    o = SlowFastParams(**kw)
    g = sfs.Params.default(**{k: getattr(o, k) for k in ("tau_min_conf", "tau_high_conf", "sigma2_stable", "k_max",
                                                         "w_hist", "k_slow", "k_fast", "max_steps", "min_high_count")})
    return o, g


def state_to_dict(state_row):
    v = state_row.tolist()
    return dict(zip(sfs.STATE_FIELDS, v[: len(sfs.STATE_FIELDS)]))


def oracle_state_as_ints(st: SlowFastState, w_hist: int):
    d = dict(phase=st.phase, s_cycle=st.s_cycle, hi=st.hi, step_count=st.step_count, hist_len=len(st.H),
             k_remaining=st.k, n_masked=sum(st.masked), done=int(st.done))
    for i, e in enumerate(st.H):
        d[f"hist{i}"] = e
    return d


def write_state(state_tensor, b, **fields):
    """Poke fields of sequence b's sfs_state (host-side edit of a device tensor)."""
    row = state_tensor[b].cpu()
    for k, v in fields.items():
        row[sfs.STATE_FIELDS.index(k)] = v
    state_tensor[b] = row.to(state_tensor.device)


def bf16_bits(t: torch.Tensor):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
