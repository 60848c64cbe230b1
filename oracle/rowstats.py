"""ORACLE (test infrastructure): Python face of `rowstats.c`.

`row_stats(logits)` returns, per row, the greedy token (Section 3.1, Eq. 3), the canonical fixed-point
softmax denominator S_q (Q28; the value every decision is taken on) and the plain double-precision
confidence c_i = softmax(x)[argmax] (Section 3.1, confidence equation).
"""
import ctypes
import os

import numpy as np

from . import build as _build

QBITS = 28
_lib = None


def _load():
    global _lib
    if _lib is None:
        path = _build.build()
        lib = ctypes.CDLL(path)
        for name in ("sfs_oracle_rowstats_f32", "sfs_oracle_rowstats_bf16"):
            getattr(lib, name).restype = None
        lib.sfs_oracle_qbits.restype = ctypes.c_int
        assert lib.sfs_oracle_qbits() == QBITS
        _lib = lib
    return _lib


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def row_stats(logits):
    """logits: [R, V] numpy array, float32, or uint16 holding bf16 bit patterns.

    Returns dict(argmax int32[R], vmax float32[R], sq uint64[R], conf_exact float64[R]).
    """
    lib = _load()
    x = np.ascontiguousarray(logits)
    assert x.ndim == 2
    R, V = x.shape
    amax = np.zeros(R, np.int32)
    vmax = np.zeros(R, np.float32)
    sq = np.zeros(R, np.uint64)
    conf = np.zeros(R, np.float64)
    if x.dtype == np.float32:
        fn = lib.sfs_oracle_rowstats_f32
    elif x.dtype == np.uint16:
        fn = lib.sfs_oracle_rowstats_bf16
    else:
        raise TypeError("logits must be float32 or uint16 (bf16 bits), got %s" % x.dtype)
    fn(_ptr(x), ctypes.c_long(R), ctypes.c_long(V), ctypes.c_long(V), _ptr(amax), _ptr(vmax), _ptr(sq), _ptr(conf))
    return dict(argmax=amax, vmax=vmax, sq=sq, conf_exact=conf)


def conf_from_sq(sq):
    """Informational confidence 2^Q / S_q (decisions never use this floating-point value)."""
    return float(1 << QBITS) / np.asarray(sq, dtype=np.float64)


def exceeds(sq, tau):
    """The canonical test `c_i > tau`:  double(S_q) * double(float32 tau) < 2^Q  (one IEEE multiply)."""
    tau64 = np.float64(np.float32(tau))
    return np.asarray(sq, dtype=np.float64) * tau64 < np.float64(1 << QBITS)
