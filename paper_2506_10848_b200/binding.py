"""ctypes binding of libsfs.so: same names as the C ABI (include/sfs.h), argument marshalling only.

torch tensors are accepted wherever the ABI takes a device pointer (their data_ptr() is passed); every
step of the path runs inside the library.  A missing or unloadable library raises: there is no fallback.
"""
import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_float, c_int32, c_int64, c_uint64, c_void_p

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsfs.so")

SFS_OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_OOM, ERR_STEP_LIMIT, ERR_TIMEOUT, ERR_MISSING_ROW = -1, -2, -3, -4, -5, -6, -7
LOGITS_BF16, LOGITS_F32 = 0, 1
PHASE_SLOW, PHASE_FAST = 0, 1
SAMPLER_SLOWFAST, SAMPLER_LOW_CONFIDENCE, SAMPLER_RANDOM = 0, 1, 2
CONF_QBITS = 28
MAX_W_HIST = 8
TRACE_INTS = 8


class Config(Structure):
    _fields_ = [(n, c_int32) for n in ("n_layers", "d_model", "n_heads", "head_dim", "d_ff", "vocab", "mask_id")] + \
               [(n, c_float) for n in ("rms_eps", "rope_theta", "logit_scale")]


class Weights(Structure):
    _fields_ = [("tok_emb", c_void_p), ("final_norm", c_void_p), ("lm_head", c_void_p)] + \
               [(n, POINTER(c_void_p)) for n in ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")]


class Params(Structure):
    _fields_ = [("tau_min_conf", c_float), ("tau_high_conf", c_float), ("sigma2_stable", c_float),
                ("k_max", c_int32), ("w_hist", c_int32), ("k_slow", c_int32), ("k_fast", c_int32),
                ("max_steps", c_int32), ("min_high_count", c_int32),
                ("sampler", c_int32), ("block_len", c_int32), ("seed_lo", ctypes.c_uint32), ("seed_hi", ctypes.c_uint32)]

    @staticmethod
    def default(**kw):
        p = Params(0.1, 0.85, 1.0, 8, 2, 1, 1, 0, 1, 0, 0, 0, 0)
        if "seed" in kw:
            seed = int(kw.pop("seed"))
            kw["seed_lo"], kw["seed_hi"] = seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF
        for k, v in kw.items():
            setattr(p, k, v)
        return p


class CacheParams(Structure):
    _fields_ = [("k_prompt", c_int32), ("k_response", c_int32), ("rho", ctypes.c_double)]


STATE_INTS = 32
STATE_FIELDS = ["phase", "s_cycle", "hi", "step_count", "hist_len"] + [f"hist{i}" for i in range(MAX_W_HIST)] + \
               ["k_remaining", "n_masked", "steps_done", "n_slow", "n_fast", "n_cycles", "n_fallback", "done", "status"]

_lib = None


class SfsError(RuntimeError):
    def __init__(self, status, message):
        super().__init__(f"libsfs status {status}: {message}")
        self.status = status


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} is missing: build it with `python -m paper_2506_10848_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        L.sfs_last_error.restype = c_char_p
        L.sfs_status_string.restype = c_char_p
        L.sfs_status_string.argtypes = [c_int32]
        _lib = L
    return _lib


def _ptr(t):
    """torch tensor / int / None -> c_void_p."""
    if t is None:
        return c_void_p(0)
    if isinstance(t, int):
        return c_void_p(t)
    return c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        return c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return c_void_p(stream)
    return c_void_p(stream.cuda_stream)


def _check(rc):
    if rc != SFS_OK:
        raise SfsError(rc, lib().sfs_last_error().decode())


def sfs_last_error():
    return lib().sfs_last_error().decode()


def sfs_status_string(status):
    return lib().sfs_status_string(status).decode()


def sfs_version():
    return lib().sfs_version()


def sfs_row_stats(logits, logits_dtype, vocab, ld, n_rows_dev, max_rows, argmax=None, sq=None, conf=None, stream=None):
    _check(lib().sfs_row_stats(_ptr(logits), c_int32(logits_dtype), c_int32(vocab), c_int64(ld), _ptr(n_rows_dev),
                               c_int32(max_rows), _ptr(argmax), _ptr(sq), _ptr(conf), _stream(stream)))


def sfs_row_stats_bounds(logits, vocab, ld, n_rows_dev, max_rows, lo, hi, argmax=None, stream=None):
    _check(lib().sfs_row_stats_bounds(_ptr(logits), c_int32(vocab), c_int64(ld), _ptr(n_rows_dev), c_int32(max_rows), _ptr(lo), _ptr(hi),
                                      _ptr(argmax), _stream(stream)))


def sfs_state_init(state, B, gen_len, params, stream=None):
    _check(lib().sfs_state_init(_ptr(state), c_int32(B), c_int32(gen_len), byref(params), _stream(stream)))


def sfs_select_session_create(vocab, max_batch, max_seq):
    h = c_void_p()
    _check(lib().sfs_select_session_create(c_int32(vocab), c_int32(max_batch), c_int32(max_seq), byref(h)))
    return h


def sfs_session_destroy(session):
    _check(lib().sfs_session_destroy(session))


def sfs_select(session, logits, logits_dtype, ld, rows, n_rows_dev, max_rows, tokens, mask, B, S, P, state, params,
               sel_count=None, sel_pos=None, sel_tok=None, next_rows=None, next_n_rows=None, trace=None, stream=None):
    _check(lib().sfs_select(session, _ptr(logits), c_int32(logits_dtype), c_int64(ld), _ptr(rows), _ptr(n_rows_dev),
                            c_int32(max_rows), _ptr(tokens), _ptr(mask), c_int32(B), c_int32(S), c_int32(P),
                            _ptr(state), byref(params), _ptr(sel_count), _ptr(sel_pos), _ptr(sel_tok),
                            _ptr(next_rows), _ptr(next_n_rows), _ptr(trace), _stream(stream)))


def sfs_linear(A, lda, Bm, ldb, C, ldc, M, N, K, out_dtype=0, scale=1.0, stream=None):
    _check(lib().sfs_linear(_ptr(A), c_int64(lda), _ptr(Bm), c_int64(ldb), _ptr(C), c_int64(ldc), c_int32(M), c_int32(N),
                            c_int32(K), c_int32(out_dtype), c_float(scale), _stream(stream)))


def sfs_check_device_status(stream=None):
    rc = lib().sfs_check_device_status(_stream(stream))
    if rc != SFS_OK:
        raise SfsError(rc, lib().sfs_last_error().decode())


def sfs_attention(qk, vt, out, B, S, n_heads, head_dim, stream=None):
    _check(lib().sfs_attention(_ptr(qk), _ptr(vt), _ptr(out), c_int32(B), c_int32(S), c_int32(n_heads), c_int32(head_dim),
                               _stream(stream)))


class Model:
    """Owns the sfs_model handle and keeps the weight tensors (borrowed by the library) alive."""

    def __init__(self, shape, weights):
        """shape: an object with the sfs_config field names; weights: dict of CUDA bf16 tensors as produced by
        workloads.model_weights(..., device='cuda')."""
        self.cfg = Config(*(int(getattr(shape, n)) for n in ("n_layers", "d_model", "n_heads", "head_dim", "d_ff", "vocab", "mask_id")),
                          *(float(getattr(shape, n)) for n in ("rms_eps", "rope_theta", "logit_scale")))
        self.weights = weights
        nl = self.cfg.n_layers
        self._tables = {}
        w = Weights()
        w.tok_emb, w.final_norm, w.lm_head = (weights[k].data_ptr() for k in ("tok_emb", "final_norm", "lm_head"))
        for name in ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down"):
            arr = (c_void_p * nl)(*[weights["layers"][l][name].data_ptr() for l in range(nl)])
            self._tables[name] = arr
            setattr(w, name, ctypes.cast(arr, POINTER(c_void_p)))
        self.handle = c_void_p()
        _check(lib().sfs_model_create(byref(self.cfg), byref(w), byref(self.handle)))

    def close(self):
        if self.handle:
            lib().sfs_model_destroy(self.handle)
            self.handle = c_void_p()


def sfs_session_create(model, max_batch, max_seq):
    h = c_void_p()
    _check(lib().sfs_session_create(model.handle if isinstance(model, Model) else model, c_int32(max_batch), c_int32(max_seq), byref(h)))
    return h


def sfs_forward(session, tokens, B, S, rows, n_rows_dev, max_rows, logits, logits_dtype, stream=None):
    _check(lib().sfs_forward(session, _ptr(tokens), c_int32(B), c_int32(S), _ptr(rows), _ptr(n_rows_dev), c_int32(max_rows),
                             _ptr(logits), c_int32(logits_dtype), _stream(stream)))


def sfs_cache_enable(session, k_prompt=100, k_response=5, rho=0.25, off=False):
    if off:
        _check(lib().sfs_cache_enable(session, None))
        return
    p = CacheParams(int(k_prompt), int(k_response), float(rho))
    _check(lib().sfs_cache_enable(session, byref(p)))


def sfs_cache_reset(session):
    _check(lib().sfs_cache_reset(session))


def sfs_cache_dump(session, sets=None, sims=None):
    _check(lib().sfs_cache_dump(session, _ptr(sets), _ptr(sims)))


def sfs_forward_cached(session, tokens, B, S, P, state, rows, n_rows_dev, max_rows, logits, logits_dtype, sets=None, sims=None,
                       stream=None):
    """Returns n_sel, the number of recomputed rows per sequence and layer in this step."""
    n = c_int32(0)
    _check(lib().sfs_forward_cached(session, _ptr(tokens), c_int32(B), c_int32(S), c_int32(P), _ptr(state), _ptr(rows), _ptr(n_rows_dev),
                                    c_int32(max_rows), _ptr(logits), c_int32(logits_dtype), _ptr(sets), _ptr(sims), byref(n),
                                    _stream(stream)))
    return n.value


def sfs_generate(session, prompt, B, P, gen_len, params, out_tokens, state_out=None, trace=None, max_trace_steps=0, stream=None):
    _check(lib().sfs_generate(session, _ptr(prompt), c_int32(B), c_int32(P), c_int32(gen_len), byref(params), _ptr(out_tokens),
                              _ptr(state_out), _ptr(trace), c_int32(max_trace_steps), _stream(stream)))


def sfs_generate_begin(session, prompt, B, P, gen_len, params, stream=None):
    _check(lib().sfs_generate_begin(session, _ptr(prompt), c_int32(B), c_int32(P), c_int32(gen_len), byref(params), _stream(stream)))


def sfs_generate_steps(session, n_steps, trace=None, max_trace_steps=0, logits_dump=None, rows_dump=None, n_rows_dump=None, stream=None):
    _check(lib().sfs_generate_steps(session, c_int32(n_steps), _ptr(trace), c_int32(max_trace_steps), _ptr(logits_dump),
                                    _ptr(rows_dump), _ptr(n_rows_dump), _stream(stream)))


def sfs_generate_end(session, out_tokens=None, state_out=None, stream=None):
    """Returns (n_active, steps_enqueued)."""
    na, ns = c_int32(0), c_int32(0)
    _check(lib().sfs_generate_end(session, _ptr(out_tokens), _ptr(state_out), byref(na), byref(ns), _stream(stream)))
    return na.value, ns.value


K_CLASSES = ["embed", "rmsnorm", "gemm_qkv", "rope", "attention", "gemm_o", "gemm_gate_up", "gemm_down", "gemm_lm_head",
             "row_stats", "select", "cache"]


def sfs_profile(session, enable, read=True):
    """Returns (ms per class dict, launches per class dict, total launches) gathered since the previous call."""
    n = len(K_CLASSES)
    ms = (c_float * n)()
    cnt = (c_int64 * n)()
    tot = c_int64(0)
    _check(lib().sfs_profile(session, c_int32(1 if enable else 0), ms if read else None, cnt if read else None, byref(tot)))
    return dict(zip(K_CLASSES, list(ms))), dict(zip(K_CLASSES, list(cnt))), tot.value


STATIC_MAX_POSITIONS, STATIC_MAX_BATCH = 16384, 64


def sfs_select_static(vocab, logits, logits_dtype, ld, rows, n_rows_dev, max_rows, tokens, mask, B, S, P, state, params,
                      sel_count=None, sel_pos=None, sel_tok=None, next_rows=None, next_n_rows=None, trace=None, stream=None):
    """sfs_select without a session: the scratch is a fixed array inside the library, so nothing is allocated."""
    _check(lib().sfs_select_static(c_int32(vocab), _ptr(logits), c_int32(logits_dtype), c_int64(ld), _ptr(rows), _ptr(n_rows_dev),
                                   c_int32(max_rows), _ptr(tokens), _ptr(mask), c_int32(B), c_int32(S), c_int32(P),
                                   _ptr(state), byref(params), _ptr(sel_count), _ptr(sel_pos), _ptr(sel_tok),
                                   _ptr(next_rows), _ptr(next_n_rows), _ptr(trace), _stream(stream)))
