"""SlowFast Sampling hot path for masked-diffusion LLMs on B200 (sm_100a).

The product is the C-ABI library `libsfs.so` (declared in include/sfs.h, built from csrc/); `binding`
is a thin ctypes layer over it.  Nothing is loaded at import time; the library is opened on first use
and a missing library is an error, never a fallback.
"""
__all__ = ["binding", "workloads", "build"]
