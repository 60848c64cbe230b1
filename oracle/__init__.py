"""ORACLE — test infrastructure only.

A plain, slow CPU restatement of what the SlowFast-Sampling hot path computes: the mask predictor's
forward pass (numpy), the per-row sampling statistics (C, `rowstats.c`) and the slow/fast selection
rules (pure Python).  Nothing here is imported by the product package; only the tests, the smoke check
and the benchmark's CPU-baseline leg use it.  It shares no code, constants or headers with the CUDA path.
"""
