#!/usr/bin/env python
"""Benchmark of the SlowFast denoising hot path at the LLaDA-8B shape.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 8b|tiny]

One "step" is one denoising step of the whole hot path: forward over prompt + partially masked response,
LM head for the masked rows in scope, row statistics, SlowFast selection.  The workload is the
LLaDA-8B-shaped random-init model, batch 1, 256 prompt ids + 256 masked positions (synthetic, seeded).
K steps are timed with CUDA events on the launching stream after W warm-up steps; when a generation
finishes inside the region the next one starts at once.  Prints one JSON line.

Under torchrun (N > 1) every rank runs an independent replica on its own GPU (the path has no exchange
step); the value is the sum of the ranks' tokens over the slowest rank's time.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"], bf16_tflops_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def gemm_traffic_from_profiles():
    """DRAM read + write bytes per GEMM launch, from the tracked summary of the ncu capture of this kernel; None when the
    kernel's source file is no longer the one that was captured (the counters would describe another kernel)."""
    import hashlib
    import re
    path = os.path.join(ROOT, "profiles", "gemm_kernel_llada8b_dram_traffic.md")
    src = os.path.join(ROOT, "paper_2506_10848_b200", "csrc", "gemm_tcgen05.cu")
    try:
        text = open(path).read()
        sha = hashlib.sha256(open(src, "rb").read()).hexdigest()
    except OSError:
        return None
    m_t = re.search(r"traffic_bytes_per_launch:\s*([0-9.eE+]+)", text)
    m_h = re.search(r"kernel_source_sha256:\s*([0-9a-f]{64})", text)
    if not m_t or not m_h or m_h.group(1) != sha:
        return None
    return float(m_t.group(1))


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def step_flops(shape, T, S, rows):
    """Algorithmic FLOPs of one denoising step: projections, attention, LM head for `rows` rows."""
    d, ff, V, nl = shape.d_model, shape.d_ff, shape.vocab, shape.n_layers
    gemm = 2.0 * T * (4 * d * d + 3 * d * ff) * nl
    attn = 4.0 * T * S * d * nl
    head = 2.0 * rows * d * V
    return gemm, attn, head


def step_bytes(shape, T, rows):
    d, ff, V, nl = shape.d_model, shape.d_ff, shape.vocab, shape.n_layers
    weights = 2.0 * ((4 * d * d + 3 * d * ff) * nl + d * V)
    act = T * nl * (2 * d * 4 * 2 + 2 * d + 2 * 2 * d + 2 * d + 2 * d + 2 * 2 * ff)      # residual r/w (fp32), h, q|k, vT, attn, hidden w+r
    logits = 2.0 * rows * V * 2
    return weights + act + logits


def run_ours(args, rank, world):
    import torch
    from paper_2506_10848_b200 import binding as sfs
    from paper_2506_10848_b200 import workloads as W

    local = int(os.environ.get("LOCAL_RANK", rank))
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if args.workload == "tiny":
        shape, P, L, B, name = W.TINY, 32, 64, 1, "tiny 2-layer d=256 model, batch 1, prompt 32 + 64 masked"
    else:
        shape, P, L, B, name = W.LLADA_8B, 256, 256, 1, "LLaDA-8B-shaped random-init model, batch 1, prompt 256 + 256 masked, no cache"
    if args.layers:
        shape = W.with_layers(shape, args.layers)
        name += f" [reduced to {args.layers} layers: a profiling case, not a bench value]"
    S = P + L
    weights = W.model_weights(shape, seed=2 + rank, device=dev)
    model = sfs.Model(shape, weights)
    session = sfs.sfs_session_create(model, B, S)
    params = sfs.Params.default()
    prompt = W.prompt_ids(B, P, shape.vocab - 2, seed=2 + rank).to(dev)
    out = torch.zeros((B, S), dtype=torch.int32, device=dev)
    K, Wm = args.steps, args.warmup
    trace = torch.zeros((K + Wm + 8, B, sfs.TRACE_INTS), dtype=torch.int32, device=dev)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: W warm-up steps, then exactly K timed steps -------------------------
    class Runner:
        def __init__(self):
            self.left = 0                         # steps left in the current generation (N = L at most)
            self.gen_base = 0                     # trace row of the current generation's first step
            self.total = 0

        def step(self, n):
            done = 0
            while done < n:
                if self.left == 0:
                    sfs.sfs_generate_begin(session, prompt, B, P, L, params)
                    self.left, self.gen_base = L, self.total
                take = min(n - done, self.left)
                sfs.sfs_generate_steps(session, take, trace[self.gen_base:], K + Wm + 8 - self.gen_base)
                self.left -= take
                done += take
                self.total += take

    r = Runner()
    r.step(Wm)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = sfs.sfs_profile(session, False, read=False)[2]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    r.step(K)
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    launches = sfs.sfs_profile(session, False, read=False)[2] - launches0
    sfs.sfs_check_device_status()
    tr = trace[Wm:Wm + K].cpu()
    tokens = int(tr[:, :, 5].sum())               # n_sel of every timed step
    productive = int((tr[:, :, 5].sum(dim=1) > 0).sum())   # steps that unmasked something (all of them, normally)

    # ---- per-kernel breakdown: the same steps again with CUDA events around every launch --------------
    prof_steps = min(K, 16)
    sfs.sfs_generate_begin(session, prompt, B, P, L, params)
    sfs.sfs_profile(session, True, read=False)
    sfs.sfs_generate_steps(session, prof_steps, None, 0)
    ms_cls, cnt_cls, _ = sfs.sfs_profile(session, False, read=True)
    gemm_classes = ["gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down", "gemm_lm_head"]
    gemm_ms = sum(ms_cls[c] for c in gemm_classes)
    gemm_launches = sum(cnt_cls[c] for c in gemm_classes)
    T = B * S
    # the first prof_steps steps of a generation see B*L, B*L-1, ... masked rows (one token per step here)
    head_rows = sum(max(B * L - i, 1) for i in range(prof_steps)) / prof_steps
    g_fl, a_fl, h_fl = step_flops(shape, T, S, head_rows)
    gemm_tflops = (g_fl + h_fl) * prof_steps / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else None

    # ---- end to end through sfs_generate with host buffers --------------------------------------------
    e2e = None
    if args.e2e:
        host_prompt = prompt.cpu().pin_memory()
        host_out = torch.zeros((B, S), dtype=torch.int32).pin_memory()
        d_prompt = torch.zeros_like(prompt)
        barrier()
        t0 = time.perf_counter()
        d_prompt.copy_(host_prompt, non_blocking=True)
        state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=dev)
        sfs.sfs_generate(session, d_prompt, B, P, L, params, out, state)
        host_out.copy_(out, non_blocking=True)
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        gsteps = int(state[:, sfs.STATE_FIELDS.index("steps_done")].max())
        e2e = {"value": B * L / (t1 - t0), "unit": "tokens/s", "h2d_bytes_per_step": B * P * 4 / max(gsteps, 1),
               "d2h_bytes_per_step": B * S * 4 / max(gsteps, 1), "steps": gsteps, "seconds": t1 - t0,
               "note": "one sfs_generate call: pinned host prompt -> device, full SlowFast loop, tokens -> pinned host"}

    extras = None
    if args.extras and world == 1 and args.workload == "8b" and not args.layers:
        sfs.sfs_session_destroy(session)
        session = None
        torch.cuda.empty_cache()
        extras = run_extras(torch, sfs, W, model, shape, dev, measured_peaks(), weights)
    res = dict(extras=extras, productive=productive, ms=ms, tokens=tokens, launches=launches, clocks=clocks, ms_cls=ms_cls, cnt_cls=cnt_cls, gemm_ms=gemm_ms,
               gemm_launches=gemm_launches, gemm_tflops=gemm_tflops, prof_steps=prof_steps, e2e=e2e, name=name, shape=shape,
               T=T, S=S, B=B, L=L, P=P, head_rows=head_rows)
    if session is not None:
        sfs.sfs_session_destroy(session)
    model.close()
    return res


def time_back_to_back(torch, fn, n):
    """Device time per call of n calls enqueued back to back (CUDA events on the launching stream)."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(n):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / n


def run_epilogue(torch, sfs, W, shape, dev, peaks):
    """The sampling-epilogue microbenchmark: row statistics on cold bf16 logits, one slow and one fast selection step."""
    out = {}
    V = shape.vocab
    # ---- sampling epilogue: bf16 [256, V] logits with planted winners; 4 rotating copies (259 MB > L2) keep every launch cold
    R = 256
    bufs = [W.planted_logits(R, V, seed=1, device=dev) for _ in range(4)]
    arg = torch.empty(R, dtype=torch.int32, device=dev); sq = torch.empty(R, dtype=torch.int64, device=dev)
    rs = lambda i: sfs.sfs_row_stats(bufs[i % 4], sfs.LOGITS_BF16, V, V, None, R, argmax=arg, sq=sq)
    time_back_to_back(torch, rs, 8)
    us_canonical = time_back_to_back(torch, rs, 32) * 1e3
    # the pass that streams the logits from HBM inside sfs_select / sfs_generate: exact argmax + enclosure of S_q per row
    lo_b = torch.empty(R, dtype=torch.int64, device=dev); hi_b = torch.empty(R, dtype=torch.int64, device=dev)
    rb = lambda i: sfs.sfs_row_stats_bounds(bufs[i % 4], V, V, None, R, lo_b, hi_b, arg)
    time_back_to_back(torch, rb, 8)
    us = time_back_to_back(torch, rb, 32) * 1e3
    # one slow and one fast selection step on those logits (row statistics + transition rule)
    ssel = sfs.sfs_select_session_create(V, 1, R)
    rows = torch.arange(R, dtype=torch.int32, device=dev)
    params = sfs.Params.default()
    lo, hi = W.span(R, seed=1)

    def sel_step(i, fast):
        tok = torch.full((1, R), shape.mask_id, dtype=torch.int32, device=dev); msk = torch.ones((1, R), dtype=torch.uint8, device=dev)
        st = torch.zeros((1, sfs.STATE_INTS), dtype=torch.int32, device=dev)
        sfs.sfs_state_init(st, 1, R, params)
        if fast:
            row = st[0].cpu(); row[sfs.STATE_FIELDS.index("phase")] = 1; row[sfs.STATE_FIELDS.index("s_cycle")] = lo
            row[sfs.STATE_FIELDS.index("hi")] = hi; st[0] = row.to(dev)
        cnt = torch.zeros(1, dtype=torch.int32, device=dev)
        torch.cuda.synchronize()
        return time_back_to_back(torch, lambda j: sfs.sfs_select(ssel, bufs[(i + j) % 4], sfs.LOGITS_BF16, V, rows, None, R, tok, msk, 1, R, 0, st,
                                                                  params, sel_count=cnt), 1) * 1e3

    def sel_chain(fast, n=12):
        """n complete selection steps back to back on cold logits (fresh state each: the same decision every time)."""
        sts, toks, msks = [], [], []
        for _ in range(n):
            tok = torch.full((1, R), shape.mask_id, dtype=torch.int32, device=dev); msk = torch.ones((1, R), dtype=torch.uint8, device=dev)
            st = torch.zeros((1, sfs.STATE_INTS), dtype=torch.int32, device=dev)
            sfs.sfs_state_init(st, 1, R, params)
            if fast:
                row = st[0].cpu(); row[sfs.STATE_FIELDS.index("phase")] = 1; row[sfs.STATE_FIELDS.index("s_cycle")] = lo
                row[sfs.STATE_FIELDS.index("hi")] = hi; st[0] = row.to(dev)
            sts.append(st); toks.append(tok); msks.append(msk)
        cnt = torch.zeros(1, dtype=torch.int32, device=dev)
        torch.cuda.synchronize()
        return time_back_to_back(torch, lambda j: sfs.sfs_select(ssel, bufs[j % 4], sfs.LOGITS_BF16, V, rows, None, R, toks[j], msks[j], 1, R, 0,
                                                                  sts[j], params, sel_count=cnt), n) * 1e3
    sel_step(0, False)
    slow_us, fast_us = sel_step(1, False), sel_step(2, True)
    sel_chain(False, 4)
    slow_chain_us, fast_chain_us = sel_chain(False), sel_chain(True)
    sfs.sfs_session_destroy(ssel)
    gbs = R * V * 2 / us * 1e-3
    out["epilogue"] = {"workload": f"bf16 logits [{R}, {V}], planted winners, seed 1; cold (4 rotating copies > L2)", "row_stats_us": us,
                       "hbm_gbs": gbs, "frac_of_measured_hbm_peak": gbs / peaks["hbm_gbs"],
                       "kernel": "rowstats_bounds_bf16: the one pass over HBM of the selection step (exact argmax, enclosure of S_q); rows whose "
                                 "enclosure leaves the step's comparisons open are recomputed canonically from L2 by a second launch",
                       "canonical_all_rows_us": us_canonical, "canonical_all_rows_hbm_gbs": R * V * 2 / us_canonical * 1e-3,
                       "select_slow_step_us": slow_us, "select_fast_step_us": fast_us,
                       "select_slow_step_enqueue_bound_us": slow_chain_us, "select_fast_step_enqueue_bound_us": fast_chain_us,
                       "select_step_note": "whole sfs_select call (four launches: streaming pass, decision, canonical recompute of the listed rows, "
                                           "selection): one call timed alone, launch latency included; and 12 calls enqueued back to back, which is "
                                           "bound by the host's enqueue rate through the Python binding, not by the device (per-kernel device times: "
                                           "profiles/rowstats_bounds_256x126464.md)",
                       "span": [lo, hi]}
    del bufs
    torch.cuda.empty_cache()
    return out


def run_extras(torch, sfs, W, model, shape, dev, peaks, weights=None):
    """The other workloads of the benchmark definition, measured on the same model: the sampling-epilogue
    microbenchmark, the cached run (prompt 1024 + 512 masked) and the batch of 8 sequences (512 + 256)."""
    out = run_epilogue(torch, sfs, W, shape, dev, peaks)
    V = shape.vocab
    params = sfs.Params.default()

    def timed_steps(session, n):
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
        evs[0].record()
        for i in range(n):
            sfs.sfs_generate_steps(session, 1, None, 0)
            evs[i + 1].record()
        torch.cuda.synchronize()
        return [evs[i].elapsed_time(evs[i + 1]) for i in range(n)]

    # ---- feature cache: prompt 1024 + 512 masked and the long response 1024 + 1024, at both (K_p, K_r) settings of Table 4
    def cached_run(P, L, settings):
        B = 1
        session = sfs.sfs_session_create(model, B, P + L)
        prompt = W.prompt_ids(B, P, V - 2, seed=3).to(dev)
        sfs.sfs_generate_begin(session, prompt, B, P, L, params)
        timed_steps(session, 2)
        plain = timed_steps(session, 5)
        res = {"workload": f"8B shape, batch 1, prompt {P} + {L} masked, seed 3", "uncached_ms_per_step": sum(plain) / len(plain)}
        # roofline of a step that recomputes ceil(rho L) rows: every weight streams once; FLOPs of the recomputed rows, the value
        # projection of all response rows and the LM head of the masked rows
        d, ff, nl = shape.d_model, shape.d_ff, shape.n_layers
        for (kp, kr, rho) in settings:
            sfs.sfs_cache_enable(session, kp, kr, rho)
            sfs.sfs_generate_begin(session, prompt, B, P, L, params)
            n = min(kr, 30) * 2 + 1
            ts = timed_steps(session, n)                        # step 0: full refresh; steps kr, 2 kr: response refresh
            sfs.sfs_check_device_status()
            refresh = [ts[i] for i in range(1, n) if i % kr == 0]
            part = [ts[i] for i in range(1, n) if i % kr != 0]
            cyc = (sum(refresh) / len(refresh) + (kr - 1) * sum(part) / len(part)) / kr
            nr = -(-int(rho * L * 4096) // 4096)
            fl = 2.0 * nr * (4 * d * d + 3 * d * ff) * nl + 2.0 * L * d * d * nl + 4.0 * nr * (P + L) * d * nl + 2.0 * L * d * V
            by = 2.0 * ((4 * d * d + 3 * d * ff) * nl + d * V) + nl * (P + L) * d * 2 * 2 + 2.0 * L * V * 2
            roof = max(fl / (peaks["bf16_tflops"] * 1e12), by / (peaks["hbm_gbs"] * 1e9)) * 1e3
            res[f"kp{kp}_kr{kr}"] = {"params": f"K_p {kp}, K_r {kr}, rho {rho}", "cached_ms_per_step_cycle_avg": cyc,
                                    "cached_partial_step_ms": sum(part) / len(part), "cached_response_refresh_step_ms": sum(refresh) / len(refresh),
                                    "cached_full_refresh_step_ms": ts[0], "speedup": res["uncached_ms_per_step"] / cyc,
                                    "partial_step_roofline_ms": roof, "partial_step_roofline_frac": roof / (sum(part) / len(part)),
                                    "partial_step_roofline_bound": "hbm" if by / (peaks["hbm_gbs"] * 1e9) >= fl / (peaks["bf16_tflops"] * 1e12) else "tensor"}
        sfs.sfs_cache_enable(session, 1, 1, 0.0, off=True)
        sfs.sfs_session_destroy(session)
        torch.cuda.empty_cache()
        return res

    out["cached_1024_512"] = cached_run(1024, 512, [(100, 5, 0.25), (500, 30, 0.25)])
    out["cached_1024_1024"] = cached_run(1024, 1024, [(100, 5, 0.25), (500, 30, 0.25)])

    # ---- batch of 8 independent sequences, prompt 512 + 256 masked
    B, P, L = 8, 512, 256
    session = sfs.sfs_session_create(model, B, P + L)
    prompt = W.prompt_ids(B, P, V - 2, seed=4).to(dev)
    sfs.sfs_generate_begin(session, prompt, B, P, L, params)
    timed_steps(session, 2)
    ts = timed_steps(session, 6)
    sfs.sfs_check_device_status()
    ms = sum(ts) / len(ts)
    g_fl, a_fl, h_fl = step_flops(shape, B * (P + L), P + L, B * L)
    roof = max((g_fl + a_fl + h_fl) / (peaks["bf16_tflops"] * 1e12), step_bytes(shape, B * (P + L), B * L) / (peaks["hbm_gbs"] * 1e9)) * 1e3
    roof_sus = max((g_fl + a_fl + h_fl) / (peaks["bf16_tflops_sustained"] * 1e12), step_bytes(shape, B * (P + L), B * L) / (peaks["hbm_gbs"] * 1e9)) * 1e3
    out["batch8_512_256"] = {"workload": "8B shape, batch 8, prompt 512 + 256 masked, seed 4", "ms_per_step": ms, "tokens_per_s": B / (ms * 1e-3),
                             "step_roofline_ms": roof, "step_roofline_frac": roof / ms,
                             "step_roofline_ms_sustained_peak": roof_sus, "step_roofline_frac_sustained_peak": roof_sus / ms,
                             "note": "one token per sequence and step with random-init logits"}
    sfs.sfs_session_destroy(session)
    torch.cuda.empty_cache()

    # ---- the main workload again with confident logits: the same weights under a logit scale of 300, so that both
    # thresholds fire and the accelerated stage unmasks many tokens per step (random-init logits never do)
    if weights is not None:
        dct = shape.asdict(); dct["logit_scale"] = 300.0
        m2 = sfs.Model(W.Shape(**dct), weights)
        B, P, L = 1, 256, 256
        session = sfs.sfs_session_create(m2, B, P + L)
        prompt = W.prompt_ids(B, P, V - 2, seed=2).to(dev)
        outb = torch.zeros((B, P + L), dtype=torch.int32, device=dev)
        state = torch.zeros((B, sfs.STATE_INTS), dtype=torch.int32, device=dev)
        def gen(pp):
            sfs.sfs_generate(session, prompt, B, P, L, pp, outb, state)          # warm-up: plans for this session
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            sfs.sfs_generate(session, prompt, B, P, L, pp, outb, state)
            e1.record()
            torch.cuda.synchronize()
            sfs.sfs_check_device_status()
            return int(state[0, sfs.STATE_FIELDS.index("steps_done")]), e0.elapsed_time(e1)

        steps, ms = gen(params)
        _, enq = sfs.sfs_generate_end(session)
        out["confident_256_256"] = {"workload": "8B shape, batch 1, prompt 256 + 256 masked, logits x300 (synthetic confidence), seed 2",
                                    "denoise_steps": steps, "steps_enqueued": enq, "surplus_steps": enq - steps, "tokens": L, "ms_total": ms,
                                    "ms_per_step": ms / max(steps, 1), "tokens_per_s": L / (ms * 1e-3),
                                    "note": "wall time of one sfs_generate call; at most 2 steps are enqueued ahead of the device"}
        # the LLaDA strategies of Section 3.1 on the same logits (the 1.00x rows of the paper's tables): step counts and time
        base = {}
        for name, kw in (("low_confidence_N256", dict(sampler=sfs.SAMPLER_LOW_CONFIDENCE)),
                         ("semi_ar_block32_low_confidence_N256", dict(sampler=sfs.SAMPLER_LOW_CONFIDENCE, block_len=32)),
                         ("low_confidence_N64", dict(sampler=sfs.SAMPLER_LOW_CONFIDENCE, max_steps=64)),
                         ("random_N256", dict(sampler=sfs.SAMPLER_RANDOM, seed=2))):
            st_, ms_ = gen(sfs.Params.default(**kw))
            base[name] = {"denoise_steps": st_, "ms_total": ms_, "tokens_per_s": L / (ms_ * 1e-3)}
        out["confident_256_256"]["llada_strategies_same_logits"] = base
        out["confident_256_256"]["step_ratio_vs_low_confidence_N256"] = base["low_confidence_N256"]["denoise_steps"] / max(steps, 1)
        out["confident_256_256"]["time_ratio_vs_low_confidence_N256"] = base["low_confidence_N256"]["ms_total"] / ms
        sfs.sfs_session_destroy(session)
        m2.close()
        torch.cuda.empty_cache()

        # ---- context for the GEMM roofline: the library's GEMM (torch.matmul, i.e. cuBLAS) on the same weights at the same row
        # counts, one call per weight matrix, 32 layers back to back (every pass streams the 13 GB of layer weights, as a step does).
        # Not part of the path and not a target: it says what the measured-peak denominator turns into at these shapes.
        d, ff, nl = shape.d_model, shape.d_ff, shape.n_layers
        lib = {}
        for T in (512, 6144):
            x = torch.randn((T, d), device=dev, dtype=torch.float32).to(torch.bfloat16)
            hid = torch.randn((T, ff), device=dev, dtype=torch.float32).to(torch.bfloat16)
            o_d = torch.empty((T, d), device=dev, dtype=torch.bfloat16)
            o_ff = torch.empty((T, ff), device=dev, dtype=torch.bfloat16)

            def one_pass():
                for lw in weights["layers"]:
                    for name in ("wq", "wk", "wv", "wo"):
                        torch.matmul(x, lw[name].t(), out=o_d)
                    torch.matmul(x, lw["w_gate"].t(), out=o_ff)
                    torch.matmul(x, lw["w_up"].t(), out=o_ff)
                    torch.matmul(hid, lw["w_down"].t(), out=o_d)

            n_pass = 160 if T == 512 else 16                   # about a second each: under the power cap like the timed step
            one_pass(); one_pass()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(n_pass):
                one_pass()
            e1.record()
            torch.cuda.synchronize()
            ms_pass = e0.elapsed_time(e1) / n_pass
            fl = 2.0 * T * (4 * d * d + 3 * d * ff) * nl
            lib[f"rows_{T}"] = {"ms_per_pass": ms_pass, "tflops": fl / (ms_pass * 1e-3) / 1e12, "gemm_calls_per_pass": 7 * nl}
            del x, hid, o_d, o_ff
        lib["note"] = ("torch.matmul (cuBLAS) bf16 on the layer weights, 7 calls per layer, no fusion, outputs discarded, about one second "
                       "per row count; context for roofline.achieved, whose kernels also do the SwiGLU, residual and transposed-V epilogues")
        out["library_gemm_context"] = lib
        torch.cuda.empty_cache()
    return out


def aggregate(torch, ms, tokens, launches, world, device):
    """Whole-job numbers over the ranks: slowest rank's time, summed tokens and launches."""
    if world <= 1:
        return ms, tokens, launches
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    k = torch.tensor([tokens, launches], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(k, op=torch.distributed.ReduceOp.SUM)
    return float(t[0]), int(k[0]), int(k[1])


ORACLE_LAYERS, ORACLE_HEAD_ROWS = 8, 64


def oracle_inputs(shape, P, L, seed=2):
    """Weights (fp32 numpy) of the sampled layers and the token ids: built once, outside every timed region."""
    import numpy as np
    from paper_2506_10848_b200 import workloads as W
    n_sampled = min(ORACLE_LAYERS, shape.n_layers)
    one = W.with_layers(shape, n_sampled)
    w = W.weights_to_numpy(W.model_weights(one, seed=seed), np.float32)
    tok = np.concatenate([W.prompt_ids(1, P, shape.vocab - 2, seed=seed).numpy(),
                          np.full((1, L), shape.mask_id, np.int32)], axis=1)
    return one, w, tok


def oracle_sample(shape, P, L, inputs=None):
    """One bounded sample of the oracle at the 8B shape (about ten seconds of host work): ORACLE_LAYERS transformer
    layers over the full sequence, the LM head and row statistics for ORACLE_HEAD_ROWS rows, and one selection step;
    extrapolated to a whole step."""
    import numpy as np
    from oracle import forward as F
    from oracle import rowstats as RS
    from oracle.scheduler import SlowFastParams, SlowFastState, rows_needed, slowfast_step

    one, w, tok = inputs if inputs is not None else oracle_inputs(shape, P, L)
    n_sampled = one.n_layers
    cfg = F.ModelConfig(**one.asdict())
    head_rows = min(ORACLE_HEAD_ROWS, L)
    t0 = time.perf_counter()
    logits = F.forward(cfg, w, tok, rows=[(0, P + i) for i in range(head_rows)], dtype=np.float32)
    t1 = time.perf_counter()
    # time the LM head + row statistics separately on the same rows to extrapolate to L rows
    hf = np.random.default_rng(0).standard_normal((head_rows, shape.d_model)).astype(np.float32)
    t2 = time.perf_counter()
    lg = hf @ w["lm_head"].T
    st = RS.row_stats(np.ascontiguousarray(lg, dtype=np.float32))
    t3 = time.perf_counter()
    stt = SlowFastState.fresh(L, SlowFastParams())
    rows = rows_needed(stt)
    a = {i: int(st["argmax"][i % head_rows]) for i in rows}
    sq = {i: int(st["sq"][i % head_rows]) for i in rows}
    slowfast_step(stt, a, sq, SlowFastParams())
    t4 = time.perf_counter()
    per_row = (t3 - t2) / head_rows
    layer_s = ((t1 - t0) - (t3 - t2)) / n_sampled        # forward minus its own head, per layer
    step_s = shape.n_layers * max(layer_s, 1e-6) + per_row * (L / 2.0) + (t4 - t3)
    return dict(step_seconds=step_s, layer_seconds=layer_s, head_row_seconds=per_row, sample_seconds=t4 - t0)


def run_reference(args, rank, world):
    from paper_2506_10848_b200 import workloads as W
    shape, P, L = (W.TINY, 32, 64) if args.workload == "tiny" else (W.LLADA_8B, 256, 256)
    inputs = oracle_inputs(shape, P, L)
    for _ in range(max(args.warmup, 0) and 1):
        oracle_sample(shape, P, L, inputs)
    ts = []
    for _ in range(max(1, min(args.steps, 3))):
        ts.append(oracle_sample(shape, P, L, inputs))
    step_s = sorted(t["step_seconds"] for t in ts)[len(ts) // 2]
    cores = os.cpu_count()
    value = 1.0 / step_s                                   # one token per step on random-init logits
    line = {"impl": "reference", "metric": "generated tokens/s at the LLaDA-8B shape (SlowFast, no cache)", "value": value,
            "unit": "tokens/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "LLaDA-8B-shaped random-init model, batch 1, prompt 256 + 256 masked, no cache"
                       if args.workload != "tiny" else "tiny"},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                             "sample": f"per step: {ORACLE_LAYERS} of the 32 layers over all 512 tokens + LM head and row statistics for "
                                       f"{ORACLE_HEAD_ROWS} rows + one selection step, in fp32 numpy; step time extrapolated as "
                                       "32 x layer + L/2 rows x head"},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="8b", choices=["8b", "tiny"])
    ap.add_argument("--layers", type=int, default=0, help="keep only this many layers (small case for ncu captures)")
    ap.add_argument("--no-e2e", dest="e2e", action="store_false")
    ap.add_argument("--no-extras", dest="extras", action="store_false", help="skip the epilogue / cached / batch-8 workloads")
    ap.add_argument("--no-cpu-baseline", dest="cpu", action="store_false")
    ap.add_argument("--epilogue-only", action="store_true", help="run only the sampling-epilogue microbenchmark (small case for ncu captures)")
    ap.add_argument("--cached-only", action="store_true",
                    help="run only a few feature-cache steps (prompt 1024 + 512 masked, K_p 100, K_r 5; with --layers: a small case for ncu launch lists)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, rank, world)
        return

    import torch
    if world > 1:
        torch.distributed.init_process_group("nccl")
    import __graft_entry__ as entry
    if rank == 0:
        entry.build()
    if world > 1:
        torch.distributed.barrier()
    if args.epilogue_only:
        # a profiling case, not a bench line: the microbenchmark alone (260 MB on the device)
        if rank == 0:
            from paper_2506_10848_b200 import binding as sfs
            from paper_2506_10848_b200 import workloads as W
            torch.cuda.set_device(0)
            print(json.dumps({"profiling_case": "sampling epilogue only", **run_epilogue(torch, sfs, W, W.LLADA_8B, "cuda:0", measured_peaks())}))
        return
    if args.cached_only:
        # a profiling case, not a bench line: a full refresh, four partial steps, a response refresh and one more partial step
        if rank == 0:
            from paper_2506_10848_b200 import binding as sfs
            from paper_2506_10848_b200 import workloads as W
            torch.cuda.set_device(0)
            shape = W.with_layers(W.LLADA_8B, args.layers) if args.layers else W.LLADA_8B
            model = sfs.Model(shape, W.model_weights(shape, seed=2, device="cuda:0"))
            session = sfs.sfs_session_create(model, 1, 1536)
            prompt = W.prompt_ids(1, 1024, shape.vocab - 2, seed=3).to("cuda:0")
            sfs.sfs_cache_enable(session, 100, 5, 0.25)
            sfs.sfs_generate_begin(session, prompt, 1, 1024, 512, sfs.Params.default())
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            sfs.sfs_generate_steps(session, 1, None, 0)
            e0.record()
            sfs.sfs_generate_steps(session, 4, None, 0)
            e1.record()
            sfs.sfs_generate_steps(session, 2, None, 0)
            torch.cuda.synchronize()
            sfs.sfs_check_device_status()
            print(json.dumps({"profiling_case": "feature-cache steps only", "layers": shape.n_layers,
                              "cached_partial_step_ms": e0.elapsed_time(e1) / 4}))
            sfs.sfs_session_destroy(session)
            model.close()
        return
    res = run_ours(args, rank, world)

    ms, tokens = res["ms"], res["tokens"]
    ms, tokens, launches = aggregate(torch, ms, tokens, res["launches"], world, "cuda")
    if rank != 0:
        if world > 1:
            torch.distributed.destroy_process_group()
        return

    peaks = measured_peaks()
    shape = res["shape"]
    K = args.steps
    ms_step = ms / K
    g_fl, a_fl, h_fl = step_flops(shape, res["T"], res["S"], res["head_rows"])
    step_roof_ms = max((g_fl + a_fl + h_fl) / (peaks["bf16_tflops"] * 1e12), step_bytes(shape, res["T"], res["head_rows"]) / (peaks["hbm_gbs"] * 1e9)) * 1e3
    step_roof_sus_ms = max((g_fl + a_fl + h_fl) / (peaks["bf16_tflops_sustained"] * 1e12), step_bytes(shape, res["T"], res["head_rows"]) / (peaks["hbm_gbs"] * 1e9)) * 1e3
    # the kernel is timed inside the step loop: a run of a second or more settles under the power cap, where cuBLAS itself
    # sustains the lower rate; a shorter run is held against the burst rate
    long_run = ms >= 1000.0
    gemm_peak = peaks["bf16_tflops_sustained"] if long_run else peaks["bf16_tflops"]
    roofline = {"bound": "tensor", "achieved": res["gemm_tflops"], "peak": gemm_peak, "unit": "TFLOP/s",
                "frac": (res["gemm_tflops"] / gemm_peak) if res["gemm_tflops"] else None,
                "frac_of_burst_peak": (res["gemm_tflops"] / peaks["bf16_tflops"]) if res["gemm_tflops"] else None,
                # DRAM read + write bytes per GEMM launch, read from the tracked ncu summary (null when the kernel changed since)
                "traffic": gemm_traffic_from_profiles() if (args.workload == "8b" and not args.layers) else None,
                "kernel": "gemm_kernel (tcgen05 projections: QKV, O, gate/up+SwiGLU, down, LM head)",
                "peak_source": peaks["source"] + (" (sustained cuBLAS bf16: the timed region ran %.1f s under the power cap)" % (ms * 1e-3) if long_run
                                                  else " (burst cuBLAS bf16: the timed region ran %.2f s)" % (ms * 1e-3)),
                "launches_timed": res["gemm_launches"], "ms_timed": res["gemm_ms"], "steps_timed": res["prof_steps"]}
    line = {"metric": "generated tokens/s at the LLaDA-8B shape (SlowFast, no cache)", "value": tokens / (ms * 1e-3),
            "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": args.warmup, "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": res["name"], "l2": "inputs larger than L2 (16 GB of weights streamed every step)",
                       "params": "tau_min 0.1, tau_high 0.85, K_max 8, W_hist 2, sigma2 1.0, k_slow = k_fast = 1, N = L"},
            "tokens_unmasked": tokens, "productive_steps": res["productive"], "gpu_launches": launches, "clocks": res["clocks"],
            # FLOPs at the burst cuBLAS peak (the stricter bar), and at the rate cuBLAS itself sustains under the power cap
            "step_roofline_ms": step_roof_ms, "step_roofline_frac": step_roof_ms / ms_step,
            "step_roofline_ms_sustained_peak": step_roof_sus_ms, "step_roofline_frac_sustained_peak": step_roof_sus_ms / ms_step,
            "kernel_ms_per_step": {k: v / res["prof_steps"] for k, v in res["ms_cls"].items()},
            "roofline": roofline, "e2e": res["e2e"]}
    if res["extras"]:
        line.update(res["extras"])
    if args.cpu and world == 1:
        from paper_2506_10848_b200 import workloads as W
        P, L = (32, 64) if args.workload == "tiny" else (256, 256)
        smp = oracle_sample(shape, P, L)
        line["cpu_baseline"] = {"value": 1.0 / smp["step_seconds"], "unit": "tokens/s", "cores": os.cpu_count(), "kind": "oracle",
                                "sample": f"{min(ORACLE_LAYERS, shape.n_layers)} of the {shape.n_layers} layers over all tokens + LM head and row statistics for "
                                          f"{min(ORACLE_HEAD_ROWS, L)} rows + one "
                                          f"selection step (fp32 numpy, {smp['sample_seconds']:.1f} s); step time extrapolated as "
                                          f"{shape.n_layers} x layer + L/2 rows x head; one token per step"}
    print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
