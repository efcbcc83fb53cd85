#!/usr/bin/env python
"""Benchmark of the rollout denoising step (attention -> LM head/confidence -> unmask selection).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A "step" is one pass of the whole hot path over one batch: dare_denoise_block on the LLaDA-8B-shaped
workload (batch 16 rollouts, prompt 512 + generation 256 in blocks of 32, top-k = 2 per step, so 16 steps
per block and 128 steps per generation; after 128 steps the token state is re-masked and the prefix length
returns to the prompt).  The metric is denoised (committed) tokens per second.

The default invocation (one GPU, no --workload) times that workload as the line's own value and then runs
short legs of the other workloads the metric is defined on (Dream-7B-shaped step, dual-cache block-diffusion
step, 4-layer end-to-end loop), attached under "workloads", each with its own roofline: for the dual-cache
step that is the K/V read rate of the attention kernel against the measured HBM bandwidth.

N > 1: every rank runs the same workload on its own rollouts (batch rows are independent, no data-path
collective); value = tokens of all ranks / max-over-ranks time ("weak" scaling).  Started without torchrun,
`--gpus N` starts the N ranks itself (torch.distributed.run on 127.0.0.1).

`--impl reference` times the CPU oracle (oracle/dare_oracle.py) as it stands on a bounded sample of the same
workload, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2604_04215_b200 import inputs as I  # noqa: E402

METRIC = "denoised_tokens_per_sec"
UNIT = "tokens/s"
NPOOL = 4   # distinct activation sets cycled through the steps
NOMINAL_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the workload's dominant kernel, from the ncu
# captures summarised under profiles/ (LM head: W leaves HBM once; dual-cache attention: the quarter-batch capture
# scaled by the batch, traffic grows in proportion to the rollouts)
DOMINANT_TRAFFIC_BYTES = {"llada8b": 1.0681e9, "dualcache": 4 * (1.3595e9 + 4.8e6)}
EXTRA_WORKLOADS = ("dream7b", "dualcache", "llada_loop")


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock, power and throttle reasons with nvidia-smi for the life of the run; `window` summarises
    the samples that fell into a wall-clock interval."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def window(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"], "samples": 0}
        time.sleep(0.12)                                # let the sample that covers the end of the window arrive
        sm, mx, pw, reasons = [], [], [], set()
        near = None                                     # the sample closest to the window, if none falls inside
        for ts, line in list(self.lines):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                rec = (float(f[0]), float(f[1]), float(f[2]))
            except ValueError:
                continue
            if ts < t0 or ts > t1 + 0.06:
                d = min(abs(ts - t0), abs(ts - t1))
                if near is None or d < near[0]:
                    near = (d, rec)
                continue
            sm.append(rec[0]); mx.append(rec[1]); pw.append(rec[2])
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            if near is None:
                return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"], "samples": 0}
            return {"sm_mhz": near[1][0], "sm_max_mhz": near[1][1], "power_w_max": near[1][2], "reasons": [],
                    "samples": 0, "note": f"window shorter than the sampling period; nearest sample {near[0] * 1e3:.0f} ms away"}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "power_w_max": float(max(pw)),
                "reasons": sorted(reasons), "samples": len(sm)}

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()       # the exact child started above
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        self.proc = None


def _rank_env():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0")))


def _barrier(world):
    torch.cuda.synchronize()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        torch.cuda.synchronize()


def _pick_peak(peaks, key_burst, key_sustained, seconds, clocks):
    """The denominator that matches the run.  The sustained figure (the library GEMM looped for seconds under the power
    limit) applies when the region itself lasted a second or more, or when its clock samples show the GPU held down:
    a power-cap sample AND a median SM clock at or below 0.8 of the maximum (one stray sample with the reason set, in a
    region of tens of milliseconds at nearly full clock, does not make a run power-limited).  Otherwise the burst
    figure applies."""
    if seconds >= 1.0:
        return peaks[key_sustained], "sustained"
    if clocks is not None and "sw_power_cap" in (clocks.get("reasons") or []):
        mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
        if mhz and mx and mhz <= 0.8 * mx:
            return peaks[key_sustained], "sustained"
    return peaks[key_burst], "burst"


def _tensor_roofline(kernel, flops_per_launch, ms_per_launch, peaks, seconds, clocks, traffic, extra=None):
    achieved = flops_per_launch / (ms_per_launch * 1e-3) / 1e12
    peak, which = _pick_peak(peaks, "bf16_tflops", "bf16_tflops_sustained", seconds, clocks)
    mhz = clocks.get("sm_mhz") if clocks else None
    r = {"bound": "tensor", "kernel": kernel, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
         "frac": achieved / peak, "traffic": traffic,
         "peak_source": f"{peaks['source']} {which} (instrumented region {seconds:.3f} s, "
                        f"{'power cap seen, SM clock held at or below 0.8 of its maximum' if which == 'sustained' and seconds < 1.0 else 'not held down by the power cap' if which == 'burst' else 'a second or longer'})",
         "frac_burst": achieved / peaks["bf16_tflops"], "frac_sustained": achieved / peaks["bf16_tflops_sustained"],
         "frac_nominal": achieved / NOMINAL_TFLOPS, "ms_per_launch": ms_per_launch,
         "sm_mhz": mhz, "cycles_per_launch": None if mhz is None else ms_per_launch * mhz * 1e3}
    if extra:
        r.update(extra)
    return r


def _hbm_roofline(kernel, bytes_per_launch, ms_per_launch, peaks, clocks, traffic, extra=None):
    achieved = bytes_per_launch / (ms_per_launch * 1e-3) / 1e9
    mhz = clocks.get("sm_mhz") if clocks else None
    r = {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
         "frac": achieved / peaks["hbm_gbs"], "traffic": traffic, "peak_source": peaks["source"] + " copy bandwidth",
         "frac_nominal": achieved / NOMINAL_HBM_GBS, "ms_per_launch": ms_per_launch, "sm_mhz": mhz}
    if extra:
        r.update(extra)
    return r


def _workload_label(wl):
    sel = "top-k " + str(wl.k) if wl.mode == I.SELECT_TOPK else "tau " + str(wl.threshold)
    suf = f" suffix{wl.suffix_cap}" if wl.suffix_cap else ""
    return (f"{wl.name}: B{wl.batch} L{wl.block_len} Hq{wl.n_q_heads}/Hkv{wl.n_kv_heads} d{wl.head_dim} D{wl.hidden} "
            f"V{wl.vocab} prompt{wl.prompt_len}+gen{wl.gen_len}{suf} {sel}")


def bench_step_workload(dare, ctx, wl, steps, warmup, rank, world, sampler, with_e2e, with_heads):
    """Times `steps` denoising steps of one single-layer workload through dare_denoise_block (device-resident
    inputs), then an instrumented pass of whole generations through the three entry points with CUDA events in
    between, optionally the end-to-end leg from pinned host memory.  Returns the pieces of the JSON line."""
    from paper_2604_04215_b200.dist import reduce_step_stats
    B, L = wl.batch, wl.block_len
    steps_per_block = -(-L // wl.k) if wl.mode == I.SELECT_TOPK else L
    steps_per_gen = steps_per_block * wl.n_blocks

    # ---- resident state: weights, in-place KV cache (filled over its whole capacity), pristine tokens
    w_h = I.normal_bf16(0, I.TID_W, (wl.vocab, wl.hidden), 0.02)           # same weights on every rank
    k_pre_h, v_pre_h, k_suf_h, v_suf_h = I.make_caches(wl)
    tok0_h = I.fresh_tokens(wl)
    w = w_h.cuda(); k_pre = k_pre_h.cuda(); v_pre = v_pre_h.cuda()
    k_suf = k_suf_h.cuda() if k_suf_h is not None else None
    v_suf = v_suf_h.cuda() if v_suf_h is not None else None
    suffix_len = torch.full((B,), wl.suffix_cap, dtype=torch.int32, device="cuda") if wl.suffix_cap else None
    tok0 = tok0_h.cuda()
    tokens = tok0.clone()
    plen_blocks = [torch.full((B,), wl.prompt_len + b * L, dtype=torch.int32, device="cuda") for b in range(wl.n_blocks)]
    # ---- per-step activations: a small pool, pinned on the host for the end-to-end leg
    pool_h = []
    for i in range(NPOOL):
        q, _, _, x = I.make_step_activations(wl, i, inplace_block=True)
        pool_h.append((q.pin_memory(), x.pin_memory()) if with_e2e else (q, x))
    pool = [(q.cuda(), x.cuda()) for q, x in pool_h]
    attn_out = torch.empty(B, L, wl.n_q_heads, wl.head_dim, dtype=torch.bfloat16, device="cuda")
    pred = torch.empty(B * L, dtype=torch.int32, device="cuda")
    conf = torch.empty(B * L, dtype=torch.float32, device="cuda")
    n_total = steps + warmup
    nc_all = torch.zeros(max(n_total, 1), B, dtype=torch.int32, device="cuda")
    nr = torch.zeros(B, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()

    def step(t, q, x, nc, nr_out=None):
        g = t % steps_per_gen
        b = g // steps_per_block
        if g == 0:
            tokens.copy_(tok0)                                  # new generation: re-mask (one small copy)
        dare.dare_denoise_block(ctx, q, k_pre, v_pre, plen_blocks[b], None, None, k_suf, v_suf, suffix_len,
                                attn_out, None, x, w, wl.mask_id, True, tokens, wl.prompt_len + b * L,
                                wl.mode, wl.threshold, wl.k, pred, conf, nc, nr if nr_out is None else nr_out,
                                stream=stream)

    # ---- device-resident timed region
    for t in range(warmup):
        q, x = pool[t % NPOOL]
        step(t, q, x, nc_all[t])
    _barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0 = time.time()
    launches0 = dare.dare_kernel_launches()
    e0.record(stream)
    for t in range(warmup, n_total):
        q, x = pool[t % NPOOL]
        step(t, q, x, nc_all[t])
    e1.record(stream)
    launches = dare.dare_kernel_launches() - launches0      # the library's own count of its launches in the region
    _barrier(world)
    w1 = time.time()
    clocks = sampler.window(w0, w1) if sampler else None
    ms = e0.elapsed_time(e1)
    committed = int(nc_all[warmup:n_total].sum().item())
    if ctx.device_status() != 0:
        raise RuntimeError("device status word is non-zero after the timed region")
    ms_max, committed_all = reduce_step_stats(ms, committed, device="cuda")
    value = committed_all / (ms_max * 1e-3)

    # ---- end to end: the step's activations come from pinned host memory, results go back to the host.  This leg runs
    #      directly behind the timed region so that both see the GPU in the same clock and power state.
    e2e_out = None
    # A short timed region (tens of milliseconds) ran on a GPU that had been idle and was not yet held down by its power
    # limit; the legs that follow it would each inherit the load of the one before.  They are to describe the same
    # kernels under the same conditions, so after a short region each leg starts from a GPU left idle for a moment, as
    # the timed region did; after a long one (power-limited already) they simply carry on.
    settle_s = 0.3 if ms_max < 100.0 else 0.0
    if with_e2e:
        time.sleep(settle_s)
        n_e2e = min(max(steps, steps_per_gen), 4 * steps_per_gen)   # at least one whole generation: the fill of the
                                                                    # two-stage pipeline is paid once per run, not per step
        # Double-buffered both ways: a copy stream uploads step t + 1's activations while step t computes, and the
        # host reads step t's counts and tokens while step t + 1 runs: the step does not depend on the host, so the
        # host stays one step behind, as dare_generate does.  The two count vectors are page-locked host tensors that
        # the step's last kernel writes directly (three small copies behind every step cost ~40 us of stream time,
        # one costs ~15); the block's tokens are copied to pinned memory right behind the step.
        # Every step still uploads its own inputs from pinned memory and every step's results are read on the host.
        bufs = [(torch.empty_like(pool[0][0]), torch.empty_like(pool[0][1])) for _ in range(2)]
        nc_h = [torch.zeros(B, dtype=torch.int32).pin_memory() for _ in range(2)]
        nr_h = [torch.zeros(B, dtype=torch.int32).pin_memory() for _ in range(2)]
        tok_blk_h = [torch.zeros(B, L, dtype=torch.int32).pin_memory() for _ in range(2)]
        read_back = [torch.cuda.Event(), torch.cuda.Event()]
        copy_stream = torch.cuda.Stream()
        uploaded = [torch.cuda.Event(), torch.cuda.Event()]
        consumed = [torch.cuda.Event(), torch.cuda.Event()]

        def upload(t):
            qh, xh = pool_h[t % NPOOL]
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(consumed[t & 1])          # the step that last read this buffer has finished
                bufs[t & 1][0].copy_(qh, non_blocking=True)
                bufs[t & 1][1].copy_(xh, non_blocking=True)
                uploaded[t & 1].record(copy_stream)

        # the upload alone (no compute beside it): what the host link delivers for one step's inputs
        up0, up1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(copy_stream):
            up0.record(copy_stream)
            for i in range(8):
                bufs[i & 1][0].copy_(pool_h[i % NPOOL][0], non_blocking=True)
                bufs[i & 1][1].copy_(pool_h[i % NPOOL][1], non_blocking=True)
            up1.record(copy_stream)
        torch.cuda.synchronize()
        upload_ms = up0.elapsed_time(up1) / 8
        _barrier(world)
        for ev_ in consumed:
            ev_.record(stream)
        e2e_tokens = 0
        ta = time.perf_counter()
        upload(0)
        for t in range(n_e2e):
            if t + 1 < n_e2e:
                upload(t + 1)
            stream.wait_event(uploaded[t & 1])
            step(t, bufs[t & 1][0], bufs[t & 1][1], nc_h[t & 1], nr_h[t & 1])
            consumed[t & 1].record(stream)
            g = t % steps_per_gen
            bs = wl.prompt_len + (g // steps_per_block) * L
            tok_blk_h[t & 1].copy_(tokens[:, bs:bs + L], non_blocking=True)
            read_back[t & 1].record(stream)
            if t >= 1:
                read_back[(t - 1) & 1].synchronize()
                e2e_tokens += int(nc_h[(t - 1) & 1].sum())
        read_back[(n_e2e - 1) & 1].synchronize()
        e2e_tokens += int(nc_h[(n_e2e - 1) & 1].sum())
        torch.cuda.synchronize()
        tb = time.perf_counter()
        e2e_s, e2e_n = reduce_step_stats(tb - ta, e2e_tokens, device="cuda")
        h2d = pool_h[0][0].numel() * 2 + pool_h[0][1].numel() * 2
        d2h = 4 * (B + B + B * L)
        e2e_out = {"value": e2e_n / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": d2h, "steps": n_e2e, "ms_per_step": e2e_s / n_e2e * 1e3,
                      "h2d_ms_per_step_alone": upload_ms, "h2d_GBps_alone": h2d / (upload_ms * 1e-3) / 1e9}

    # ---- host time of the public call alone (no device work waited for): what the step costs the calling thread
    n_host = 200
    torch.cuda.synchronize()
    tokens.copy_(tok0)
    th = time.perf_counter()
    for t in range(n_host):
        q, x = pool[t % NPOOL]
        dare.dare_denoise_block(ctx, q, k_pre, v_pre, plen_blocks[0], None, None, k_suf, v_suf, suffix_len,
                                attn_out, None, x, w, wl.mask_id, True, tokens, wl.prompt_len,
                                wl.mode, wl.threshold, wl.k, pred, conf, nc_all[0], nr, stream=stream)
    host_us = (time.perf_counter() - th) / n_host * 1e6       # (the queue never fills: 200 steps stay ahead of the GPU)
    torch.cuda.synchronize()

    # ---- instrumented pass: whole generations issued as the three entry points with events between them, to
    #      attribute time to each kernel.  The GPU is first given work to chew on so that the host runs ahead of it
    #      and no event interval contains host time.
    n_inst = max(1, min(steps // steps_per_gen, 4)) * steps_per_gen
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(n_inst)]
    nc_inst = torch.zeros(n_inst, B, dtype=torch.int32, device="cuda")
    nr_inst = torch.zeros(n_inst, B, dtype=torch.int32, device="cuda")
    rts = [torch.empty(B * L, dtype=torch.int32, device="cuda") for _ in range(2)]
    spacer = torch.empty(1 << 28, dtype=torch.float32, device="cuda")      # 1 GiB: each fill takes ~0.3 ms
    tokens.copy_(tok0)
    torch.cuda.synchronize()
    time.sleep(settle_s)
    i0 = time.time()
    for _ in range(6):
        spacer.fill_(0.0)
    for t in range(n_inst):
        g = t % steps_per_gen
        b = g // steps_per_block
        if g == 0:
            tokens.copy_(tok0)
        q, x = pool[t % NPOOL]
        bs = wl.prompt_len + b * L
        rt = rts[t & 1]
        rt.view(B, L).copy_(tokens[:, bs:bs + L])                 # the block's tokens as the LM head's row list
        ev[t][0].record(stream)
        dare.dare_attn_block(ctx, q, k_pre, v_pre, plen_blocks[b], None, None, k_suf, v_suf, suffix_len, attn_out,
                             None, stream=stream)
        ev[t][1].record(stream)
        dare.dare_lmhead_confidence(ctx, x, w, rt, wl.mask_id, True, pred, conf, stream=stream)
        ev[t][2].record(stream)
        dare.dare_unmask_select(ctx, tokens, bs, L, pred, conf, wl.mask_id, wl.mode, wl.threshold, wl.k,
                                nc_inst[t], nr_inst[t], stream=stream)
        ev[t][3].record(stream)
    torch.cuda.synchronize()
    i1 = time.time()
    del spacer
    # Clock samples for the pass: its own window, and, when it carried on directly behind a long timed region (no idle
    # in between), that region's samples as well: a pass of 0.2 s catches two or three samples, taken between launches,
    # and the GPU's state is the one the seconds of the same load before it left.
    inst_clocks = (sampler.window(w0 if settle_s == 0.0 else i0, i1)) if sampler else None
    lm_each = np.array([ev[t][1].elapsed_time(ev[t][2]) for t in range(n_inst)])
    attn_each = np.array([ev[t][0].elapsed_time(ev[t][1]) for t in range(n_inst)])
    lm_ms, attn_ms_events = float(lm_each.mean()), float(attn_each.mean())
    # The attention launch is short (tens of microseconds), and an interval between two events around a single launch
    # carries a few microseconds that are the events' own: the kernel is therefore timed as it runs in the step, in a
    # row of launches with nothing in between, per block (the prefix grows by L per block; K/V exceed L2, so every
    # launch reads them from HBM again).
    reps = 10
    attn_blocks = []
    for b in range(wl.n_blocks):
        ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        q = pool[b % NPOOL][0]
        dare.dare_attn_block(ctx, q, k_pre, v_pre, plen_blocks[b], None, None, k_suf, v_suf, suffix_len, attn_out, None,
                             stream=stream)
        ea.record(stream)
        for _ in range(reps):
            dare.dare_attn_block(ctx, q, k_pre, v_pre, plen_blocks[b], None, None, k_suf, v_suf, suffix_len, attn_out,
                                 None, stream=stream)
        eb.record(stream)
        torch.cuda.synchronize()
        attn_blocks.append(ea.elapsed_time(eb) / reps)
    attn_ms = float(np.mean(attn_blocks))
    sel_ms = float(np.mean([ev[t][2].elapsed_time(ev[t][3]) for t in range(n_inst)]))
    # rows that were still masked when each step began = committed in it + left after it (read back, not assumed)
    masked = (nc_inst + nr_inst).sum(dim=1).cpu().numpy().astype(np.float64)
    masked_avg = float(masked.mean())
    peaks = _peaks()
    inst_seconds = float(ev[0][0].elapsed_time(ev[n_inst - 1][3])) * 1e-3
    lm_flops = 2.0 * masked_avg * wl.hidden * wl.vocab          # algorithmic: masked rows only
    w_bytes = 2.0 * wl.vocab * wl.hidden
    # time the same launches would take at the roofline: per step the slower of the contraction at the tensor peak
    # and one pass over W at the measured HBM bandwidth (few masked rows => the W read bounds it)
    lm_peak, _ = _pick_peak(peaks, "bf16_tflops", "bf16_tflops_sustained", inst_seconds, inst_clocks)
    ideal_ms = float(np.mean(np.maximum(2.0 * masked * wl.hidden * wl.vocab / (lm_peak * 1e12),
                                        w_bytes / (peaks["hbm_gbs"] * 1e9)))) * 1e3
    by_rows = {}
    for m_rows in sorted(set(masked.astype(int).tolist())):
        sel = masked.astype(int) == m_rows
        by_rows[str(m_rows)] = round(float(lm_each[sel].mean()) * 1e3, 1)
    lm_roof = _tensor_roofline(
        "lmhead_greedy_kernel (+ row compaction and merge kernels)", lm_flops, lm_ms, peaks, inst_seconds, inst_clocks,
        DOMINANT_TRAFFIC_BYTES.get(wl.name) if wl.name == "llada8b" else None,
        {"masked_rows_avg": masked_avg, "frac_of_tensor_or_hbm_bound_time": ideal_ms / lm_ms,
         "us_by_masked_rows": by_rows, "instrumented_steps": n_inst})
    prefix_avg = float(np.mean([wl.prompt_len + ((t % steps_per_gen) // steps_per_block) * L + L for t in range(n_inst)]))
    kv_bytes = 2.0 * 2 * B * wl.n_kv_heads * wl.head_dim * (prefix_avg + wl.suffix_cap)
    qo_bytes = 2.0 * 2 * B * L * wl.n_q_heads * wl.head_dim
    attn_flops = 4.0 * B * L * wl.n_q_heads * wl.head_dim * (prefix_avg + wl.suffix_cap)
    attn_roof = _hbm_roofline(
        "attn_block_kernel" if L * (wl.n_q_heads // wl.n_kv_heads) < 96 else "attn_block_tc_kernel", kv_bytes + qo_bytes,
        attn_ms, peaks, inst_clocks, DOMINANT_TRAFFIC_BYTES.get(wl.name) if wl.name == "dualcache" else None,
        {"kv_bytes": kv_bytes, "kv_GBps": kv_bytes / (attn_ms * 1e-3) / 1e9,
         "kv_read_frac_hbm": kv_bytes / (attn_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
         "tflops": attn_flops / (attn_ms * 1e-3) / 1e12})
    breakdown = {"attn_ms": attn_ms, "attn_ms_single_launch_between_events": attn_ms_events,
                 "attn_ms_first_and_last_block": [attn_blocks[0], attn_blocks[-1]],
                 "lmhead_ms": lm_ms, "select_ms": sel_ms, "attn_GBps": attn_roof["achieved"],
                 "attn_frac_hbm": attn_roof["frac"], "attn_tflops": attn_roof["tflops"],
                 "lmhead_tflops": lm_roof["achieved"], "lmhead_frac": lm_roof["frac"],
                 "host_us_per_dare_denoise_block_call": host_us,
                 "note": "parts timed one entry point at a time; inside dare_denoise_block the attention runs beside the "
                         "LM head's GEMM (in the SMs its early finishers leave), so a step takes less than their sum"}

    # ---- the LM head's variants on all rows (sampling epilogue, log-probability head and its backward)
    if with_heads and wl.M % 8 == 0 and wl.vocab % 8 == 0:
        M_, V_ = wl.M, wl.vocab
        tg = I.uniform_int(1, I.TID_TOK, (M_,), 0, V_ - 1).cuda()
        gl = torch.ones(M_, dtype=torch.float32, device="cuda")
        lse_b = torch.empty(M_, dtype=torch.float32, device="cuda")
        lp_b = torch.empty(M_, dtype=torch.float32, device="cuda")
        w_t = dare.dare_transpose_bf16(ctx, w)
        bf = torch.bfloat16
        bwd = {"dz": torch.empty(M_, V_, dtype=bf, device="cuda"), "dzt": torch.empty(V_, M_, dtype=bf, device="cuda"),
               "d_hidden": torch.empty(M_, wl.hidden, dtype=bf, device="cuda"),
               "d_w": torch.empty(V_, wl.hidden, dtype=bf, device="cuda")}
        x0 = pool[0][1]
        cases = (("lmhead_all_rows_ms", lambda: dare.dare_lmhead_confidence(ctx, x0, w, None, wl.mask_id, True, pred, conf, stream=stream)),
                 ("lmhead_sample_all_rows_ms", lambda: dare.dare_lmhead_sample(ctx, x0, w, None, wl.mask_id, True, 1.0, 1, 1, pred, conf, stream=stream)),
                 ("lmhead_logprob_all_rows_ms", lambda: dare.dare_lmhead_logprob(ctx, x0, w, tg, wl.mask_id, True, logprob=lp_b, lse=lse_b, stream=stream)),
                 ("lmhead_logprob_backward_all_rows_ms", lambda: dare.dare_lmhead_logprob_backward(ctx, x0, w, w_t, tg, lse_b, gl, wl.mask_id, True, stream=stream, **bwd)))
        for name, fn in cases:
            for _ in range(2):
                fn()
            es = [torch.cuda.Event(enable_timing=True) for _ in range(9)]
            es[0].record(stream)
            for i in range(8):
                fn()
                es[i + 1].record(stream)
            torch.cuda.synchronize()
            breakdown[name] = float(np.median([es[i].elapsed_time(es[i + 1]) for i in range(8)]))
        del bwd, w_t

    out = {"value": value, "ms_per_step": ms_max / steps, "steps": steps, "clocks": clocks, "breakdown": breakdown,
           "lm_roofline": lm_roof, "attn_roofline": attn_roof,
           "gpu_launches": launches,
           "label": _workload_label(wl), "host": (w_h, (k_pre_h, v_pre_h, k_suf_h, v_suf_h))}

    if e2e_out is not None:
        out["e2e"] = e2e_out
    return out


def run_ours(args):
    from paper_2604_04215_b200 import binding as dare

    rank, world, local = _rank_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    sampler = None
    if rank == 0:
        sampler = ClockSampler(local)
        sampler.start()
        time.sleep(0.3)
    name = args.workload or "llada8b"
    wl = I.scaled(I.WORKLOADS[name], seed=rank)
    if args.batch:
        wl = I.scaled(wl, batch=args.batch)      # smaller copies of a workload (profiler captures)
    ctx = dare.Context(local)
    res = bench_step_workload(dare, ctx, wl, args.steps, args.warmup, rank, world, sampler, with_e2e=True,
                              with_heads=args.steps >= 64)
    w_h, caches_h = res.pop("host")
    dominant = "attn_roofline" if wl.name == "dualcache" else "lm_roofline"
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = time_oracle(wl, w_h, caches_h, budget_s=20.0)
    del w_h, caches_h

    # ---- the other workloads the metric is defined on, as short legs of the default single-GPU invocation
    extra = {}
    if args.workload is None and world == 1 and not args.no_extra_workloads:
        torch.cuda.empty_cache()
        for other in EXTRA_WORKLOADS:
            if other in I.MODEL_WORKLOADS:
                r = bench_loop_workload(dare, ctx, I.MODEL_WORKLOADS[other], steps=1, warmup=1, rank=rank, world=world,
                                        sampler=sampler, dual=False, temperature=0.0, with_e2e=False)
                extra[other] = {"value": r["value"], "unit": UNIT, "ms_per_step": r["ms_per_step"], "steps": r["steps"],
                                "config": r["label"], "clocks": r["clocks"], "roofline": r["roofline"]}
            else:
                owl = I.WORKLOADS[other]
                n = max(args.steps, 16) if args.steps < 256 else 256
                r = bench_step_workload(dare, ctx, owl, n, max(3, min(args.warmup, 8)), rank, world, sampler,
                                        with_e2e=False, with_heads=False)
                r.pop("host")
                dom = "attn_roofline" if other == "dualcache" else "lm_roofline"
                extra[other] = {"value": r["value"], "unit": UNIT, "ms_per_step": r["ms_per_step"], "steps": r["steps"],
                                "config": r["label"], "clocks": r["clocks"], "roofline": r[dom],
                                "breakdown": r["breakdown"]}
            torch.cuda.empty_cache()

    if rank == 0:
        out = {"metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
               "warmup": args.warmup, "ms_per_step": res["ms_per_step"], "higher_is_better": True,
               "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
               "config": {"workload": res["label"],
                          "l2": "inputs larger than L2 (the LM-head weight, 1.0 GB, and the KV cache are re-read every step)",
                          "parallelism": f"dp{world} (independent rollouts per GPU, no collective)"},
               "clocks": res["clocks"], "e2e": res["e2e"], "gpu_launches": res["gpu_launches"],
               "roofline": res[dominant], "breakdown": res["breakdown"], "cpu_baseline": cpu_baseline}
        if extra:
            out["workloads"] = extra
        print(json.dumps(out))
    if sampler:
        sampler.stop()
    ctx.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def _model_objects(dare, ctx, mw, wts_h, max_rows=None):
    layers = [{k: v.cuda() for k, v in l.items()} for l in wts_h["layers"]]
    return dare.Model(ctx, n_layers=mw.n_layers, hidden=mw.hidden, n_q_heads=mw.n_q_heads, n_kv_heads=mw.n_kv_heads,
                      head_dim=mw.head_dim, ffn=mw.ffn, vocab=mw.vocab, mask_id=mw.mask_id,
                      embedding=wts_h["embedding"].cuda(), layers=layers, lm_head=wts_h["lm_head"].cuda(),
                      max_positions=mw.row_len,
                      max_rows=max_rows or mw.batch * max(mw.prompt_len, mw.block_len),
                      max_batch=mw.batch, rms_eps=mw.rms_eps, rope_base=mw.rope_base)


def bench_loop_workload(dare, ctx, mw, steps, warmup, rank, world, sampler, dual, temperature, with_e2e):
    """The end-to-end loop workload: prefill + block-by-block denoising on the 4-layer stack (dare_generate).
    `steps` counts denoising steps; whole generations are timed (steps / steps-per-generation, at least one)."""
    from paper_2604_04215_b200.dist import reduce_step_stats
    wts_h = I.make_model_weights(mw)                                   # same weights on every rank
    mw_rank = I.ModelWorkload(**{**mw.__dict__, "seed": rank})         # its own prompts
    model = _model_objects(dare, ctx, mw, wts_h, max_rows=mw.batch * (mw.prompt_len + mw.gen_len) if dual else None)
    B, L, P, G = mw.batch, mw.block_len, mw.prompt_len, mw.gen_len
    loop = dare.dare_generate_dual if dual else dare.dare_generate
    if temperature > 0:              # sampled rollouts (temperature + Gumbel-max) instead of the argmax
        dare.dare_model_set_sampling(model, temperature, 1234 + rank, 0)
    tok0_h = I.fresh_model_tokens(mw_rank).pin_memory()
    tok0 = tok0_h.cuda()
    tok = tok0.clone()
    kc, vc = model.new_cache(B, mw.row_len)
    pred = torch.empty(B * L, dtype=torch.int32, device="cuda")
    conf = torch.empty(B * L, dtype=torch.float32, device="cuda")
    nr = torch.zeros(B, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()
    max_steps_per_gen = (G // L) * (L if mw.mode == I.SELECT_THRESHOLD else -(-L // mw.k))
    n_gen = max(1, int(round(steps / max_steps_per_gen)))
    n_warm = max(1, int(round(warmup / max_steps_per_gen))) if warmup > 0 else 0

    def generation(src):
        tok.copy_(src, non_blocking=True)
        return loop(model, tok, P, G, L, kc, vc, mw.mode, mw.threshold, mw.k, pred, conf, nr, stream=stream)

    for _ in range(n_warm):
        generation(tok0)
    _barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0 = time.time()
    launches0 = dare.dare_kernel_launches()
    e0.record(stream)
    steps_taken, committed = 0, 0
    for _ in range(n_gen):
        steps_taken += sum(generation(tok0))
        committed += B * G
    e1.record(stream)
    launches = dare.dare_kernel_launches() - launches0      # the library's own count (graph replays included)
    _barrier(world)
    w1 = time.time()
    clocks = sampler.window(w0, w1) if sampler else None
    ms = e0.elapsed_time(e1)
    if not bool((tok[:, P:] != mw.mask_id).all()) or ctx.device_status() != 0:
        raise RuntimeError("the loop left masks behind or the device status word is non-zero")
    ms_max, committed_all = reduce_step_stats(ms, committed, device="cuda")
    value = committed_all / (ms_max * 1e-3)
    if world > 1:
        # the one exchange of the sharded job: every rank gets all rollouts' final tokens (outside the timed region;
        # B * (P + G) int32 per rank)
        from paper_2604_04215_b200.dist import gather_tokens
        all_tok = gather_tokens(tok)
        if all_tok.shape[0] != world * B or not bool((all_tok[:, P:] != mw.mask_id).all()):
            raise RuntimeError("gathered tokens are incomplete")

    # ---- the projections of one layer at the step's row count, timed one by one for the roofline
    M = B * L
    D, F = mw.hidden, mw.ffn
    nq, nkv = mw.n_q_heads * mw.head_dim, mw.n_kv_heads * mw.head_dim
    lw = model._keep[1][0]
    a_d = I.normal_bf16(1, I.TID_X, (M, D)).cuda()
    a_f = I.normal_bf16(1, I.TID_Q, (M, F)).cuda()
    a_q = I.normal_bf16(1, I.TID_KBLK, (M, nq)).cuda()
    x_res = I.normal_bf16(1, I.TID_VBLK, (M, D)).cuda()
    o_qkv = torch.empty(M, nq + 2 * nkv, dtype=torch.bfloat16, device="cuda")
    o_act = torch.empty(M, F, dtype=torch.bfloat16, device="cuda")
    cases = [("qkv", lambda: dare.dare_linear(ctx, dare.LINEAR_STORE, a_d, lw["wqkv"], out=o_qkv), 2.0 * M * D * (nq + 2 * nkv)),
             ("attn_out", lambda: dare.dare_linear(ctx, dare.LINEAR_RESIDUAL, a_q, lw["wo"], residual=x_res, out=x_res), 2.0 * M * nq * D),
             ("gate_up_swiglu", lambda: dare.dare_linear(ctx, dare.LINEAR_SWIGLU, a_d, lw["wg"], w2=lw["wu"], out=o_act), 4.0 * M * D * F),
             ("down", lambda: dare.dare_linear(ctx, dare.LINEAR_RESIDUAL, a_f, lw["wd"], residual=x_res, out=x_res), 2.0 * M * F * D)]
    reps = 20
    per = {}
    tot_ms, tot_flop = 0.0, 0.0
    p0 = time.time()
    for name, fn, flop in cases:
        for _ in range(3):
            fn()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        evs[0].record(stream)
        for i in range(reps):
            # repeated on the same weight matrix: the smallest one (attn_out, 34 MB) can stay in L2 between
            # repeats, which flatters only that projection; the others exceed what L2 keeps
            fn()
            evs[i + 1].record(stream)
        torch.cuda.synchronize()
        t = float(np.mean([evs[i].elapsed_time(evs[i + 1]) for i in range(reps)]))
        per[name] = {"ms": t, "tflops": flop / (t * 1e-3) / 1e12}
        tot_ms += t
        tot_flop += flop
    p1 = time.time()
    peaks = _peaks()
    # the projections run inside the loop: the loop's own duration and clock record pick the denominator
    roofline = _tensor_roofline("gemm_pair_kernel (the four projections of one layer at M = B*L rows, timed one by one)",
                                tot_flop, tot_ms, peaks, ms_max * 1e-3, clocks, None,
                                {"per_projection": per, "clocks_while_timed_alone": sampler.window(p0, p1) if sampler else None})

    out = {"value": value, "ms_per_step": ms_max / max(steps_taken, 1), "steps": steps_taken, "clocks": clocks,
           "roofline": roofline, "gpu_launches": launches, "generations": n_gen, "ms_per_generation": ms_max / n_gen,
           "label": f"{mw.name}: {mw.n_layers} layers D{D} Hq{mw.n_q_heads}/Hkv{mw.n_kv_heads} d{mw.head_dim} F{F} "
                    f"V{mw.vocab} B{B} prompt{P}+gen{G} L{L} tau {mw.threshold}, "
                    + ("dual cache (whole-sequence refresh per block)" if dual else "prefix cache")
                    + (f", sampled head T={temperature}" if temperature > 0 else ""),
           "host": wts_h}

    # ---- end to end: prompts come from pinned host memory, the generated tokens go back to the host
    if with_e2e:
        out_h = torch.empty_like(tok0_h).pin_memory()
        _barrier(world)
        ta = time.perf_counter()
        e2e_tokens = 0
        for _ in range(n_gen):
            generation(tok0_h)
            out_h.copy_(tok, non_blocking=True)
            torch.cuda.synchronize()
            e2e_tokens += int((out_h[:, P:] != mw.mask_id).sum())
        tb = time.perf_counter()
        e2e_s, e2e_n = reduce_step_stats(tb - ta, e2e_tokens, device="cuda")
        out["e2e"] = {"value": e2e_n / e2e_s, "unit": UNIT, "h2d_bytes_per_step": tok0_h.numel() * 4 / max_steps_per_gen,
                      "d2h_bytes_per_step": out_h.numel() * 4 / max_steps_per_gen, "generations": n_gen}
    model.close()
    return out


def run_model(args):
    from paper_2604_04215_b200 import binding as dare

    rank, world, local = _rank_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    sampler = None
    if rank == 0:
        sampler = ClockSampler(local)
        sampler.start()
        time.sleep(0.3)
    mw = I.MODEL_WORKLOADS[args.workload]
    ctx = dare.Context(local)
    res = bench_loop_workload(dare, ctx, mw, args.steps, args.warmup, rank, world, sampler, args.cache == "dual",
                              args.temperature, with_e2e=True)
    wts_h = res.pop("host")
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = time_model_oracle(mw, wts_h, budget_s=20.0)
    if rank == 0:
        out = {"metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": res["steps"],
               "warmup": args.warmup, "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
               "config": {"workload": res["label"], "generations": res["generations"],
                          "ms_per_generation": res["ms_per_generation"],
                          "l2": "inputs larger than L2 (2.8 GB of weights are re-read every step)",
                          "parallelism": f"dp{world} (independent rollouts per GPU, no collective)"},
               "clocks": res["clocks"], "e2e": res["e2e"], "gpu_launches": res["gpu_launches"],
               "roofline": res["roofline"], "cpu_baseline": cpu_baseline}
        print(json.dumps(out))
    if sampler:
        sampler.stop()
    ctx.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def _blas_threads():
    """Threads of the BLAS pool behind numpy's matmul (where the oracle spends its time)."""
    try:
        from threadpoolctl import threadpool_info
        n = [p["num_threads"] for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return int(os.cpu_count() or 1)


def time_model_oracle(mw, wts_h, budget_s=20.0, max_steps=8):
    """Times the loop oracle, as it stands, on a bounded sample: denoising steps of ONE rollout right after its
    prefill (the prefill itself is not timed)."""
    from oracle import dare_model_oracle as MO
    f = lambda t: t.to(torch.float64).numpy()
    cfg = MO.ModelConfig(mw.n_layers, mw.hidden, mw.n_q_heads, mw.n_kv_heads, mw.head_dim, mw.ffn, mw.vocab,
                         mw.mask_id, mw.rms_eps, mw.rope_base)
    layers = [MO.LayerWeights(f(l["wqkv"]), f(l["wo"]), f(l["wg"]), f(l["wu"]), f(l["wd"])) for l in wts_h["layers"]]
    wts = MO.ModelWeights(f(wts_h["embedding"]), layers, f(wts_h["lm_head"]))
    one = I.ModelWorkload(**{**mw.__dict__, "batch": 1})
    tok = I.fresh_model_tokens(one).numpy()
    cache = MO.new_cache(cfg, 1, mw.row_len)
    MO.forward_block_cached(cfg, wts, tok, 0, mw.prompt_len, cache)
    committed, steps = 0, 0
    t0 = time.perf_counter()
    while steps < max_steps and (time.perf_counter() - t0 < budget_s or steps == 0):
        res = MO.denoise_step_cached(cfg, wts, tok, mw.prompt_len, mw.block_len, cache, mw.mode, mw.threshold, mw.k)
        committed += int(res["n_committed"].sum())
        tok = res["tokens"]
        steps += 1
    dt = time.perf_counter() - t0
    return {"value": committed / dt, "unit": UNIT, "cores": _blas_threads(), "kind": "oracle",
            "sample": f"{steps} denoising steps of 1 rollout out of {mw.batch} (all layers, full vocabulary) after its "
                      f"prefill, {dt:.1f} s; tokens/s of that single rollout, not scaled; fp64 numpy, its matrix "
                      f"products in numpy's BLAS pool (cores = that pool's threads)",
            "seconds_per_step_one_rollout": dt / steps}


def time_oracle(wl, w_h, caches_h, budget_s=20.0, max_steps=64):
    """Times the oracle, as it stands, on a bounded sample: ONE rollout (of the batch) per step."""
    from oracle import dare_oracle as O
    sub = I.scaled(wl, batch=1)
    k_pre, v_pre, k_suf, v_suf = [None if c is None else c[:1].to(torch.float64).numpy() for c in caches_h]
    w64 = w_h.to(torch.float64).numpy()
    tokens = I.fresh_tokens(sub).numpy()
    L = wl.block_len
    plen = np.array([wl.prompt_len])
    slen = np.array([wl.suffix_cap]) if wl.suffix_cap else None
    committed, steps = 0, 0
    t0 = time.perf_counter()
    while steps < max_steps and (time.perf_counter() - t0 < budget_s or steps == 0):
        q, _, _, x = I.make_step_activations(sub, steps % NPOOL, inplace_block=True)
        res = O.denoise_step(q.to(torch.float64).numpy(), k_pre, v_pre, plen, None, None, k_suf, v_suf, slen,
                             x.to(torch.float64).numpy(), w64, tokens, wl.prompt_len, L, wl.mask_id, wl.mode,
                             wl.threshold, wl.k)
        committed += int(res["n_committed"].sum())
        tokens = res["tokens"]
        if (tokens[:, wl.prompt_len:wl.prompt_len + L] != wl.mask_id).all():
            tokens = I.fresh_tokens(sub).numpy()
        steps += 1
    dt = time.perf_counter() - t0
    return {"value": committed / dt, "unit": UNIT, "cores": _blas_threads(), "kind": "oracle",
            "sample": f"{steps} steps of 1 rollout out of {wl.batch} (all heads, full vocabulary), {dt:.1f} s; "
                      f"tokens/s of that single rollout, not scaled; fp64 numpy, its matrix products in numpy's BLAS "
                      f"pool (cores = that pool's threads)",
            "seconds_per_step_one_rollout": dt / steps}


def run_reference(args):
    rank, world, _ = _rank_env()
    if world > 1:
        # the ranks only meet (the launch plumbing is the same as for our arm); rank 0 alone times the oracle
        import torch.distributed as dist
        dist.init_process_group("gloo")
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return
    name = args.workload or "llada8b"
    if name in I.MODEL_WORKLOADS:
        mw = I.MODEL_WORKLOADS[name]
        res = time_model_oracle(mw, I.make_model_weights(mw), budget_s=1e9, max_steps=max(1, min(args.steps, 8)))
        print(json.dumps({"impl": "reference", "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": args.gpus,
                          "steps": max(1, min(args.steps, 8)), "warmup": 0,
                          "ms_per_step": res["seconds_per_step_one_rollout"] * 1e3, "higher_is_better": True,
                          "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                          "config": {"workload": f"{mw.name} (bounded sample: one rollout, steps after its prefill)"},
                          "cpu_baseline": {"value": res["value"], "unit": UNIT, "cores": res["cores"], "kind": "oracle",
                                           "sample": res["sample"]},
                          "e2e": {"value": res["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                          "gpu_launches": 0}))
        return
    wl = I.WORKLOADS[name]
    w_h = I.normal_bf16(0, I.TID_W, (wl.vocab, wl.hidden), 0.02)
    caches = I.make_caches(I.scaled(wl, batch=1))
    n = max(1, min(args.steps, 16))
    nw = max(0, min(args.warmup, 2))
    if nw:
        time_oracle(wl, w_h, caches, budget_s=0.0, max_steps=nw)
    res = time_oracle(wl, w_h, caches, budget_s=1e9, max_steps=n)
    out = {"impl": "reference", "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": args.gpus,
           "steps": n, "warmup": nw, "ms_per_step": res["seconds_per_step_one_rollout"] * 1e3,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": f"{_workload_label(wl)} (bounded sample: one rollout of the batch per step)"},
           "cpu_baseline": {"value": res["value"], "unit": UNIT, "cores": res["cores"], "kind": "oracle",
                            "sample": res["sample"]},
           "e2e": {"value": res["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def spawn_ranks(n: int) -> int:
    """`--gpus N` without a launcher around it: start the N ranks here, one process per GPU on this node, through
    torch.distributed.run with the rendezvous on 127.0.0.1, and hand back its exit code.  The ranks re-enter this
    file with RANK / LOCAL_RANK / WORLD_SIZE set, exactly as under an external torchrun."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "WARN")
    return subprocess.run(cmd, env=env).returncode


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1536)
    ap.add_argument("--warmup", type=int, default=32)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=sorted(I.WORKLOADS) + sorted(I.MODEL_WORKLOADS),
                    help="default: llada8b as the line's value plus short legs of dream7b, dualcache and llada_loop")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra-workloads", action="store_true")
    ap.add_argument("--temperature", type=float, default=0.0,
                    help="loop workloads: > 0 samples the tokens (temperature + Gumbel-max) instead of the argmax")
    ap.add_argument("--cache", default="prefix", choices=["prefix", "dual"],
                    help="loop workloads: prefix cache (block-causal) or dual cache (bidirectional, refresh per block)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (0 = as defined)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus))
    if args.gpus != int(os.environ.get("WORLD_SIZE", "1")):
        raise SystemExit(f"--gpus {args.gpus} does not match WORLD_SIZE={os.environ.get('WORLD_SIZE')}")
    if args.impl == "reference":
        run_reference(args)
    elif args.workload in I.MODEL_WORKLOADS:
        run_model(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
