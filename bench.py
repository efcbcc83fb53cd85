#!/usr/bin/env python
"""Benchmark of the rollout denoising step (attention -> LM head/confidence -> unmask selection).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A "step" is one pass of the whole hot path over one batch: dare_denoise_block on the LLaDA-8B-shaped
workload (batch 16 rollouts, prompt 512 + generation 256 in blocks of 32, top-k = 2 per step, so 16 steps
per block and 128 steps per generation; after 128 steps the token state is re-masked and the prefix length
returns to the prompt).  The metric is denoised (committed) tokens per second.

N > 1 (torchrun): every rank runs the same workload on its own rollouts (batch rows are independent, no
data-path collective); value = tokens of all ranks / max-over-ranks time ("weak" scaling).

`--impl reference` times the CPU oracle (oracle/dare_oracle.py) as it stands on a bounded sample of the same
workload, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
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
# dram__bytes_read.sum + dram__bytes_write.sum of one lmhead_partial_kernel launch, from the ncu capture
# summarised in profiles/lmhead_partial_kernel_llada8b.md (W, 1.036 GB, dominates: it leaves HBM once)
LMHEAD_TRAFFIC_BYTES = {"llada8b": 1.0669e9}


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
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
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"]}
        time.sleep(0.15)
        self.proc.terminate()       # the exact child started above
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        for ts, line in self.lines:
            if ts < t0 or ts > t1 + 0.1:
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


def run_ours(args):
    from paper_2604_04215_b200 import binding as dare
    from paper_2604_04215_b200.dist import reduce_step_stats

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    wl = I.scaled(I.WORKLOADS[args.workload], seed=rank)
    if args.batch:
        wl = I.scaled(wl, batch=args.batch)      # smaller copies of a workload (profiler captures)
    ctx = dare.Context(local)
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
        pool_h.append((q.pin_memory(), x.pin_memory()))
    pool = [(q.cuda(), x.cuda()) for q, x in pool_h]
    attn_out = torch.empty(B, L, wl.n_q_heads, wl.head_dim, dtype=torch.bfloat16, device="cuda")
    pred = torch.empty(B * L, dtype=torch.int32, device="cuda")
    conf = torch.empty(B * L, dtype=torch.float32, device="cuda")
    n_total = args.steps + args.warmup
    nc_all = torch.zeros(max(n_total, 1), B, dtype=torch.int32, device="cuda")
    nr = torch.zeros(B, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()

    def step(t, q, x, nc):
        g = t % steps_per_gen
        b = g // steps_per_block
        if g == 0:
            tokens.copy_(tok0)                                  # new generation: re-mask (one small copy)
        dare.dare_denoise_block(ctx, q, k_pre, v_pre, plen_blocks[b], None, None, k_suf, v_suf, suffix_len,
                                attn_out, None, x, w, wl.mask_id, True, tokens, wl.prompt_len + b * L,
                                wl.mode, wl.threshold, wl.k, pred, conf, nc, nr, stream=stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize()

    # ---- device-resident timed region
    for t in range(args.warmup):
        q, x = pool[t % NPOOL]
        step(t, q, x, nc_all[t])
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0 = time.time()
    e0.record(stream)
    for t in range(args.warmup, n_total):
        q, x = pool[t % NPOOL]
        step(t, q, x, nc_all[t])
    e1.record(stream)
    barrier()
    w1 = time.time()
    clocks = sampler.stop(w0, w1) if rank == 0 else None
    ms = e0.elapsed_time(e1)
    committed = int(nc_all[args.warmup:n_total].sum().item())
    if ctx.device_status() != 0:
        raise RuntimeError("device status word is non-zero after the timed region")
    ms_max, committed_all = reduce_step_stats(ms, committed, device="cuda")
    value = committed_all / (ms_max * 1e-3)

    # ---- instrumented pass: the same steps issued as the three entry points with events between them, to
    #      attribute time to the dominant kernel (LM head) for the roofline
    n_inst = min(args.steps, 2 * steps_per_gen)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(n_inst)]
    nc_inst = torch.zeros(max(n_inst, 1), B, dtype=torch.int32, device="cuda")
    nr_inst = torch.zeros(max(n_inst, 1), B, dtype=torch.int32, device="cuda")
    tokens.copy_(tok0)
    torch.cuda.synchronize()
    for t in range(n_inst):
        g = t % steps_per_gen
        b = g // steps_per_block
        if g == 0:
            tokens.copy_(tok0)
        q, x = pool[t % NPOOL]
        bs = wl.prompt_len + b * L
        ev[t][0].record(stream)
        dare.dare_attn_block(ctx, q, k_pre, v_pre, plen_blocks[b], None, None, k_suf, v_suf, suffix_len, attn_out,
                             None, stream=stream)
        ev[t][1].record(stream)
        rt = tokens[:, bs:bs + L].contiguous().view(-1)
        ev[t][1].record(stream)
        dare.dare_lmhead_confidence(ctx, x, w, rt, wl.mask_id, True, pred, conf, stream=stream)
        ev[t][2].record(stream)
        dare.dare_unmask_select(ctx, tokens, bs, L, pred, conf, wl.mask_id, wl.mode, wl.threshold, wl.k,
                                nc_inst[t], nr_inst[t], stream=stream)
        ev[t][3].record(stream)
    torch.cuda.synchronize()
    lm_ms = float(np.mean([ev[t][1].elapsed_time(ev[t][2]) for t in range(n_inst)]))
    attn_ms = float(np.mean([ev[t][0].elapsed_time(ev[t][1]) for t in range(n_inst)]))
    sel_ms = float(np.mean([ev[t][2].elapsed_time(ev[t][3]) for t in range(n_inst)]))
    # rows that were still masked when each step began = committed in it + left after it (read back, not assumed)
    masked = (nc_inst[:n_inst] + nr_inst[:n_inst]).sum(dim=1).cpu().numpy().astype(np.float64)
    masked_avg = float(masked.mean())
    executed_rows = float((np.ceil(masked / 128.0) * 128.0).mean())      # the GEMM works on 128-row tiles
    peaks = _peaks()
    lm_flops = 2.0 * masked_avg * wl.hidden * wl.vocab          # algorithmic: masked rows only
    achieved = lm_flops / (lm_ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops_sustained"]
    # time the same launches would take at the roofline: per step the slower of the contraction at the measured
    # tensor peak and one pass over W at the measured HBM bandwidth (few masked rows => the W read bounds it)
    w_bytes = 2.0 * wl.vocab * wl.hidden
    ideal_ms = float(np.mean(np.maximum(2.0 * masked * wl.hidden * wl.vocab / (peak * 1e12),
                                        w_bytes / (peaks["hbm_gbs"] * 1e9)))) * 1e3
    roofline = {"bound": "tensor", "kernel": "lmhead_partial_kernel (+ row compaction and merge kernels)",
                "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "traffic": LMHEAD_TRAFFIC_BYTES.get(wl.name), "peak_source": peaks["source"] + " sustained",
                "executed_tflops": 2.0 * executed_rows * wl.hidden * wl.vocab / (lm_ms * 1e-3) / 1e12,
                "ms_per_launch": lm_ms, "masked_rows_avg": masked_avg,
                "frac_of_tensor_or_hbm_bound_time": ideal_ms / lm_ms,
                "frac_of_nominal_2250": achieved / 2250.0}
    kv_bytes = 2.0 * 2 * B * wl.n_kv_heads * wl.head_dim * (
        float(np.mean([wl.prompt_len + ((t % steps_per_gen) // steps_per_block) * L + L for t in range(n_inst)])) + wl.suffix_cap)
    qo_bytes = 2.0 * 2 * B * L * wl.n_q_heads * wl.head_dim
    attn_gbs = (kv_bytes + qo_bytes) / (attn_ms * 1e-3) / 1e9
    # greedy against sampled head with every row masked (the sampling epilogue draws M * V Gumbel variates);
    # skipped in the few-step runs used under the profiler
    full_ms = {}
    bwd = {}
    if args.steps >= 64 and wl.M % 8 == 0 and wl.vocab % 8 == 0:
        # log-probability head and its backward on all rows (the likelihood / actor-update side of the same head)
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
        logprob_fn = lambda: dare.dare_lmhead_logprob(ctx, pool[0][1], w, tg, wl.mask_id, True, logprob=lp_b, lse=lse_b, stream=stream)
        backward_fn = lambda: dare.dare_lmhead_logprob_backward(ctx, pool[0][1], w, w_t, tg, lse_b, gl, wl.mask_id, True, stream=stream, **bwd)
    for name, fn in (() if args.steps < 64 else (("lmhead_all_rows_ms", lambda: dare.dare_lmhead_confidence(ctx, pool[0][1], w, None, wl.mask_id, True, pred, conf, stream=stream)),
                     ("lmhead_sample_all_rows_ms", lambda: dare.dare_lmhead_sample(ctx, pool[0][1], w, None, wl.mask_id, True, 1.0, 1, 1, pred, conf, stream=stream)))
                     + ((("lmhead_logprob_all_rows_ms", logprob_fn), ("lmhead_logprob_backward_all_rows_ms", backward_fn)) if bwd else ())):
        for _ in range(2):
            fn()
        es = [torch.cuda.Event(enable_timing=True) for _ in range(9)]
        es[0].record(stream)
        for i in range(8):
            fn()
            es[i + 1].record(stream)
        torch.cuda.synchronize()
        full_ms[name] = float(np.median([es[i].elapsed_time(es[i + 1]) for i in range(8)]))
    breakdown = {"attn_ms": attn_ms, "lmhead_ms": lm_ms, "select_ms": sel_ms, "attn_GBps": attn_gbs,
                 "attn_frac_hbm": attn_gbs / peaks["hbm_gbs"], **full_ms}

    # ---- end to end: the step's activations come from pinned host memory, results go back to the host
    n_e2e = min(args.steps, 4 * steps_per_gen)
    # Double-buffered both ways: a copy stream uploads step t + 1's activations while step t computes, and the host
    # reads step t's counts and tokens (copied to pinned memory right behind the step) while step t + 1 runs: the
    # step does not depend on the host, so the host stays one step behind, as dare_generate does.  Every step still
    # uploads its own inputs from pinned memory and every step's results are read on the host.
    bufs = [(torch.empty_like(pool[0][0]), torch.empty_like(pool[0][1])) for _ in range(2)]
    nc_h = [torch.zeros(B, dtype=torch.int32).pin_memory() for _ in range(2)]
    nr_h = [torch.zeros(B, dtype=torch.int32).pin_memory() for _ in range(2)]
    tok_blk_h = [torch.zeros(B, L, dtype=torch.int32).pin_memory() for _ in range(2)]
    nc_d = [torch.zeros(B, dtype=torch.int32, device="cuda") for _ in range(2)]
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

    barrier()
    for ev_ in consumed:
        ev_.record(stream)
    e2e_tokens = 0
    ta = time.perf_counter()
    upload(0)
    for t in range(n_e2e):
        if t + 1 < n_e2e:
            upload(t + 1)
        stream.wait_event(uploaded[t & 1])
        step(t, bufs[t & 1][0], bufs[t & 1][1], nc_d[t & 1])
        consumed[t & 1].record(stream)
        g = t % steps_per_gen
        bs = wl.prompt_len + (g // steps_per_block) * L
        nc_h[t & 1].copy_(nc_d[t & 1], non_blocking=True)
        nr_h[t & 1].copy_(nr, non_blocking=True)
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
    e2e = {"value": e2e_n / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "steps": n_e2e}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = time_oracle(wl, w_h, (k_pre_h, v_pre_h, k_suf_h, v_suf_h), budget_s=20.0)

    if rank == 0:
        # per step: attention, LM-head row compaction, LM-head GEMM, LM-head merge, selection
        attn_launches = 1   # (+ 1 combine launch when the attention plan splits KV: not in this workload)
        out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
               "warmup": args.warmup, "ms_per_step": ms_max / args.steps, "higher_is_better": True,
               "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
               "config": {"workload": f"{wl.name}: B{B} L{L} Hq{wl.n_q_heads}/Hkv{wl.n_kv_heads} d{wl.head_dim} "
                                      f"D{wl.hidden} V{wl.vocab} prompt{wl.prompt_len}+gen{wl.gen_len} "
                                      f"{'top-k ' + str(wl.k) if wl.mode == I.SELECT_TOPK else 'tau ' + str(wl.threshold)}",
                          "l2": "inputs larger than L2 (W 1.04 GB and KV cache 0.2 GB are re-read every step)",
                          "parallelism": f"dp{world} (independent rollouts per GPU, no collective)"},
               "clocks": clocks, "e2e": e2e, # per step: attention, row compaction, the LM-head GEMM in its two instantiations (single CTAs and CTA
               # pairs: the one whose mode does not apply to the step's row count returns at once), and the merge
               # kernel, which also does the selection for blocks of at most 32 positions
               "gpu_launches": (attn_launches + (4 if L <= 32 else 5)) * args.steps,
               "roofline": roofline, "breakdown": breakdown, "cpu_baseline": cpu_baseline}
        print(json.dumps(out))
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


def run_model(args):
    """The end-to-end loop workload: prefill + block-by-block denoising on the 4-layer stack (dare_generate).
    --steps counts denoising steps; whole generations are timed (steps / steps-per-generation, at least one)."""
    from paper_2604_04215_b200 import binding as dare
    from paper_2604_04215_b200.dist import reduce_step_stats

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    mw = I.MODEL_WORKLOADS[args.workload]
    wts_h = I.make_model_weights(mw)                                   # same weights on every rank
    mw_rank = I.ModelWorkload(**{**mw.__dict__, "seed": rank})         # its own prompts
    ctx = dare.Context(local)
    dual = args.cache == "dual"           # whole-sequence refresh before each block, steps see prefix + block + suffix
    model = _model_objects(dare, ctx, mw, wts_h, max_rows=mw.batch * (mw.prompt_len + mw.gen_len) if dual else None)
    B, L, P, G = mw.batch, mw.block_len, mw.prompt_len, mw.gen_len
    loop = dare.dare_generate_dual if dual else dare.dare_generate
    if args.temperature > 0:              # sampled rollouts (temperature + Gumbel-max) instead of the argmax
        dare.dare_model_set_sampling(model, args.temperature, 1234 + rank, 0)
    tok0_h = I.fresh_model_tokens(mw_rank).pin_memory()
    tok0 = tok0_h.cuda()
    tok = tok0.clone()
    kc, vc = model.new_cache(B, mw.row_len)
    pred = torch.empty(B * L, dtype=torch.int32, device="cuda")
    conf = torch.empty(B * L, dtype=torch.float32, device="cuda")
    nr = torch.zeros(B, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()
    max_steps_per_gen = (G // L) * (L if mw.mode == I.SELECT_THRESHOLD else -(-L // mw.k))
    n_gen = max(1, int(round(args.steps / max_steps_per_gen)))
    n_warm = max(1, int(round(args.warmup / max_steps_per_gen))) if args.warmup > 0 else 0

    def generation(src):
        tok.copy_(src, non_blocking=True)
        return loop(model, tok, P, G, L, kc, vc, mw.mode, mw.threshold, mw.k, pred, conf, nr, stream=stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(n_warm):
        generation(tok0)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0 = time.time()
    e0.record(stream)
    steps_taken, committed = 0, 0
    for _ in range(n_gen):
        steps_taken += sum(generation(tok0))
        committed += B * G
    e1.record(stream)
    barrier()
    w1 = time.time()
    clocks = sampler.stop(w0, w1) if rank == 0 else None
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
    peaks = _peaks()
    peak = peaks["bf16_tflops_sustained"]
    achieved = tot_flop / (tot_ms * 1e-3) / 1e12
    roofline = {"bound": "tensor", "kernel": "gemm_bf16_kernel (the four projections of one layer at M = B*L rows)",
                "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak, "traffic": None,
                "peak_source": peaks["source"] + " sustained", "per_projection": per,
                "frac_of_nominal_2250": achieved / 2250.0}

    # ---- end to end: prompts come from pinned host memory, the generated tokens go back to the host
    out_h = torch.empty_like(tok0_h).pin_memory()
    barrier()
    ta = time.perf_counter()
    e2e_tokens = 0
    for _ in range(n_gen):
        generation(tok0_h)
        out_h.copy_(tok, non_blocking=True)
        torch.cuda.synchronize()
        e2e_tokens += int((out_h[:, P:] != mw.mask_id).sum())
    tb = time.perf_counter()
    e2e_s, e2e_n = reduce_step_stats(tb - ta, e2e_tokens, device="cuda")
    e2e = {"value": e2e_n / e2e_s, "unit": UNIT, "h2d_bytes_per_step": tok0_h.numel() * 4 / max_steps_per_gen,
           "d2h_bytes_per_step": out_h.numel() * 4 / max_steps_per_gen, "generations": n_gen}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = time_model_oracle(mw, wts_h, budget_s=20.0)
    if rank == 0:
        per_fwd = 2 + 8 * mw.n_layers                   # embedding, final norm, 8 launches per layer
        # per generation: the prefill (prefix cache) or one refresh per block (dual cache), then per block its steps
        # plus the trailing one, each a forward + LM head (4 kernels: compaction, the GEMM in its two
        # instantiations, merge with the selection folded in for L <= 32, else a fifth kernel)
        launches = n_gen * ((G // L if dual else 1) * per_fwd + (steps_taken // n_gen + G // L) * (per_fwd + (4 if L <= 32 else 5)))
        out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps_taken, "warmup": args.warmup,
               "ms_per_step": ms_max / max(steps_taken, 1), "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
               "config": {"workload": f"{mw.name}: {mw.n_layers} layers D{D} Hq{mw.n_q_heads}/Hkv{mw.n_kv_heads} "
                                      f"d{mw.head_dim} F{F} V{mw.vocab} B{B} prompt{P}+gen{G} L{L} tau {mw.threshold}, "
                                      + ("dual cache (whole-sequence refresh per block)" if dual else "prefix cache")
                                      + (f", sampled head T={args.temperature}" if args.temperature > 0 else ""),
                          "generations": n_gen, "ms_per_generation": ms_max / n_gen,
                          "l2": "inputs larger than L2 (2.8 GB of weights are re-read every step)",
                          "parallelism": f"dp{world} (independent rollouts per GPU, no collective)"},
               "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline,
               "cpu_baseline": cpu_baseline}
        print(json.dumps(out))
    model.close()
    ctx.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


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
    return {"value": committed / dt, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
            "sample": f"{steps} denoising steps of 1 rollout out of {mw.batch} (all layers, full vocabulary) after its "
                      f"prefill, {dt:.1f} s; tokens/s of that single rollout, not scaled",
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
    return {"value": committed / dt, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
            "sample": f"{steps} steps of 1 rollout out of {wl.batch} (all heads, full vocabulary), {dt:.1f} s; "
                      f"tokens/s of that single rollout, not scaled",
            "seconds_per_step_one_rollout": dt / steps}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    if args.workload in I.MODEL_WORKLOADS:
        mw = I.MODEL_WORKLOADS[args.workload]
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
    wl = I.WORKLOADS[args.workload]
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
           "config": {"workload": f"{wl.name} (bounded sample: one rollout of the batch per step)"},
           "cpu_baseline": {"value": res["value"], "unit": UNIT, "cores": res["cores"], "kind": "oracle",
                            "sample": res["sample"]},
           "e2e": {"value": res["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1536)
    ap.add_argument("--warmup", type=int, default=32)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llada8b", choices=sorted(I.WORKLOADS) + sorted(I.MODEL_WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--temperature", type=float, default=0.0,
                    help="loop workloads: > 0 samples the tokens (temperature + Gumbel-max) instead of the argmax")
    ap.add_argument("--cache", default="prefix", choices=["prefix", "dual"],
                    help="loop workloads: prefix cache (block-causal) or dual cache (bidirectional, refresh per block)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (0 = as defined)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload in I.MODEL_WORKLOADS:
        run_model(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
