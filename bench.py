#!/usr/bin/env python
"""Benchmark of the streaming dual-KV-cache attention hot path on B200.

One *step* is one pass of the whole hot path over one batch of the workload: st_reset, then every
source unit appended with its chunk-prefill attention (stream A) while the reasoning tokens are decoded
one by one against the visible source prefix and the reasoning cache (stream B), i.e. Algorithm 1's two
loops for all sequences of the batch, single attention layer.

  metric  reasoning-decode tokens/s per layer (chunk prefill running concurrently on a second stream)
  value   reasoning tokens of all ranks / max-over-ranks device time, inputs resident in HBM
  e2e     same pass with q/k/v/out in pinned HOST memory (ST_IO_HOST): every call copies its inputs
          host->device and its output device->host inside the timed region

The default workload is config index 2 (32 q / 8 kv heads, batch 32, 4096 source + 8192 reasoning tokens
per sequence, two streams): the smallest configuration whose KV working set (1.5 GiB) exceeds L2, so the
HBM roofline of the decode kernel means something. ``--config`` selects another one.

``--impl reference`` times the fp64 CPU oracle on a bounded sample of the same workload.
Multi-GPU (torchrun): every rank runs its own batch of sequences (weak scaling, no data-path collective).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

# DRAM bytes per algorithmic byte of st_k_decode, from an ncu capture of the small decode case (--profile-case decode:
# 274.0 MB moved on average for 268.6 MB of K/V, query and output): a full-size launch holds too much memory to
# capture. The profiler flushes the caches in front of every launch; in the real run a step finds up to ~50 MB of the
# step before it in L2 (the steps walk the caches in alternating directions), so the real traffic is a little lower.
DECODE_DRAM_PER_ALGORITHMIC_BYTE = 1.020
# The same ratio for st_k_attn_tc from the small prefill case (--profile-case prefill: 191.6 and 202.4 MB moved for 209.7
# and 220.2 MB of K/V, queries and output rows; below 1 because the rows a launch writes are still in L2 when it ends).
PREFILL_DRAM_PER_ALGORITHMIC_BYTE = 0.916

METRIC = "reasoning-decode tok/s per layer (chunk prefill concurrent on a second stream)"
UNIT = "tok/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload index 0..4")
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch (debugging)")
    ap.add_argument("--time-every", type=int, default=16,
                    help="bracket every N-th launch of the decode kernel with CUDA events in the timed region "
                         "(a bracketed launch cannot overlap its prologue with the kernel in front of it)")
    ap.add_argument("--spans", action="store_true",
                    help="side measurement: reasoning units and the final stage teacher-forced as spans "
                         "(st_reason_extend) on one stream; prints its own JSON line")
    ap.add_argument("--arrival", action="store_true",
                    help="side measurement: batch / interleaved / streaming routes under the paper's input arrival "
                         "process (150 words per minute); prints its own JSON line")
    ap.add_argument("--linear", action="store_true",
                    help="side measurement: the projection kernel on the attention-block shapes; prints its own JSON line")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-config", action="store_true",
                    help="skip the compact measurements of workloads 4 and 3 that the default run appends as per_config")
    ap.add_argument("--side-layers", type=int, default=4,
                    help="layers of workload 3's 36-layer stack that the per_config measurement runs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--oracle-rows", type=int, default=0, help="rows per oracle sample (0 = sized for ~15 s)")
    ap.add_argument("--profile-case", default=None, choices=["decode", "prefill"],
                    help="small stand-alone case for profiler captures (a few GB on the device, few launches)")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def gen_inputs(index, scheds, seed=0):
    """Flat CPU bf16 q/k/v of the batch; sequences are drawn in parallel threads (numpy releases the GIL)."""
    from concurrent.futures import ThreadPoolExecutor
    from paper_2510_17238_b200 import workloads
    with ThreadPoolExecutor(max_workers=min(len(scheds), len(os.sched_getaffinity(0)))) as ex:
        parts = list(ex.map(lambda bs: workloads.qkv(index, bs[1], bs[0], seed=seed), enumerate(scheds)))
    return tuple(torch.cat([p[i] for p in parts]) for i in range(3))


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        self.path = tempfile.NamedTemporaryFile(prefix="clocks_", suffix=".csv", delete=False).name
        self.proc = None
        self.dev = device_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.dev), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                p = [x.strip() for x in line.split(",")]
                if len(p) < 7:
                    continue
                try:
                    sm.append(float(p[0]))
                    mx.append(float(p[1]))
                except ValueError:
                    continue
                for name, val in zip(names, p[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def decode_algorithmic_bytes(plan, scheds, w):
    """Bytes the decode kernel must move, per decode call of one pass (in call order): every visible K/V byte of
    both caches once (4096 B per token: 8 kv heads x 128 channels x bf16 x {K, V}), the rotated query in, the
    fp32 row out."""
    from paper_2510_17238_b200 import runner
    kv_tok_bytes = 2 * w.n_kv_heads * w.head_dim * 2
    prefix = [np.concatenate([[0], np.cumsum(s.src_unit_len)]) for s in scheds]
    r_done = np.zeros(len(scheds), np.int64)
    per_call = []
    for c in plan.calls:
        if c.kind == runner.APPEND:
            continue
        counts = np.diff(c.cu)
        if c.kind == runner.DECODE:
            total = 0
            for b, u in zip(c.seq_ids, c.vis if c.vis is not None else [c.unit + 1] * len(c.seq_ids)):
                vis = scheds[b].S if u == -2 else int(prefix[b][u])
                total += (vis + int(r_done[b]) + 1) * kv_tok_bytes + w.n_q_heads * w.head_dim * (2 + 4)
            per_call.append(total)
        for b, m in zip(c.seq_ids, counts):
            r_done[b] += m
    return np.asarray(per_call, np.float64)


def prefill_algorithmic_flops(scheds, w):
    """QK^T and PV flops of every unmasked (query, key) pair of the chunk-prefill calls."""
    total = 0
    for s in scheds:
        p = 0
        for n in s.src_unit_len:
            total += 4 * w.n_q_heads * w.head_dim * (n * p + n * (n + 1) // 2)
            p += n
    return total


def span_algorithmic_flops(plan, scheds, w):
    """QK^T and PV flops of every unmasked (query, key) pair of the reasoning spans of one pass: a reasoning row
    at position r of a unit that sees `vis` source tokens has vis + r + 1 keys."""
    from paper_2510_17238_b200 import runner
    prefix = [np.concatenate([[0], np.cumsum(s.src_unit_len)]) for s in scheds]
    r_done = np.zeros(len(scheds), np.int64)
    total = 0
    for c in plan.calls:
        if c.kind == runner.APPEND:
            continue
        counts = np.diff(c.cu)
        for i, (b, m) in enumerate(zip(c.seq_ids, counts)):
            u = c.vis[i] if c.vis is not None else c.unit + 1
            vis = scheds[b].S if u == -2 else int(prefix[b][u])
            r0 = int(r_done[b])
            total += 4 * w.n_q_heads * w.head_dim * (int(m) * (vis + r0) + int(m) * (int(m) + 1) // 2)
            r_done[b] += m
    return total


def run_spans(args, w, scheds, local_rank):
    """Teacher-forced reasoning: every reasoning unit and the final stage as one st_reason_extend span per
    sequence, appends and spans in unit order on one stream. Reports reasoning tokens per second and the
    tensor-core attention kernel's rate over all its launches (chunk prefill and spans)."""
    from paper_2510_17238_b200 import runner
    plan = runner.make_plan(scheds, mode="extend", lookahead=1)
    ctx = runner.make_context(w, scheds, plan, device=local_rank)
    batch = runner.DeviceBatch(plan, *gen_inputs(args.config, scheds))
    L = w.n_layers
    compiled = runner.CompiledPlan(ctx, plan, [batch] * L)
    for _ in range(args.warmup):
        ctx.reset()
        compiled.replay()
    torch.cuda.synchronize()
    ctx.kernel_timing_enable(1)
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        ctx.reset()
        compiled.replay()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    n_tc, ms_tc = ctx.kernel_timing_read(1)
    ctx.kernel_timing_enable(0)
    ctx.device_status()
    peaks = measured_peaks()
    flops = (prefill_algorithmic_flops(scheds, w) + span_algorithmic_flops(plan, scheds, w)) * L * args.steps
    tflops = flops / (ms_tc / 1e3) / 1e12
    rsn_tokens = sum(s.R for s in scheds)
    print(json.dumps({
        "metric": "reasoning tok/s per layer, teacher-forced spans (st_reason_extend), one stream",
        "value": rsn_tokens * L * args.steps / (ms / 1e3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "dtype": "bf16",
        "data": "synthetic", "config": {"workload": w.name, "mode": "spans", "layers": L},
        "clocks": clocks,
        "roofline": {"bound": "tensor", "kernel": "st_k_attn_tc (chunk prefill + reasoning spans)", "achieved": tflops,
                     "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": tflops / peaks["bf16_tflops"],
                     "of": peaks["source"], "launches": n_tc, "total_ms": ms_tc, "traffic": None}}))
    ctx.close()


def run_arrival(args, local_rank):
    """Side measurement (--arrival): the three attention routes of Section 3.3 under the paper's input arrival process
    (150 words per minute). One sequence shaped like the paper's GSM-Symbolic samples (Table 4: about 5 input units,
    about 440 reasoning tokens), Qwen3-4B heads; every library call is timed on the device (CUDA events), and the
    timeline of each route is computed from those durations (paper_2510_17238_b200/arrival.py): attention only
    (x 36 layers), and with the paper's own full-model call times (Table 4: 0.041 s per prefill, 0.037 s per decode
    step) added, which is what its latency tables contain."""
    from paper_2510_17238_b200 import api, arrival, workloads
    n_units, n_src, n_rsn, final = 5, 20, 80, 40
    sched = workloads.SeqSchedule((n_src,) * n_units, (n_rsn,) * n_units, final)
    w = workloads.Workload(2, "arrival-qwen3-4b-b1-5x(20,80)+40", 32, 8, 1)
    dev = torch.device("cuda", local_rank)
    q, k, v = (t.to(dev) for t in workloads.qkv(2, sched, 0, workload=w))
    S, R = sched.S, sched.R
    stream = torch.cuda.current_stream().cuda_stream

    def timed_call(fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / 1e3

    def one_pass(batch_route):
        cfg = api.make_config(n_q_heads=32, n_kv_heads=8, max_batch=1, n_pages_source=S // 64 + 2, n_pages_reason=R // 64 + 2,
                              max_tokens_per_call=max(S, 128),
                              position_mode=api.ST_POS_CONCATENATED if batch_route else api.ST_POS_STREAMING)
        ctx = api.Context(cfg)
        out = torch.empty((max(S, 128), 32, 128), dtype=torch.float32, device=dev)
        pre, dec = [], []
        if batch_route:
            pre.append(timed_call(lambda: ctx.append_source_chunk(0, [0], [0, S], q[:S], k[:S], v[:S], out, api.ST_END_OF_UNIT, stream)))
        r = 0
        for u in range(n_units):
            if not batch_route:
                sl = slice(u * n_src, (u + 1) * n_src)
                pre.append(timed_call(lambda: ctx.append_source_chunk(0, [0], [0, n_src], q[sl], k[sl], v[sl], out, api.ST_END_OF_UNIT, stream)))
            for i in range(n_rsn):
                sl = slice(S + r, S + r + 1)
                vis = [api.ST_VIS_ALL] if batch_route else None
                flags = api.ST_END_OF_UNIT if (i == n_rsn - 1 and not batch_route) else 0
                dec.append(timed_call(lambda: ctx.reason_decode(0, [0], vis, q[sl], k[sl], v[sl], out, flags, stream)))
                r += 1
        for i in range(final):
            sl = slice(S + r, S + r + 1)
            dec.append(timed_call(lambda: ctx.reason_decode(0, [0], [api.ST_VIS_ALL], q[sl], k[sl], v[sl], out, 0, stream)))
            r += 1
        ctx.device_status()
        ctx.close()
        return pre, dec

    for _ in range(max(1, args.warmup)):
        one_pass(False)
    pre_s, dec_s = one_pass(False)
    pre_b, dec_b = one_pass(True)
    layers = 36
    routes = {}
    for label, extra_pre, extra_dec in (("attention_only_x36_layers", 0.0, 0.0), ("with_paper_full_model_call_times", 0.041, 0.037)):
        rows = {}
        for route in ("batch", "interleaved", "streaming"):
            pre, dec = (pre_b, dec_b) if route == "batch" else (pre_s, dec_s)
            tl = arrival.simulate(route, sched.src_unit_len, sched.rsn_unit_len, sched.final_len,
                                  lambda u, n: layers * pre[min(u, len(pre) - 1)] + extra_pre,
                                  lambda r: layers * dec[r] + extra_dec)
            rows[route] = {"ttft_tokens": tl.ttft_tokens, "first_reasoning_token_s": tl.first_token_s,
                           "input_end_s": tl.input_end_s, "delay_after_input_s": tl.delay_s}
        routes[label] = rows
    print(json.dumps({
        "metric": "time to the first reasoning token and delay after the end of the input, three attention routes, input at 150 words/min",
        "config": {"workload": w.name, "units": n_units, "source_tokens": S, "reasoning_tokens": R, "layers_assumed": layers,
                   "tokens_per_word": arrival.TOKENS_PER_WORD},
        "measured_call_us": {"prefill_unit_mean": 1e6 * statistics.mean(pre_s), "prefill_all_input": 1e6 * pre_b[0],
                             "decode_step_mean": 1e6 * statistics.mean(dec_s)},
        "routes": routes, "data": "synthetic",
        "note": "paper, Table 2 (GSM-Symbolic, Qwen3-4B): tokens before reasoning 94.74 (batch) -> 20.77 (streaming); "
                "Table 4: first-token latency 28.0 s -> 6.2 s; other hardware, context only"}))


def run_linear(args, local_rank):
    """Side measurement (--linear): the projection kernel st_linear on the shapes of the Qwen3-4B attention block of
    workload 2's appends (4096 tokens per call, hidden 2560, 32 q / 8 kv heads of 128): Q, K/V and output projection,
    against the measured bf16 burst peak; torch.matmul (cuBLAS) timed beside it for context."""
    from paper_2510_17238_b200 import api
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.current_stream().cuda_stream
    peaks = measured_peaks()
    rows = []
    for name, m, n, k in (("q_proj", 4096, 4096, 2560), ("kv_proj", 4096, 1024, 2560), ("o_proj", 4096, 2560, 4096)):
        x = torch.randn((m, k), device=dev).to(torch.bfloat16)
        w = (torch.randn((n, k), device=dev) / k ** 0.5).to(torch.bfloat16)
        y = torch.empty((m, n), dtype=torch.bfloat16, device=dev)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)          # larger than L2, written between repeats

        def timed(fn, reps=max(3, args.steps * 5)):
            for _ in range(max(3, args.warmup)):
                fn()
            total = 0.0
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for _ in range(reps):
                flush.zero_()
                e0.record()
                fn()
                e1.record()
                torch.cuda.synchronize()
                total += e0.elapsed_time(e1)
            return total / reps
        ms = timed(lambda: api.linear(local_rank, x, m, k, k, w, n, k, y, n, stream=stream))
        ms_lib = timed(lambda: torch.matmul(x, w.t()))
        assert api.linear_status(local_rank, stream) == api.ST_OK
        fl = 2.0 * m * n * k
        rows.append({"shape": name, "m": m, "n": n, "k": k, "us": ms * 1e3, "achieved": fl / ms / 1e9, "unit": "TFLOP/s",
                     "peak": peaks["bf16_tflops"], "frac": fl / ms / 1e9 / peaks["bf16_tflops"], "of": peaks["source"],
                     "cublas_us": ms_lib * 1e3, "cublas_tflops": fl / ms_lib / 1e9})
    print(json.dumps({"metric": "projection kernel st_linear, Qwen3-4B attention-block shapes at 4096 tokens per call",
                      "dtype": "bf16", "data": "synthetic", "l2": "256 MB written between repeats", "rows": rows}))


def oracle_sample(index, scheds, w, rows_per_sample, seed=0):
    """Times the fp64 oracle, as it stands, on seeded reasoning rows of sequence 0.

    Returns (tokens/s, description, seconds). The oracle rotates the whole sequence once; that time is
    charged pro rata (sampled rows / rows of the sequence)."""
    from oracle import streaming_attention as osa
    from paper_2510_17238_b200 import workloads
    s = scheds[0]
    q, k, v = workloads.qkv(index, s, 0, seed=seed)
    q, k, v = q.double().numpy(), k.double().numpy(), v.double().numpy()
    o = osa.build_schedule(s.src_unit_len, s.rsn_unit_len, s.final_len)
    rng = np.random.default_rng(1234)
    t0 = time.perf_counter()
    rot = osa.rotate_and_round(o, q, k, w.rope_theta)
    rot_s = time.perf_counter() - t0
    if rows_per_sample <= 0:
        t1 = time.perf_counter()
        osa.attention_rows(o, q, k, v, s.S + rng.integers(0, s.R, size=8), theta=w.rope_theta, rotated=rot)
        per_row = (time.perf_counter() - t1) / 8
        rows_per_sample = int(max(16, min(s.R, 12.0 / max(per_row, 1e-6))))
    rows = s.S + rng.integers(0, s.R, size=rows_per_sample)
    t2 = time.perf_counter()
    osa.attention_rows(o, q, k, v, rows, theta=w.rope_theta, rotated=rot)
    sec = (time.perf_counter() - t2) + rot_s * rows_per_sample / (s.S + s.R)
    desc = (f"{rows_per_sample} seeded reasoning rows of sequence 0 of {w.name}: all {w.n_q_heads} q heads, dense "
            f"masked softmax over {s.S + s.R} keys, fp64 numpy; the one-off rotation of the sequence charged pro rata")
    return rows_per_sample / sec, desc, sec


def max_over_ranks(ms, world, device):
    """Device time of the slowest rank (every rank times its own replica on its own GPU)."""
    if world <= 1:
        return float(ms)
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(tokens_per_rank, ms_max, steps, world):
    """Aggregate throughput of `world` replicas that each processed tokens_per_rank tokens per step."""
    return world * tokens_per_rank * steps / (ms_max / 1e3)


def config_dict(w, scheds, layers, world):
    """The `config` object of a JSON line: the same keys for the CUDA arm and the reference arm."""
    kv_bytes = sum(s.S + s.R for s in scheds) * 2 * w.n_kv_heads * w.head_dim * 2 * layers
    in_bytes = sum(s.S + s.R for s in scheds) * (w.n_q_heads + 2 * w.n_kv_heads) * w.head_dim * 2
    return {"workload": w.name, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads, "head_dim": 128,
            "batch_per_gpu": len(scheds), "source_tokens": scheds[0].S, "reasoning_tokens": scheds[0].R, "layers": layers,
            "page_size": 64, "streams": 2, "parallelism": f"replicas x{world} (sequences sharded, no collective)",
            "l2": ("KV working set %.2f GiB and %.1f GB of inputs against a 126 MB L2: every step streams more than L2 "
                   "holds; no flush" % (kv_bytes / 2**30, in_bytes / 1e9)) if kv_bytes > 2 * 126e6 else
                  ("KV working set %.1f MB fits in L2: launch-latency-bound configuration, no flush" % (kv_bytes / 1e6))}


def prefill_algorithmic_bytes(scheds, w):
    """Bytes the chunk-prefill attention kernel must move in one pass: per append call and sequence the K/V of the
    prefix and the chunk once (4096 B per token), the chunk's queries in (bf16) and its rows out (fp32)."""
    total = 0
    for s in scheds:
        p = 0
        for n in s.src_unit_len:
            total += (p + n) * 2 * w.n_kv_heads * w.head_dim * 2 + n * w.n_q_heads * w.head_dim * (2 + 4)
            p += n
    return total


def measure_prefill_alone(ctx, compiled, api, reps):
    """Chunk prefill with no decode stream beside it. Returns (bracketed launches, their summed ms, wall ms of one
    appends-only pass with nothing between the kernels): the first is the tensor-core kernel's own time (events around
    every launch), the second the time of the whole append chain (page-table update, K/V append, attention)."""
    append_only = (api.lib.st_append_source_chunk,)
    ctx.reset()
    compiled.replay(kinds=append_only)                       # warm-up
    torch.cuda.synchronize()
    ctx.kernel_timing_enable(True)
    for _ in range(reps):
        ctx.reset()
        compiled.replay(kinds=append_only)
    n, ms = ctx.kernel_timing_read(1)
    ctx.kernel_timing_enable(False)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stream = torch.cuda.current_stream()
    chain = []
    for _ in range(reps):
        ctx.reset()
        torch.cuda.synchronize()
        # the appends run on the plan's source stream: bracket them there
        compiled.src_stream.wait_stream(stream)
        e0.record(compiled.src_stream)
        compiled.replay(kinds=append_only)
        e1.record(compiled.src_stream)
        torch.cuda.synchronize()
        chain.append(e0.elapsed_time(e1))
    ctx.device_status()
    return n, ms / reps, min(chain)


def measure_side_config(index, args, local_rank, layers=None):
    """Compact measurement of another workload for the `per_config` list: one timed pass of the whole plan on two
    streams after three warm-up passes (decode tokens per second, decode kernel against HBM), and chunk prefill
    alone (tensor-core kernel against the bf16 peak). Workload 3 runs a stated subset of its 36 layers."""
    from paper_2510_17238_b200 import api, runner, workloads
    w = workloads.WORKLOADS[index]
    scheds = workloads.schedules(index)
    L = w.n_layers if layers is None else min(layers, w.n_layers)
    cfg_flags = api.ST_CFG_PRECISE_P if w.outlier_frac > 0 else 0   # as in the parity tests of that workload
    plan = runner.make_plan(scheds, mode="decode", lookahead=1)
    ctx = runner.make_context(w, scheds, plan, n_layers=L, device=local_rank, flags=cfg_flags)
    batch = runner.DeviceBatch(plan, *gen_inputs(index, scheds))
    s_src, s_rsn = torch.cuda.Stream(), torch.cuda.Stream()
    compiled = runner.CompiledPlan(ctx, plan, [batch] * L, s_src, s_rsn)
    for _ in range(3):
        ctx.reset()
        compiled.replay()
    torch.cuda.synchronize()
    ctx.device_status()
    period = max(1, args.time_every)
    ctx.kernel_timing_enable(period)
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(s_rsn)
    s_src.wait_event(e0)
    ctx.reset()
    compiled.replay()
    s_rsn.wait_stream(s_src)
    e1.record(s_rsn)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    n_dec, ms_dec = ctx.kernel_timing_read(0)
    ctx.kernel_timing_read(1)
    ctx.kernel_timing_enable(False)
    ctx.device_status()
    peaks = measured_peaks()
    dec_call_bytes = decode_algorithmic_bytes(plan, scheds, w)
    timed_idx = (np.arange(n_dec, dtype=np.int64) * period) % max(len(dec_call_bytes) * L, 1)
    dec_bytes_timed = float(dec_call_bytes[timed_idx // L].sum()) if n_dec else 0.0
    dec_gbs = dec_bytes_timed / (ms_dec / 1e3) / 1e9 if n_dec and ms_dec > 0 else 0.0
    n_pre, ms_pre, ms_chain = measure_prefill_alone(ctx, compiled, api, reps=2)
    flops = prefill_algorithmic_flops(scheds, w) * L
    tflops = flops / (ms_pre / 1e3) / 1e12 if ms_pre > 0 else 0.0
    out = {"workload": w.name, "layers_run": L, "layers_of_workload": w.n_layers, "two_term_probabilities": bool(cfg_flags),
           "warmup_passes": 3, "timed_passes": 1, "ms_per_pass": ms,
           "decode_tok_s": sum(s.R for s in scheds) * L / (ms / 1e3),
           "decode": {"kernel": "st_k_decode", "bound": "hbm", "achieved": dec_gbs, "unit": "GB/s", "peak": peaks["hbm_gbs"],
                      "frac": dec_gbs / peaks["hbm_gbs"], "avg_launch_us": 1e3 * ms_dec / max(n_dec, 1), "launches_timed": n_dec,
                      "algorithmic_bytes_per_launch": dec_bytes_timed / max(n_dec, 1)},
           "prefill": {"kernel": "st_k_attn_tc", "bound": "tensor", "achieved": tflops, "unit": "TFLOP/s",
                       "peak": peaks["bf16_tflops"], "frac": tflops / peaks["bf16_tflops"], "launches_per_pass": n_pre // 2,
                       "kernel_ms_per_pass": ms_pre, "append_chain_ms_per_pass": ms_chain,
                       "append_chain_tflops": flops / (ms_chain / 1e3) / 1e12,
                       "prefill_tok_s_chain": sum(s.S for s in scheds) * L / (ms_chain / 1e3),
                       # short units make chunk prefill memory-bound (G x tokens per unit below the ridge of ~250 flop/byte):
                       # the same launches against the copy bandwidth
                       "algorithmic_GBps": prefill_algorithmic_bytes(scheds, w) * L / (ms_pre / 1e3) / 1e9 if ms_pre > 0 else 0.0,
                       "frac_of_hbm": (prefill_algorithmic_bytes(scheds, w) * L / (ms_pre / 1e3) / 1e9 / peaks["hbm_gbs"]) if ms_pre > 0 else 0.0,
                       "mean_packed_rows_per_unit": float(np.mean([n * (w.n_q_heads // w.n_kv_heads) for s in scheds for n in s.src_unit_len]))},
           "of": peaks["source"], "clocks": clocks}
    ctx.close()
    del batch, compiled
    torch.cuda.empty_cache()
    return out


def run_reference(args, w, scheds, rank, world):
    """--impl reference: the oracle on the host cores, bounded sample per step."""
    if rank != 0:
        return
    cores = len(os.sched_getaffinity(0))
    vals = []
    for i in range(args.warmup + args.steps):
        tps, desc, sec = oracle_sample(args.config, scheds, w, args.oracle_rows or 64)
        if i >= args.warmup:
            vals.append((tps, sec))
    tps = statistics.mean(v[0] for v in vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * statistics.mean(v[1] for v in vals), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(w, scheds, w.n_layers, max(args.gpus, 1)),
        "cpu_baseline": {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def profile_case(kind):
    """A small case of the same kernels for profiler captures: 16 (decode) or 20 (prefill) sequences of config 2's
    head shape.

    decode : 2048 source tokens (one append) + 2040 reasoning tokens (one span) per sequence, then 8 decode
             steps at ~4090 keys per sequence: 268 MB of K/V per step (larger than L2), 8 st_k_decode launches.
    prefill: sixteen 128-token units appended one after the other (prefix 0 .. 1920): 16 st_k_attn_tc launches
             of 320 work items (two full waves on 148 SMs and 24 items that the kernel cuts in two by keys once they
             hold 20 pages); the last ones are the representative ones."""
    from paper_2510_17238_b200 import api, workloads
    w = workloads.WORKLOADS[2]
    B, S, R = (20 if kind == "prefill" else 16), 2048, 2048
    sched = workloads.SeqSchedule((S,), (R,), 0)
    dev = torch.device("cuda", 0)
    cfg = api.make_config(n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, max_batch=B, n_pages_source=B * S // 64,
                          n_pages_reason=B * R // 64, max_tokens_per_call=B * 2048)
    ctx = api.Context(cfg)
    parts = [workloads.qkv(2, sched, b) for b in range(B)]
    ids = list(range(B))
    stream = torch.cuda.current_stream().cuda_stream

    def packed(lo, hi):
        return tuple(torch.cat([p_[i][lo:hi] for p_ in parts]).to(dev) for i in range(3))

    def cu(n):
        return (np.arange(B + 1) * n).astype(np.int32)

    ctx.kernel_timing_enable(True)
    if kind == "decode":
        q, k, v = packed(0, S)
        out = torch.empty((B * S, w.n_q_heads, 128), dtype=torch.float32, device=dev)
        ctx.append_source_chunk(0, ids, cu(S), q, k, v, out, api.ST_END_OF_UNIT, stream)
        q, k, v = packed(S, S + R - 8)
        ctx.reason_extend(0, ids, cu(R - 8), None, q, k, v, out, 0, stream)
        o1 = torch.empty((B, w.n_q_heads, 128), dtype=torch.float32, device=dev)
        for r in range(R - 8, R):
            q, k, v = (torch.stack([p_[i][S + r] for p_ in parts]).to(dev) for i in range(3))
            ctx.reason_decode(0, ids, None, q, k, v, o1, 0, stream)
        torch.cuda.synchronize()
        n, ms = ctx.kernel_timing_read(0)
        bytes_per = B * (S + R - 4) * 4096
        print(json.dumps({"profile_case": "decode", "launches": n, "avg_us": 1e3 * ms / n,
                          "GBps": bytes_per / (ms / n / 1e3) / 1e9}))
    else:
        out = torch.empty((B * 128, w.n_q_heads, 128), dtype=torch.float32, device=dev)
        for u in range(S // 128):
            q, k, v = packed(u * 128, u * 128 + 128)
            ctx.append_source_chunk(0, ids, cu(128), q, k, v, out, api.ST_END_OF_UNIT, stream)
        torch.cuda.synchronize()
        n, ms = ctx.kernel_timing_read(1)
        flops = sum(4 * w.n_q_heads * 128 * (128 * p0 + 128 * 129 // 2) for p0 in range(0, S, 128)) * B
        print(json.dumps({"profile_case": "prefill", "launches": n, "total_ms": ms, "TFLOPs": flops / (ms / 1e3) / 1e12}))
    ctx.device_status()
    ctx.close()


def main():
    args = parse_args()
    if args.profile_case:
        profile_case(args.profile_case)
        return
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    from paper_2510_17238_b200 import workloads
    w = workloads.WORKLOADS[args.config]
    scheds = workloads.schedules(args.config, batch=args.batch)

    if args.impl == "reference":
        run_reference(args, w, scheds, rank, world)
        return

    import torch.distributed as dist
    from paper_2510_17238_b200 import api, runner

    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    if args.spans:
        if rank == 0:
            run_spans(args, w, scheds, local_rank)
        return
    if args.arrival:
        if rank == 0:
            run_arrival(args, local_rank)
        return
    if args.linear:
        if rank == 0:
            run_linear(args, local_rank)
        return

    plan = runner.make_plan(scheds, mode="decode", lookahead=1)
    ctx = runner.make_context(w, scheds, plan, device=local_rank)
    flat = gen_inputs(args.config, scheds, seed=rank)
    batch = runner.DeviceBatch(plan, *flat)
    s_src, s_rsn = torch.cuda.Stream(), torch.cuda.Stream()
    L = w.n_layers                                        # every layer is fed the same tensors (its own pools)
    compiled = runner.CompiledPlan(ctx, plan, [batch] * L, s_src, s_rsn)

    def one_pass(cp):
        ctx.reset()
        cp.replay()

    def timed(cp, steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()
        e0.record(s_rsn)
        s_src.wait_event(e0)
        for _ in range(steps):
            one_pass(cp)
        s_rsn.wait_stream(s_src)
        e1.record(s_rsn)
        torch.cuda.synchronize()
        return max_over_ranks(e0.elapsed_time(e1), world, "cuda")

    # ---- chunk prefill alone: the same appends with no decode stream beside them, so that the tensor-core
    # kernel's own rate is seen (in the concurrent pass its launches share the SMs with the decode kernel). It runs
    # first, a burst on a GPU that has not been under load for seconds, which is how the peak it is compared with
    # was measured (under the power cap the SM clock settles some 2-4 % lower during the long timed region below).
    solo_reps = 5
    solo_sampler = ClockSampler(local_rank)
    if rank == 0:
        solo_sampler.start()
    n_pre_solo, ms_pre_solo, ms_chain = measure_prefill_alone(ctx, compiled, api, solo_reps)
    solo_clocks = solo_sampler.stop() if rank == 0 else None

    for _ in range(args.warmup):
        one_pass(compiled)
    torch.cuda.synchronize()
    ctx.device_status()

    launches0 = ctx.launch_count()
    ctx.kernel_timing_enable(max(1, args.time_every))
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms = timed(compiled, args.steps)
    clocks = sampler.stop() if rank == 0 else None
    n_dec, ms_dec = ctx.kernel_timing_read(0)
    n_pre, ms_pre = ctx.kernel_timing_read(1)
    ctx.kernel_timing_enable(False)
    gpu_launches = ctx.launch_count() - launches0
    ctx.device_status()


    B = len(scheds)
    rsn_tokens = sum(s.R for s in scheds)
    src_tokens = sum(s.S for s in scheds)
    sec_per_step = ms / 1e3 / args.steps
    value = whole_job_tokens_per_s(rsn_tokens * L, ms, args.steps, world)   # per layer: token-layers per second

    peaks = measured_peaks()
    dec_call_bytes = decode_algorithmic_bytes(plan, scheds, w)
    dec_launches = len(dec_call_bytes)                    # decode launches of one layer in one pass
    pre_flops = prefill_algorithmic_flops(scheds, w)
    dec_avg_s = ms_dec / 1e3 / max(n_dec, 1)
    # The bracketed launches are every `period`-th decode launch of the timed region, counted from its first; launches
    # run call by call, layer by layer inside a call, pass after pass. Their own bytes go over their own time.
    period = max(1, args.time_every)
    timed_idx = (np.arange(n_dec, dtype=np.int64) * period) % max(dec_launches * L, 1)
    dec_bytes_timed = float(dec_call_bytes[timed_idx // L].sum()) if n_dec else 0.0
    dec_bytes_per_launch = dec_bytes_timed / max(n_dec, 1)
    dec_gbs = dec_bytes_timed / (ms_dec / 1e3) / 1e9 if n_dec else 0.0
    pre_flops *= L
    pre_tflops = pre_flops * args.steps / (ms_pre / 1e3) / 1e12 if n_pre and ms_pre > 0 else 0.0
    roofline = {"bound": "hbm", "kernel": "st_k_decode", "achieved": dec_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": dec_gbs / peaks["hbm_gbs"], "of": peaks["source"],
                "traffic": DECODE_DRAM_PER_ALGORITHMIC_BYTE * dec_bytes_per_launch,
                "traffic_how": "ncu dram__bytes_read.sum + dram__bytes_write.sum of the small decode case "
                               "(--profile-case decode), scaled by the K/V bytes one launch streams",
                "launches": dec_launches * L * args.steps, "launches_timed": n_dec, "avg_launch_us": dec_avg_s * 1e6,
                "algorithmic_bytes_per_launch": dec_bytes_per_launch,
                "timed": "every %d-th launch, its own bytes over its own time" % period,
                "frac_of_nominal_8TBs": dec_gbs / 8000.0}
    solo_tflops = pre_flops / (ms_pre_solo / 1e3) / 1e12 if n_pre_solo and ms_pre_solo > 0 else 0.0
    pre_bytes = prefill_algorithmic_bytes(scheds, w) * L
    roofline_prefill = {"bound": "tensor", "kernel": "st_k_attn_tc (chunk prefill)", "achieved": solo_tflops,
                        "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": solo_tflops / peaks["bf16_tflops"],
                        "of": peaks["source"] + " (burst: kernel timed alone, appends only, no decode stream)",
                        "frac_of_sustained": solo_tflops / peaks["bf16_tflops_sustained"],
                        "frac_of_nominal_2250": solo_tflops / 2250.0,
                        "launches": n_pre_solo, "total_ms_per_pass": ms_pre_solo, "clocks": solo_clocks,
                        "when": "before the warm-up passes of the timed region",
                        "algorithmic_flops_per_pass": pre_flops,
                        "traffic": PREFILL_DRAM_PER_ALGORITHMIC_BYTE * pre_bytes / max(n_pre_solo // solo_reps, 1)
                        if PREFILL_DRAM_PER_ALGORITHMIC_BYTE else None,
                        "traffic_how": "ncu dram__bytes_read.sum + dram__bytes_write.sum of the small prefill case "
                                       "(--profile-case prefill) per algorithmic byte (K/V of prefix and chunk once, queries "
                                       "in, rows out), times the average algorithmic bytes of a launch of this pass",
                        "algorithmic_bytes_per_launch": pre_bytes / max(n_pre_solo // solo_reps, 1),
                        "append_chain": {"achieved": pre_flops / (ms_chain / 1e3) / 1e12, "ms_per_pass": ms_chain,
                                         "what": "the same flops over the wall time of an appends-only pass with nothing "
                                                 "between the kernels: page-table update, K/V append and attention of "
                                                 "every call back to back",
                                         "prefill_tok_s": world * src_tokens * L / (ms_chain / 1e3)},
                        "concurrent_with_decode": {"achieved": pre_tflops, "launches": n_pre,
                                                   "total_ms_per_step": ms_pre / args.steps}}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": config_dict(w, scheds, L, world),
        "clocks": clocks, "gpu_launches": int(gpu_launches),
        "decode_kernel_tok_s": (world * rsn_tokens / (dec_call_bytes.sum() / (dec_gbs * 1e9))) if dec_gbs else None,
        "prefill_kernel_tok_s": world * src_tokens * L * args.steps / (ms_pre / 1e3) if ms_pre else None,
        "roofline": roofline, "roofline_prefill": roofline_prefill,
    }

    # ---- end to end: same pass with host buffers through the C ABI
    if not args.no_e2e:
        host_batch = runner.DeviceBatch(plan, *flat, pinned_host=True)
        cp_host = runner.CompiledPlan(ctx, plan, [host_batch] * L, s_src, s_rsn)
        one_pass(cp_host)
        e2e_steps = max(1, min(args.steps, 2))
        ms_h = timed(cp_host, e2e_steps)
        h2d = sum(t.numel() * 2 for t in host_batch.src + host_batch.rsn)
        d2h = (plan.n_src_tokens + plan.n_rsn_tokens) * w.n_q_heads * 128 * 4
        line["e2e"] = {"value": world * rsn_tokens * L / (ms_h / 1e3 / e2e_steps), "unit": UNIT,
                       "h2d_bytes_per_step": int(h2d) * L, "d2h_bytes_per_step": int(d2h) * L, "steps": e2e_steps,
                       "ms_per_step": ms_h / e2e_steps,
                       "how": "q/k/v/out in pinned host memory, ST_IO_HOST: an append copies its inputs in and its rows out "
                              "through device staging; a decode step (under 1 MiB) is read and written in place by its "
                              "kernels, every byte crossing the bus once inside the timed region"}
        del host_batch, cp_host

    # ---- the other two configurations whose rooflines mean something (N = 1 only: keeps the scaling runs short)
    if rank == 0 and world == 1 and args.config == 2 and not args.no_per_config:
        del batch, compiled
        ctx.close()
        torch.cuda.empty_cache()
        line["per_config"] = [measure_side_config(4, args, local_rank),
                              measure_side_config(3, args, local_rank, layers=args.side_layers)]

    # ---- the oracle on the host cores (rank 0, N = 1 only)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        tps, desc, sec = oracle_sample(args.config, scheds, w, args.oracle_rows)
        line["cpu_baseline"] = {"value": tps, "unit": UNIT, "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
                                "sample": desc, "seconds": sec}

    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
