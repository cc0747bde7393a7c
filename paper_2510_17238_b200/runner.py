"""Host-side driver: walks streaming-unit schedules and issues the library calls.

Nothing here computes attention. A ``Plan`` is the list of C-ABI calls for a batch of sequences
in unit-synchronous order (Algorithm 1's two loops, flattened by the host):

    append unit 1 | append unit 2 | reason unit 1 | append unit 3 | reason unit 2 | ... | final depth

i.e. the prefill side runs ``lookahead`` units ahead of the reasoning side, which is the "input
ahead" branch of Algorithm 1: the reasoning calls then see only the slice of the source cache that
keeps N_EOS == N_EOT + 1. A ``DeviceBatch`` holds the packed, call-ordered tensors on the GPU, and
``run`` replays the plan on one or two CUDA streams.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

from . import api

APPEND, DECODE, EXTEND = 0, 1, 2


@dataclass
class Call:
    kind: int
    seq_ids: np.ndarray          # int32 [n]
    cu: np.ndarray               # int32 [n+1] packed row offsets inside the call
    vis: object                  # int32 [n] visible_units, or None (library default)
    flags: int
    row0: int                    # first packed row of the call on its side (source / reasoning)
    unit: int                    # 0-based unit, -1 for final depth


@dataclass
class Plan:
    calls: list
    src_rows: np.ndarray         # [rows] index into the flat [source ; reasoning] token list, call order
    rsn_rows: np.ndarray
    seq_offset: np.ndarray       # [B+1] start of every sequence in the flat token list
    max_call_tokens: int
    n_src_tokens: int
    n_rsn_tokens: int


def make_plan(scheds, mode: str = "decode", lookahead: int = 1, final_chunk: int = 128,
              explicit_units: bool = False, lag_units: int = 0) -> Plan:
    """mode 'decode': reasoning tokens one by one; 'extend': one span per reasoning unit.

    lag_units > 0: reasoning unit u asks for source unit min(u + lag_units, U) explicitly (lag 1 is the literal
    reading of Eq. 2's indicator); the prefill side must then run at least lag_units + 1 units ahead."""
    if lag_units > 0 and lookahead < lag_units + 1:
        raise ValueError("lookahead must be at least lag_units + 1")
    B = len(scheds)
    U = max(len(s.src_unit_len) for s in scheds)
    off = np.zeros(B + 1, np.int64)
    for b, s in enumerate(scheds):
        off[b + 1] = off[b] + s.S + s.R
    src_done = np.zeros(B, np.int64)
    rsn_done = np.zeros(B, np.int64)
    calls, src_rows, rsn_rows = [], [], []
    n_src = n_rsn = 0
    max_tokens = 1
    ragged = any(len(set(s.rsn_unit_len)) > 1 or s.rsn_unit_len != scheds[0].rsn_unit_len for s in scheds) or \
        any(len(s.src_unit_len) != U for s in scheds)
    explicit = explicit_units or ragged or lag_units > 0
    seen_unit = lambda b, u: min(u + 1 + lag_units, len(scheds[b].src_unit_len))

    def emit_append(u):
        nonlocal n_src, max_tokens
        ids = [b for b, s in enumerate(scheds) if u < len(s.src_unit_len)]
        if not ids:
            return
        cu = [0]
        for b in ids:
            n = scheds[b].src_unit_len[u]
            src_rows.append(off[b] + src_done[b] + np.arange(n))
            src_done[b] += n
            cu.append(cu[-1] + n)
        calls.append(Call(APPEND, np.asarray(ids, np.int32), np.asarray(cu, np.int32), None,
                          api.ST_END_OF_UNIT, n_src, u))
        n_src += cu[-1]
        max_tokens = max(max_tokens, cu[-1])

    def emit_reasoning(ids, counts, vis, flags, unit):
        """One extend call (counts tokens per sequence) or one decode call (all counts == 1)."""
        nonlocal n_rsn, max_tokens
        cu = [0]
        for b, m in zip(ids, counts):
            rsn_rows.append(off[b] + scheds[b].S + rsn_done[b] + np.arange(m))
            rsn_done[b] += m
            cu.append(cu[-1] + m)
        kind = DECODE if (mode == "decode" and all(m == 1 for m in counts)) else EXTEND
        calls.append(Call(kind, np.asarray(ids, np.int32), np.asarray(cu, np.int32),
                          None if vis is None else np.asarray(vis, np.int32), flags, n_rsn, unit))
        n_rsn += cu[-1]
        max_tokens = max(max_tokens, cu[-1])

    def emit_unit_reasoning(u):
        ids = [b for b, s in enumerate(scheds) if u < len(s.rsn_unit_len)]
        if not ids:
            return
        m = [scheds[b].rsn_unit_len[u] for b in ids]
        vis = [seen_unit(b, u) for b in ids] if explicit else None
        if mode == "extend":
            emit_reasoning(ids, m, vis, api.ST_END_OF_UNIT, u)
            return
        steps = max(m)
        uniform = len(set(m)) == 1
        for t in range(steps):
            act = [(b, mm) for b, mm in zip(ids, m) if mm > t]
            last = uniform and t == steps - 1
            emit_reasoning([b for b, _ in act], [1] * len(act), None if vis is None else [seen_unit(b, u) for b, _ in act],
                           api.ST_END_OF_UNIT if last else 0, u)
        if not uniform or steps == 0:
            # close the unit for every sequence with an empty span that only carries the flag
            emit_reasoning(ids, [0] * len(ids), vis, api.ST_END_OF_UNIT, u)

    for u in range(min(lookahead, U)):
        emit_append(u)
    for u in range(U):
        if u + lookahead < U:
            emit_append(u + lookahead)
        emit_unit_reasoning(u)
    # final-depth reasoning: the whole source is visible
    fin = [(b, s.final_len) for b, s in enumerate(scheds) if s.final_len > 0]
    if fin:
        done = {b: 0 for b, _ in fin}
        step = 1 if mode == "decode" else final_chunk
        while True:
            act = [(b, min(step, f - done[b])) for b, f in fin if done[b] < f]
            if not act:
                break
            emit_reasoning([b for b, _ in act], [c for _, c in act], [api.ST_VIS_ALL] * len(act), 0, -1)
            for b, c in act:
                done[b] += c

    cat = lambda xs: np.concatenate(xs).astype(np.int64) if xs else np.zeros(0, np.int64)
    return Plan(calls, cat(src_rows), cat(rsn_rows), off, int(max_tokens), int(n_src), int(n_rsn))


def pool_pages(scheds):
    ps = sum((s.S + 63) // 64 for s in scheds)
    pr = sum((s.R + 63) // 64 for s in scheds)
    return max(ps, 1), max(pr, 1)


def make_context(workload, scheds, plan: Plan, n_layers=None, device=0, extra_pages=0, flags=0,
                 position_mode=0, qk_norm=None) -> api.Context:
    ps, pr = pool_pages(scheds)
    cfg = api.make_config(
        n_layers=workload.n_layers if n_layers is None else n_layers,
        n_q_heads=workload.n_q_heads, n_kv_heads=workload.n_kv_heads, max_batch=len(scheds),
        n_pages_source=ps + extra_pages, n_pages_reason=pr + extra_pages,
        max_source_len=max(s.S for s in scheds), max_reason_len=max(max(s.R for s in scheds), 1),
        max_tokens_per_call=plan.max_call_tokens, device=device, rope_theta=workload.rope_theta, flags=flags,
        position_mode=position_mode, qk_norm=qk_norm)
    return api.Context(cfg)


class DeviceBatch:
    """Packed, call-ordered q/k/v (bf16) and out (fp32) tensors of one layer on the GPU."""

    def __init__(self, plan: Plan, flat_q, flat_k, flat_v, device="cuda", pinned_host=False, pageable_host=False):
        """flat_*: CPU bf16 tensors [sum(S_b + R_b), H, 128], sequences concatenated in batch order.
        pinned_host / pageable_host: keep inputs and outputs in host memory (page-locked or ordinary) for ST_IO_HOST."""
        self.plan = plan
        Hq = flat_q.shape[1]
        if pinned_host or pageable_host:
            # host-resident variant (end-to-end timing, tests of the host path): inputs and outputs live in host memory
            pin = (lambda t: t.pin_memory()) if pinned_host else (lambda t: t)
            pick = lambda t, idx: pin(t[torch.from_numpy(idx)].contiguous())
            mk_out = lambda n: pin(torch.empty((n, Hq, 128), dtype=torch.float32))
        else:
            dq, dk, dv = (t.to(device, non_blocking=False) for t in (flat_q, flat_k, flat_v))
            si = torch.from_numpy(plan.src_rows).to(device)
            ri = torch.from_numpy(plan.rsn_rows).to(device)
            idx_dev = {id(plan.src_rows): si, id(plan.rsn_rows): ri}
            src = {id(flat_q): dq, id(flat_k): dk, id(flat_v): dv}
            pick = lambda t, idx: src[id(t)].index_select(0, idx_dev[id(idx)])
            mk_out = lambda n: torch.full((n, Hq, 128), float("nan"), dtype=torch.float32, device=device)
        self.src = tuple(pick(t, plan.src_rows) for t in (flat_q, flat_k, flat_v))
        self.rsn = tuple(pick(t, plan.rsn_rows) for t in (flat_q, flat_k, flat_v))
        self.out_src = mk_out(max(plan.n_src_tokens, 1))
        self.out_rsn = mk_out(max(plan.n_rsn_tokens, 1))
        self.host = pinned_host or pageable_host

    def call_args(self, call: Call):
        t = self.src if call.kind == APPEND else self.rsn
        o = self.out_src if call.kind == APPEND else self.out_rsn
        r = call.row0
        q, k, v = t
        return (q.data_ptr() + r * q.stride(0) * 2, k.data_ptr() + r * k.stride(0) * 2,
                v.data_ptr() + r * v.stride(0) * 2, o.data_ptr() + r * o.stride(0) * 4)

    def outputs_flat(self):
        """Outputs scattered back to the flat [source ; reasoning] token order (CPU fp32)."""
        total = int(self.plan.seq_offset[-1])
        Hq = self.out_src.shape[1]
        flat = torch.full((total, Hq, 128), float("nan"), dtype=torch.float32)
        if self.plan.n_src_tokens:
            flat[torch.from_numpy(self.plan.src_rows)] = self.out_src[: self.plan.n_src_tokens].cpu()
        if self.plan.n_rsn_tokens:
            flat[torch.from_numpy(self.plan.rsn_rows)] = self.out_rsn[: self.plan.n_rsn_tokens].cpu()
        return flat


def flatten_inputs(index, scheds, layer=0, seed=0, workload=None, threads=None):
    """CPU bf16 tensors of a whole batch in the flat layout (sequence after sequence).

    Sequences are drawn independently (one generator key each), in parallel threads when asked."""
    import os
    from concurrent.futures import ThreadPoolExecutor
    from . import workloads
    draw = lambda bs: workloads.qkv(index, bs[1], bs[0], layer=layer, seed=seed, workload=workload)
    n_thr = min(len(scheds), len(os.sched_getaffinity(0))) if threads is None else threads
    if n_thr > 1:
        with ThreadPoolExecutor(max_workers=n_thr) as ex:
            parts = list(ex.map(draw, enumerate(scheds)))
    else:
        parts = [draw(bs) for bs in enumerate(scheds)]
    return tuple(torch.cat([p[i] for p in parts]) for i in range(3))


class CompiledPlan:
    """Pre-marshalled ctypes arguments of every call of a plan for one or more layers."""

    def __init__(self, ctx: api.Context, plan: Plan, batches, stream_src=None, stream_rsn=None,
                 extra_flags: int = 0):
        """batches: one DeviceBatch per layer. Streams: torch.cuda.Stream or None (current stream)."""
        self.ctx = ctx
        self.plan = plan
        self.keep = []
        self.items = []
        self.src_stream = stream_src if stream_src is not None else torch.cuda.current_stream()
        L = len(batches)
        s_src = stream_src.cuda_stream if stream_src is not None else torch.cuda.current_stream().cuda_stream
        s_rsn = stream_rsn.cuda_stream if stream_rsn is not None else s_src
        io_flag = api.ST_IO_HOST if batches[0].host else 0
        h = ctx.handle
        for call in plan.calls:
            ps, ks = api._i32(call.seq_ids)
            pc, kc = api._i32(call.cu)
            pv, kv = api._i32(call.vis)
            self.keep += [ks, kc, kv]
            n = len(call.seq_ids)
            flags = call.flags | extra_flags | io_flag
            for layer in range(L):
                q, k, v, o = batches[layer].call_args(call)
                if call.kind == APPEND:
                    self.items.append((api.lib.st_append_source_chunk, (h, layer, ps, pc, n, q, k, v, o, flags, s_src)))
                elif call.kind == DECODE:
                    self.items.append((api.lib.st_reason_decode, (h, layer, ps, n, pv, q, k, v, o, flags, s_rsn)))
                else:
                    self.items.append((api.lib.st_reason_extend, (h, layer, ps, pc, n, pv, q, k, v, o, flags, s_rsn)))

    def replay(self, kinds=None):
        """Issue every call (or only those whose function is in ``kinds``). Raises on the first error."""
        for fn, args in self.items:
            if kinds is not None and fn not in kinds:
                continue
            rc = fn(*args)
            if rc != 0:
                raise api.StError(rc, self.ctx.last_error())
        return len(self.items)
