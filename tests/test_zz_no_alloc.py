"""st_decode_attention_static: the decode attention entry point that allocates nothing.

Some hosts of the library cannot allocate device memory when they call it (their own memory manager
owns the GPU, or they cannot take the device-wide stall of cudaMalloc), so this entry point keeps the
split-K workspace in an array built into the library. The GPU test drives a small batch through the
regular calls and, for two decode steps in a row, computes the same rows again through the
allocation-free entry point: it must reproduce st_reason_decode within the parity tolerance of the
other tests (in fact bit for bit, since the same kernels run on the same split plan), and the fp64
oracle's rows within the same tolerance. The page tables of this call are the caller's, so the test
also hands it a table with a page id outside the pool and expects an error status instead of a fault.

This file sorts last on purpose, so a run that stops at the first failure has run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import streaming_attention as osa
from paper_2510_17238_b200 import api, workloads

MAX_ABS_TOL = 1e-2
REL_L2_TOL = 5e-3


def test_static_entry_rejects_oversized_calls_with_a_message():
    # validation happens before any CUDA call, so this part needs no GPU
    call = lambda **kw: api.decode_attention_static(**{**dict(
        device=0, pool_source=1024, n_pages_source=4, pool_reason=1024, n_pages_reason=4, page_table_source=1024,
        table_stride_source=4, page_table_reason=1024, table_stride_reason=4, slots=[0], source_len=[1], reason_len=[1],
        q_rotated=1024, out=1024, n_q_heads=32, n_kv_heads=8, check=False), **kw})
    n = 65                                                  # 65 sequences x 8 kv heads > 512 pairs
    rc, msg = call(slots=[0] * n, source_len=[1] * n, reason_len=[1] * n)
    assert rc == api.ST_ERR_INVALID_ARG and "at most" in msg and "512" in msg
    rc, msg = call(slots=[0] * 113, source_len=[1] * 113, reason_len=[1] * 113, n_q_heads=8, n_kv_heads=1)
    assert rc == api.ST_ERR_INVALID_ARG and "112" in msg
    rc, msg = call(reason_len=[0])
    assert rc == api.ST_ERR_INVALID_ARG and "reason_len" in msg
    rc, msg = call(table_stride_source=1, source_len=[65])
    assert rc == api.ST_ERR_INVALID_ARG and "page table" in msg
    rc, msg = call(pool_source=None)
    assert rc == api.ST_ERR_INVALID_ARG
    rc, msg = call(n_pages_reason=0)
    assert rc == api.ST_ERR_INVALID_ARG and "n_pages" in msg
    # the status reader refuses a device on which no such call has been made (and bad ordinals)
    assert api.decode_static_status(63) == api.ST_ERR_INVALID_ARG
    assert api.decode_static_status(-1) == api.ST_ERR_INVALID_ARG


@pytest.mark.gpu
def test_static_entry_matches_reason_decode_two_calls_in_a_row():
    dev = torch.device("cuda", 0)
    Hq, Hkv, B = 32, 8, 3
    w = workloads.Workload(0, "no-alloc", Hq, Hkv, B)
    # three sequences with different source and reasoning lengths; long enough for several splits
    scheds = [workloads.SeqSchedule((700,), (130,), 0), workloads.SeqSchedule((65,), (3,), 0),
              workloads.SeqSchedule((1200,), (64,), 0)]
    ps = sum((s.S + 63) // 64 for s in scheds) + 2
    pr = sum((s.R + 63) // 64 for s in scheds) + 2
    cfg = api.make_config(n_q_heads=Hq, n_kv_heads=Hkv, max_batch=B, n_pages_source=ps, n_pages_reason=pr,
                          max_tokens_per_call=2048)
    pool_bytes = api.st_pool_bytes(cfg)
    pool = torch.zeros(pool_bytes + 1024, dtype=torch.uint8, device=dev)
    base = (pool.data_ptr() + 1023) // 1024 * 1024           # the library wants 1024-byte alignment
    cfg.pool_base, cfg.pool_bytes = base, pool_bytes
    ctx = api.Context(cfg)
    pool_source = base
    pool_reason = base + ps * Hkv * 32768                    # one layer: the reasoning pool follows the source pool

    tensors = [workloads.qkv(0, s, b, workload=w) for b, s in enumerate(scheds)]
    ids = list(range(B))
    # source: one chunk per sequence, closing unit 1
    cu = np.concatenate([[0], np.cumsum([s.S for s in scheds])]).astype(np.int32)
    cat = lambda i, sl: torch.cat([t[i][sl(s)] for t, s in zip(tensors, scheds)]).to(dev)
    q, k, v = (cat(i, lambda s: slice(0, s.S)) for i in range(3))
    out_src = torch.empty((int(cu[-1]), Hq, 128), dtype=torch.float32, device=dev)
    ctx.append_source_chunk(0, ids, cu, q, k, v, out_src, api.ST_END_OF_UNIT)
    # reasoning: all but the last two tokens of every sequence as one span
    cu_r = np.concatenate([[0], np.cumsum([s.R - 2 for s in scheds])]).astype(np.int32)
    q, k, v = (cat(i, lambda s: slice(s.S, s.S + s.R - 2)) for i in range(3))
    out_r = torch.empty((int(cu_r[-1]), Hq, 128), dtype=torch.float32, device=dev)
    ctx.reason_extend(0, ids, cu_r, None, q, k, v, out_r)

    stream = torch.cuda.current_stream().cuda_stream
    for step in (2, 1):                                      # the last two reasoning tokens, one decode step each
        rows = [s.S + s.R - step for s in scheds]
        q, k, v = (torch.stack([t[i][r] for t, r in zip(tensors, rows)]).to(dev) for i in range(3))
        want = torch.empty((B, Hq, 128), dtype=torch.float32, device=dev)
        ctx.reason_decode(0, ids, None, q, k, v, want, stream=stream)
        state = [ctx.seq_state(b) for b in ids]
        assert [st["reason_len"] for st in state] == [s.R - step + 1 for s in scheds]

        # inputs of the allocation-free call: rotated queries (oracle arithmetic, host), page tables, lengths
        pos = [s.R - step for s in scheds]
        q_rot = np.stack([osa.round_to_bf16(osa.rope(t[0][r].double().numpy()[None], [p], w.rope_theta))[0]
                          for t, r, p in zip(tensors, rows, pos)])
        q_rot = torch.from_numpy(q_rot).to(torch.bfloat16).to(dev)
        stride_s, stride_r = 32, 8
        tab_s = torch.zeros((B, stride_s), dtype=torch.int32)
        tab_r = torch.zeros((B, stride_r), dtype=torch.int32)
        for b in ids:
            pg = ctx.debug_page_table(b, 0)
            tab_s[b, : len(pg)] = torch.from_numpy(pg.copy())
            pg = ctx.debug_page_table(b, 1)
            tab_r[b, : len(pg)] = torch.from_numpy(pg.copy())
        tab_s, tab_r = tab_s.to(dev), tab_r.to(dev)
        got = torch.full((B, Hq, 128), float("nan"), dtype=torch.float32, device=dev)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        api.decode_attention_static(0, pool_source, ps, pool_reason, pr, tab_s, stride_s, tab_r, stride_r, ids,
                                    [scheds[b].S for b in ids], [st["reason_len"] for st in state], q_rot, got,
                                    Hq, Hkv, stream=stream)
        torch.cuda.synchronize()
        assert api.decode_static_status(0, stream) == api.ST_OK
        if step == 1:
            # (the very first call may make the driver load the library image that holds the workspace)
            assert torch.cuda.mem_get_info()[0] >= free_before - (1 << 20), "the call must not allocate device memory"
        g, r = got.double().cpu().numpy(), want.double().cpu().numpy()
        assert not np.isnan(g).any()
        assert np.abs(g - r).max() <= MAX_ABS_TOL and np.linalg.norm(g - r) / np.linalg.norm(r) <= REL_L2_TOL
        # and against the fp64 oracle on the raw inputs, row by row
        for b, s in enumerate(scheds):
            o = osa.build_schedule(s.src_unit_len, s.rsn_unit_len, s.final_len)
            qd, kd, vd = (t.double().numpy() for t in tensors[b])
            ref = osa.attention_rows(o, qd, kd, vd, [rows[b]], theta=w.rope_theta)[0]
            assert np.abs(g[b] - ref).max() <= MAX_ABS_TOL
            assert np.linalg.norm(g[b] - ref) / np.linalg.norm(ref) <= REL_L2_TOL

    # A page id outside the pool in the caller's table: the kernel must not build an address from it. The call
    # still returns ST_OK (it only queues work); the status reader reports the failed check, nothing faults, and
    # the rows of the sequence -- long enough to be split over several CTAs, so that only the merge kernel would
    # write them -- stay untouched. The next call with a sound table is correct again.
    bad_s = tab_s.clone()
    bad_s[0, 3] = ps + 1000
    got_bad = torch.full((B, Hq, 128), float("nan"), dtype=torch.float32, device=dev)
    args = (ids, [scheds[b].S for b in ids], [st["reason_len"] for st in state], q_rot)
    api.decode_attention_static(0, pool_source, ps, pool_reason, pr, bad_s, stride_s, tab_r, stride_r, *args, got_bad,
                                Hq, Hkv, stream=stream)
    assert api.decode_static_status(0, stream) == api.ST_ERR_DEVICE_CHECK
    assert torch.isnan(got_bad[0]).all(), "rows of the sequence with the bad page id must not be written"
    api.decode_attention_static(0, pool_source, ps, pool_reason, pr, tab_s, stride_s, tab_r, stride_r, *args, got_bad,
                                Hq, Hkv, stream=stream)
    assert api.decode_static_status(0, stream) == api.ST_OK
    assert torch.equal(got_bad, got)
    ctx.device_status()
    ctx.close()
