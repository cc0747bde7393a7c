"""CPU tests of the library's host side: exported symbols, schedule generator, state machine.

The library is loaded (no kernel is launched): contexts are created with ST_CFG_HOST_ONLY, which
runs validation, page planning and the per-sequence streaming state without device memory.
"""
import os
import re

import numpy as np
import pytest

from oracle import streaming_attention as osa
from paper_2510_17238_b200 import api, runner, workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def host_ctx(**kw):
    base = dict(n_layers=1, n_q_heads=16, n_kv_heads=8, max_batch=4, n_pages_source=8, n_pages_reason=8,
                max_tokens_per_call=1024, flags=api.ST_CFG_HOST_ONLY)
    base.update(kw)
    return api.Context(api.make_config(**base))


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "streaming_thinker.h")).read()
    declared = set(re.findall(r"ST_API\s+[\w\s\*]+?\b(st_\w+)\s*\(", text))
    assert len(declared) >= 16
    for name in declared:
        assert hasattr(api.lib, name), f"{name} is declared but not exported"
    assert declared == set(api.EXPORTED)


def test_pool_bytes_and_config_validation():
    cfg = api.make_config(n_layers=3, n_q_heads=32, n_kv_heads=8, max_batch=2, n_pages_source=10, n_pages_reason=6,
                          max_tokens_per_call=8)
    assert api.st_pool_bytes(cfg) == 3 * 16 * 8 * 32768
    for bad in (dict(n_q_heads=12), dict(n_q_heads=72), dict(n_layers=0), dict(max_batch=0), dict(rope_theta=0.0),
                dict(max_tokens_per_call=0)):
        kw = dict(n_layers=1, n_q_heads=16, n_kv_heads=8, max_batch=1, n_pages_source=1, n_pages_reason=1,
                  max_tokens_per_call=8, flags=api.ST_CFG_HOST_ONLY)
        kw.update(bad)
        assert api.st_pool_bytes(api.make_config(**kw)) == 0
        with pytest.raises(api.StError) as e:
            api.Context(api.make_config(**kw))
        assert e.value.code == api.ST_ERR_INVALID_ARG
    c = api.make_config(flags=api.ST_CFG_HOST_ONLY)
    c.head_dim = 64
    with pytest.raises(api.StError):
        api.Context(c)


def test_schedule_generator_reproduces_hand_written_examples():
    """The library's host-side schedule generator against the masks typed by hand from the paper's rules."""
    from test_oracle_pins import _worked_examples
    for b in _worked_examples():
        pos, vis, S, R = api.schedule_build(b["n"], b["m"], b["f"], 0)
        assert (S, R) == (sum(b["n"]), sum(b["m"]) + b["f"])
        assert pos[: S + R].tolist() == b["pos"] and vis[:R].tolist() == b["vis"]
        assert api.schedule_dense_mask(b["n"], b["m"], b["f"], 0).tolist() == b["rows"]


def test_kernel_timing_arguments():
    """The sampling period of the kernel timers: a negative period is refused, a host-only context brackets nothing."""
    ctx = host_ctx()
    with pytest.raises(api.StError) as e:
        ctx.kernel_timing_enable(-1)
    assert e.value.code == api.ST_ERR_INVALID_ARG
    ctx.kernel_timing_enable(4)
    assert ctx.kernel_timing_read(0) == (0, 0.0) and ctx.kernel_timing_read(1) == (0, 0.0)
    ctx.kernel_timing_enable(0)
    ctx.close()


@pytest.mark.parametrize("n,m,f,lag", [
    ([32] * 4, [16] * 4, 64, 0), ([2, 3, 1], [1, 2, 2], 2, 0), ([5], [0], 3, 0), ([1] * 6, [1] * 6, 0, 1),
    ([7, 0, 9], [0, 4, 0], 0, 0), ([4, 4], [4, 4], 4, 5),
])
def test_schedule_generator_matches_oracle_bit_exact(n, m, f, lag):
    sched = osa.build_schedule(n, m, f, lag_units=lag)
    pos, vis, S, R = api.schedule_build(n, m, f, lag)
    assert (S, R) == (sched.S, sched.R)
    assert pos.dtype == np.int32 and np.array_equal(pos, sched.pos_ids)
    assert np.array_equal(vis, sched.vis_len)
    mask = api.schedule_dense_mask(n, m, f, lag)
    assert mask.dtype == np.uint8 and np.array_equal(mask, osa.dense_mask(sched))


def test_schedule_generator_on_ragged_workloads():
    for idx, nseq in ((3, 3), (4, 1)):
        for s in workloads.schedules(idx, batch=nseq):
            sched = osa.build_schedule(s.src_unit_len, s.rsn_unit_len, s.final_len)
            pos, vis, S, R = api.schedule_build(s.src_unit_len, s.rsn_unit_len, s.final_len)
            assert np.array_equal(pos, sched.pos_ids) and np.array_equal(vis, sched.vis_len)
    s = workloads.schedules(3, batch=1)[0]
    small = workloads.SeqSchedule(s.src_unit_len[:6], s.rsn_unit_len[:6], 5)
    assert np.array_equal(api.schedule_dense_mask(small.src_unit_len, small.rsn_unit_len, 5),
                          osa.dense_mask(osa.build_schedule(small.src_unit_len, small.rsn_unit_len, 5)))
    assert api.lib.st_schedule_build(None, None, -1, 0, 0, None, None, None, None) == api.ST_ERR_INVALID_ARG


def test_workload_recipes():
    s4 = workloads.schedules(4)
    assert len(s4) == 16 and all(s.S == 32768 and s.R == 16384 for s in s4)
    assert all(8 <= n <= 256 for s in s4 for n in s.src_unit_len[:-1])
    s3 = workloads.schedules(3)
    assert len(s3) == 64 and all(len(s.src_unit_len) == 32 for s in s3)
    lens = np.array([n for s in s3 for n in s.src_unit_len])
    assert lens.min() >= 8 and lens.max() <= 256 and 40 < lens.mean() < 56
    assert [(s.S, s.R) for s in workloads.schedules(2)[:1]] == [(4096, 8192)]
    assert [(s.S, s.R) for s in workloads.schedules(1)[:1]] == [(1024, 1024)]
    assert [(s.S, s.R) for s in workloads.schedules(0)] == [(128, 128)]
    q, k, v = workloads.qkv(4, workloads.SeqSchedule((8,), (2,), 0), 0)
    assert q.shape == (10, 40, 128) and k.shape == (10, 8, 128)
    assert float(q.float().abs().max()) > 8.0          # outlier channels are present
    q2, _, _ = workloads.qkv(4, workloads.SeqSchedule((8,), (2,), 0), 0)
    assert (q == q2).all()


POSITION_MODE_NAMES = {api.ST_POS_STREAMING: "streaming", api.ST_POS_CONCATENATED: "concatenated",
                       api.ST_POS_UNIT_ALIGNED: "unit_aligned"}


def drive_plan_host_only(scheds, mode, n_layers=1, lookahead=1, position_mode=api.ST_POS_STREAMING):
    """Replays a plan on a host-only context and checks, call by call, that the positions and
    visibility the kernels would receive equal the oracle's schedule."""
    plan = runner.make_plan(scheds, mode=mode, lookahead=lookahead)
    w = workloads.WORKLOADS[0]
    ctx = runner.make_context(w, scheds, plan, n_layers=n_layers, flags=api.ST_CFG_HOST_ONLY, position_mode=position_mode)
    oracles = [osa.build_schedule(s.src_unit_len, s.rsn_unit_len, s.final_len,
                                  position_mode=POSITION_MODE_NAMES[position_mode]) for s in scheds]
    src_i = rsn_i = 0
    for call in plan.calls:
        for layer in range(n_layers):
            if call.kind == runner.APPEND:
                ctx.append_source_chunk(layer, call.seq_ids, call.cu, None, None, None, None, call.flags)
            elif call.kind == runner.DECODE:
                ctx.reason_decode(layer, call.seq_ids, call.vis, None, None, None, None, call.flags)
            else:
                ctx.reason_extend(layer, call.seq_ids, call.cu, call.vis, None, None, None, None, call.flags)
            pos, vs, vr = ctx.debug_last_call_meta()
            n = int(call.cu[-1])
            assert len(pos) == n
            rows = plan.src_rows[src_i:src_i + n] if call.kind == runner.APPEND else plan.rsn_rows[rsn_i:rsn_i + n]
            for j, flat in enumerate(rows):
                b = int(np.searchsorted(plan.seq_offset, flat, side="right") - 1)
                t = int(flat - plan.seq_offset[b])
                o = oracles[b]
                assert pos[j] == o.pos_ids[t]
                if t < o.S:
                    assert call.kind == runner.APPEND and vs[j] == t + 1 and vr[j] == 0
                else:
                    assert vs[j] == o.vis_len[t - o.S] and vr[j] == (t - o.S) + 1
        if call.kind == runner.APPEND:
            src_i += int(call.cu[-1])
        else:
            rsn_i += int(call.cu[-1])
    assert src_i == plan.n_src_tokens == sum(s.S for s in scheds)
    assert rsn_i == plan.n_rsn_tokens == sum(s.R for s in scheds)
    for b, s in enumerate(scheds):
        st = ctx.seq_state(b)
        assert st["source_len"] == s.S and st["reason_len"] == s.R
        assert st["n_eos"] == len(s.src_unit_len) and st["n_eot"] == len(s.rsn_unit_len)
    return ctx, plan


@pytest.mark.parametrize("mode", ["decode", "extend"])
def test_plan_positions_and_visibility_bit_exact_uniform(mode):
    drive_plan_host_only(workloads.schedules(0), mode)
    drive_plan_host_only([workloads.scaled_schedule(3, 70, 5, 9)] * 3, mode, n_layers=2, lookahead=2)


@pytest.mark.parametrize("mode", ["decode", "extend"])
def test_plan_positions_and_visibility_bit_exact_ragged(mode):
    full = workloads.schedules(3, batch=5)
    scheds = [workloads.SeqSchedule(s.src_unit_len[:4], tuple(min(x, 9) for x in s.rsn_unit_len[:4]), b)
              for b, s in enumerate(full)]
    scheds[1] = workloads.SeqSchedule(scheds[1].src_unit_len, (0, 3, 0, 2), 0)
    drive_plan_host_only(scheds, mode)


@pytest.mark.parametrize("mode", ["decode", "extend"])
def test_plan_positions_in_the_other_position_modes(mode):
    """Original RoPE ids (reasoning token t at T + t; the whole input is appended first, as in the batch setting the
    paper compares the encodings in) and the unit-aligned variant, call by call against the oracle's ids."""
    uniform = [workloads.scaled_schedule(3, 70, 5, 9)] * 2
    ragged = [workloads.SeqSchedule((30, 70, 64, 5), (3, 2, 4, 2), 3), workloads.SeqSchedule((64, 1, 129), (2, 0, 3), 0)]
    drive_plan_host_only(uniform, mode, lookahead=3, position_mode=api.ST_POS_CONCATENATED)
    drive_plan_host_only(ragged, mode, n_layers=2, lookahead=4, position_mode=api.ST_POS_CONCATENATED)
    drive_plan_host_only(uniform, mode, n_layers=2, position_mode=api.ST_POS_UNIT_ALIGNED)
    drive_plan_host_only(ragged, mode, lookahead=2, position_mode=api.ST_POS_UNIT_ALIGNED)
    with pytest.raises(api.StError):
        host_ctx(position_mode=7)


def test_algorithm1_counters_and_not_ready():
    ctx = host_ctx()
    ids = [0]
    # nothing appended: default visibility asks for unit 1 -> wait
    assert ctx.reason_decode(0, ids, None, None, None, None, None, check=False) == api.ST_ERR_NOT_READY
    assert ctx.seq_state(0)["reason_len"] == 0
    # an open (unfinished) source unit is not visible either
    ctx.append_source_chunk(0, ids, [0, 10], None, None, None, None, 0)
    assert ctx.seq_state(0) == {"source_len": 10, "reason_len": 0, "n_eos": 0, "n_eot": 0}
    assert ctx.reason_decode(0, ids, None, None, None, None, None, check=False) == api.ST_ERR_NOT_READY
    assert "not been appended" in ctx.last_error()
    # explicit unit 0 sees no source; ST_VIS_ALL sees the open unit too
    ctx.reason_decode(0, ids, [0], None, None, None, None)
    assert ctx.debug_last_call_meta()[1].tolist() == [0]
    ctx.reason_decode(0, ids, [api.ST_VIS_ALL], None, None, None, None)
    assert ctx.debug_last_call_meta()[1].tolist() == [10]
    # close the unit with a second chunk: N_EOS = 1, P_1 = 15
    ctx.append_source_chunk(0, ids, [0, 5], None, None, None, None, api.ST_END_OF_UNIT)
    ctx.append_source_chunk(0, ids, [0, 7], None, None, None, None, api.ST_END_OF_UNIT)   # unit 2, input runs ahead
    ctx.reason_decode(0, ids, None, None, None, None, None, api.ST_END_OF_UNIT)          # unit 1 -> sees P_1 only
    pos, vs, vr = ctx.debug_last_call_meta()
    assert (pos.tolist(), vs.tolist(), vr.tolist()) == ([2], [15], [3])
    ctx.reason_decode(0, ids, None, None, None, None, None)                              # unit 2 -> sees P_2
    assert ctx.debug_last_call_meta()[1].tolist() == [22]
    ctx.reason_decode(0, ids, [3], None, None, None, None, check=False)
    assert ctx.reason_decode(0, ids, [3], None, None, None, None, check=False) == api.ST_ERR_NOT_READY
    assert ctx.reason_decode(0, ids, [-7], None, None, None, None, check=False) == api.ST_ERR_INVALID_ARG
    assert ctx.seq_state(0) == {"source_len": 22, "reason_len": 4, "n_eos": 2, "n_eot": 1}


def test_invalid_arguments_change_nothing():
    ctx = host_ctx()
    before = ctx.pages_free()
    E = api.ST_ERR_INVALID_ARG
    assert ctx.append_source_chunk(0, [0, 0], [0, 1, 2], None, None, None, None, check=False) == E   # duplicate id
    assert ctx.append_source_chunk(0, [9], [0, 1], None, None, None, None, check=False) == E          # id range
    assert ctx.append_source_chunk(1, [0], [0, 1], None, None, None, None, check=False) == E          # layer range
    assert ctx.append_source_chunk(0, [0], [1, 2], None, None, None, None, check=False) == E          # cu[0] != 0
    assert ctx.append_source_chunk(0, [0, 1], [0, 5, 3], None, None, None, None, check=False) == E    # decreasing
    assert ctx.append_source_chunk(0, [0], [0, 4096], None, None, None, None, check=False) == E       # too many tokens
    assert ctx.append_source_chunk(0, [0], [0, 1], None, None, None, None, 64, check=False) == E      # unknown flag
    assert ctx.pages_free() == before and ctx.seq_state(0)["source_len"] == 0


def test_page_pool_exhaustion_and_reset():
    ctx = host_ctx(n_pages_source=3, n_pages_reason=1, max_batch=2)
    ctx.append_source_chunk(0, [0, 1], [0, 64, 129], None, None, None, None, api.ST_END_OF_UNIT)   # 1 + 2 pages
    assert ctx.pages_free() == (0, 1)
    assert ctx.append_source_chunk(0, [0], [0, 1], None, None, None, None, check=False) == api.ST_ERR_OOM_PAGES
    assert ctx.seq_state(0)["source_len"] == 64                                                  # unchanged
    ctx.append_source_chunk(0, [1], [0, 63], None, None, None, None)                               # fits in its page
    ctx.reason_extend(0, [0], [0, 64], None, None, None, None, None)
    assert ctx.reason_decode(0, [1], None, None, None, None, None, check=False) == api.ST_ERR_OOM_PAGES
    ctx.reset([0])
    assert ctx.pages_free() == (1, 1) and ctx.seq_state(0) == {"source_len": 0, "reason_len": 0, "n_eos": 0, "n_eot": 0}
    assert ctx.seq_state(1)["source_len"] == 128
    ctx.reason_decode(0, [1], None, None, None, None, None)
    ctx.reset()
    assert ctx.pages_free() == (3, 1)
    # per-sequence table bound
    ctx2 = host_ctx(n_pages_source=8, max_source_len=100)
    assert ctx2.append_source_chunk(0, [0], [0, 129], None, None, None, None, check=False) == api.ST_ERR_OOM_PAGES
    ctx2.append_source_chunk(0, [0], [0, 128], None, None, None, None)


def test_layer_protocol():
    ctx = host_ctx(n_layers=3)
    a = dict(seq_ids=[0, 1], cu_tokens=[0, 4, 9], q=None, k=None, v=None, out=None)
    assert ctx.append_source_chunk(1, **a, check=False) == api.ST_ERR_STATE            # must start at layer 0
    ctx.append_source_chunk(0, **a, flags=api.ST_END_OF_UNIT)
    assert ctx.seq_state(0)["source_len"] == 0                                         # not committed yet
    assert ctx.append_source_chunk(0, **a, check=False) == api.ST_ERR_STATE            # layer 0 twice
    assert ctx.append_source_chunk(2, **a, flags=api.ST_END_OF_UNIT, check=False) == api.ST_ERR_STATE
    assert ctx.append_source_chunk(1, [0, 1], [0, 4, 8], None, None, None, None, api.ST_END_OF_UNIT,
                                   check=False) == api.ST_ERR_STATE                    # different token counts
    assert ctx.append_source_chunk(1, **a, check=False) == api.ST_ERR_STATE            # different flags
    # the reasoning side has its own pending step and may interleave
    assert ctx.reason_decode(0, [0], None, None, None, None, None, check=False) == api.ST_ERR_NOT_READY
    ctx.append_source_chunk(1, **a, flags=api.ST_END_OF_UNIT)
    ctx.append_source_chunk(2, **a, flags=api.ST_END_OF_UNIT)
    assert ctx.seq_state(1) == {"source_len": 5, "reason_len": 0, "n_eos": 1, "n_eot": 0}
    ctx.reason_decode(0, [0], None, None, None, None, None)
    ctx.append_source_chunk(0, **a)                                                    # interleaved source step
    ctx.reason_decode(1, [0], None, None, None, None, None)
    ctx.reason_decode(2, [0], None, None, None, None, None)
    assert ctx.seq_state(0)["reason_len"] == 1


def test_a_failing_device_step_rolls_the_call_back():
    """A CUDA failure in the middle of a call (injected on the host: the n-th device step of the call reports
    ST_ERR_CUDA before it does anything) leaves the context as it was: pages back in the free list in their old
    order, lengths and counters unchanged, no step pending, so that the same call can simply be issued again."""
    steps_of_an_append = 4          # page-table update, staging, append launch, attention launch
    for fail_at in range(1, steps_of_an_append + 1):
        ctx = host_ctx(n_pages_source=6, n_pages_reason=4, max_batch=2)
        ctx.append_source_chunk(0, [0], [0, 70], None, None, None, None, api.ST_END_OF_UNIT)
        before = (ctx.pages_free(), ctx.seq_state(0), ctx.seq_state(1),
                  ctx.debug_page_table(0, 0).tolist(), ctx.debug_page_table(1, 0).tolist())
        ctx.debug_fail_after(fail_at)
        rc = ctx.append_source_chunk(0, [0, 1], [0, 100, 165], None, None, None, None, api.ST_END_OF_UNIT, check=False)
        assert rc == api.ST_ERR_CUDA and "injected" in ctx.last_error()
        after = (ctx.pages_free(), ctx.seq_state(0), ctx.seq_state(1),
                 ctx.debug_page_table(0, 0).tolist(), ctx.debug_page_table(1, 0).tolist())
        assert after == before
        # not pending: layer 0 is accepted again, takes the very same pages and commits
        ctx.append_source_chunk(0, [0, 1], [0, 100, 165], None, None, None, None, api.ST_END_OF_UNIT)
        assert ctx.seq_state(0) == {"source_len": 170, "reason_len": 0, "n_eos": 2, "n_eot": 0}
        assert ctx.debug_page_table(0, 0).tolist() == [0, 1, 2] and ctx.debug_page_table(1, 0).tolist() == [3, 4]
    # reasoning side (its first device step is the wait for the source append), and a multi-layer context: a
    # failure at a later layer keeps the step pending at that layer, so the layer can be issued again
    ctx = host_ctx(n_layers=2, n_pages_source=2, n_pages_reason=2, max_batch=1)
    for layer in (0, 1):
        ctx.append_source_chunk(layer, [0], [0, 10], None, None, None, None, api.ST_END_OF_UNIT)
    ctx.debug_fail_after(1)
    assert ctx.reason_decode(0, [0], None, None, None, None, None, check=False) == api.ST_ERR_CUDA
    assert ctx.pages_free() == (1, 2) and ctx.seq_state(0)["reason_len"] == 0
    ctx.reason_decode(0, [0], None, None, None, None, None)
    ctx.debug_fail_after(2)
    assert ctx.reason_decode(1, [0], None, None, None, None, None, check=False) == api.ST_ERR_CUDA
    assert ctx.seq_state(0)["reason_len"] == 0 and ctx.pages_free() == (1, 1)
    assert ctx.reason_decode(0, [0], None, None, None, None, None, check=False) == api.ST_ERR_STATE   # still pending
    ctx.reason_decode(1, [0], None, None, None, None, None)
    assert ctx.seq_state(0)["reason_len"] == 1


def test_packed_forward_positions_visibility_and_state():
    """st_forward_packed on a host-only context: the position ids and visibility of every packed row equal the
    oracle's schedule (with a lag and with the concatenated ids too), and the sequences end up in the state that
    streaming the same units would have left."""
    scheds = [workloads.SeqSchedule((30, 70, 64, 5), (3, 2, 4, 2), 3), workloads.SeqSchedule((64, 1, 129), (2, 0, 3), 0),
              workloads.SeqSchedule((), (), 0), workloads.SeqSchedule((7,), (0,), 5)]
    total = sum(s.S + s.R for s in scheds)
    for pm, lag in ((api.ST_POS_STREAMING, 0), (api.ST_POS_STREAMING, 1), (api.ST_POS_CONCATENATED, 0)):
        ctx = host_ctx(n_layers=2, n_pages_source=16, n_pages_reason=8, max_tokens_per_call=total, position_mode=pm)
        assert ctx.forward_packed(1, [0, 1, 2, 3], scheds, None, None, None, None, check=False) == api.ST_ERR_STATE
        ctx.forward_packed(0, [0, 1, 2, 3], scheds, None, None, None, None, lag_units=lag)
        assert ctx.seq_state(0)["source_len"] == 0                                   # not committed before the last layer
        assert ctx.reason_decode(0, [0], None, None, None, None, None, check=False) == api.ST_ERR_STATE
        assert ctx.forward_packed(1, [0, 1, 2, 3], scheds, None, None, None, None, lag_units=lag + 1, check=False) == api.ST_ERR_STATE
        ctx.forward_packed(1, [0, 1, 2, 3], scheds, None, None, None, None, lag_units=lag)
        pos, vs, vr = ctx.debug_last_call_meta()
        assert len(pos) == total
        row = 0
        for b, s in enumerate(scheds):
            o = osa.build_schedule(s.src_unit_len, s.rsn_unit_len, s.final_len, lag_units=lag,
                                   position_mode=POSITION_MODE_NAMES[pm])
            n = s.S + s.R
            assert pos[row:row + n].tolist() == o.pos_ids.tolist()
            assert vs[row:row + s.S].tolist() == list(range(1, s.S + 1)) and vr[row:row + s.S].tolist() == [0] * s.S
            assert vs[row + s.S:row + n].tolist() == o.vis_len.tolist()
            assert vr[row + s.S:row + n].tolist() == list(range(1, s.R + 1))
            st = ctx.seq_state(b)
            assert st == {"source_len": s.S, "reason_len": s.R, "n_eos": len(s.src_unit_len), "n_eot": len(s.src_unit_len)}
            row += n
        # the sequences can be decoded further, and a second packed pass needs them empty
        ctx.reason_decode(0, [0], [api.ST_VIS_ALL], None, None, None, None)
        assert ctx.forward_packed(0, [1], scheds[1:2], None, None, None, None, check=False) == api.ST_ERR_STATE
    ctx = host_ctx(n_pages_source=2, n_pages_reason=8, max_tokens_per_call=total)
    assert ctx.forward_packed(0, [0], scheds[:1], None, None, None, None, check=False) == api.ST_ERR_OOM_PAGES
    assert ctx.pages_free() == (2, 8)
    ctx = host_ctx(n_pages_source=16, n_pages_reason=8, max_tokens_per_call=total, position_mode=api.ST_POS_UNIT_ALIGNED)
    assert ctx.forward_packed(0, [0], scheds[:1], None, None, None, None, check=False) == api.ST_ERR_INVALID_ARG


def test_linear_rejects_bad_arguments():
    E = api.ST_ERR_INVALID_ARG
    ok = dict(device=0, x=1024, m=8, k=64, ldx=64, w=2048, n=16, ldw=64, y=4096, ldy=16, check=False)
    for bad in (dict(k=60), dict(n=12), dict(ldx=56), dict(ldw=68), dict(ldy=8), dict(x=1028), dict(m=0), dict(x=None)):
        assert api.linear(**{**ok, **bad})[0] == E
    assert api.cast_to_bf16(0, 1024, 2048, 12) == E
