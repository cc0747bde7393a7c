"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded inputs.

Tolerance (bf16 inputs, fp32 accumulation): max abs error <= 1e-2 and relative L2 error <= 5e-3 per
sequence; positions, visibility and stored values bit-exact; stored rotated keys bit-exact up to a
vanishing number of one-ulp rounding disagreements.
"""
import numpy as np
import pytest
import torch

from paper_2510_17238_b200 import api, runner, workloads

import parity_util as pu

pytestmark = pytest.mark.gpu


def small_workload(n_q_heads, n_kv_heads=8):
    return workloads.Workload(0, f"small-{n_q_heads}q", n_q_heads, n_kv_heads, 1)


def test_config0_decode_path_all_rows_and_cache():
    w = workloads.WORKLOADS[0]
    scheds = workloads.schedules(0)
    ctx, plan, batches, flats = pu.run_plan(w, scheds, 0, mode="decode")
    worst = pu.check_against_oracle(w, scheds, plan, batches[0], flats[0], what="cfg0 decode")
    assert pu.check_cache(ctx, w, scheds, plan, flats[0]) <= 2
    print("cfg0 decode worst (max_abs, rel_l2):", worst)


def test_config0_extend_path_and_reference_kernels():
    w = workloads.WORKLOADS[0]
    scheds = workloads.schedules(0)
    _, plan, batches, flats = pu.run_plan(w, scheds, 0, mode="extend")
    pu.check_against_oracle(w, scheds, plan, batches[0], flats[0], what="cfg0 extend")
    # the structurally different simple kernels must agree with the oracle too
    _, plan_r, batches_r, flats_r = pu.run_plan(w, scheds, 0, mode="decode", extra_flags=api.ST_REFERENCE_KERNELS)
    pu.check_against_oracle(w, scheds, plan_r, batches_r[0], flats_r[0], what="cfg0 reference kernels")


@pytest.mark.parametrize("mode", ["decode", "extend"])
def test_config1_batch8(mode):
    w = workloads.WORKLOADS[1]
    scheds = workloads.schedules(1)
    ctx, plan, batches, flats = pu.run_plan(w, scheds, 1, mode=mode)
    worst = pu.check_against_oracle(w, scheds, plan, batches[0], flats[0], n_random=96, full_seqs=(0,),
                                    what=f"cfg1 {mode}")
    assert pu.check_cache(ctx, w, scheds, plan, flats[0], seqs=(0, 7)) <= 4
    print("cfg1", mode, "worst (max_abs, rel_l2):", worst)


@pytest.mark.parametrize("hq", [8, 16, 32, 40, 64])
def test_ragged_edges(hq):
    """Unit lengths that straddle pages and tiles (1, 7, 8, 63, 64, 65, 255, 256), empty reasoning units,
    group sizes 1, 2, 4, 5 and 8, sequences of different unit counts."""
    w = small_workload(hq)
    scheds = [
        workloads.SeqSchedule((1, 7, 8, 63, 64, 65), (1, 0, 3, 2, 0, 5), 3),
        workloads.SeqSchedule((255, 256, 1), (4, 0, 1), 0),
        workloads.SeqSchedule((64, 64), (64, 1), 70),
        workloads.SeqSchedule((130,), (0,), 2),
    ]
    for mode in ("decode", "extend"):
        ctx, plan, batches, flats = pu.run_plan(w, scheds, 0, mode=mode, lookahead=2)
        pu.check_against_oracle(w, scheds, plan, batches[0], flats[0], what=f"ragged hq={hq} {mode}")
        assert pu.check_cache(ctx, w, scheds, plan, flats[0]) <= 2


@pytest.mark.parametrize("hq,variant", [(8, "plain"), (32, "plain"), (40, "plain"), (40, "two_term"), (16, "qk_norm"),
                                        (32, "two_streams")])
def test_key_split_of_long_items(hq, variant):
    """Work items of twenty and more cache pages in a launch that fills less than half of the SMs: the tensor-core
    kernel cuts each of them in two by keys and the part that finishes second merges. Twenty pages exactly and
    nineteen (not cut), a source prefix that ends inside a page (odd and even page counts in front of the reasoning
    pages), a second row pair with an empty second M-tile; group sizes 1, 2, 4 and 5; the one-term, the two-term and
    the normalising instantiation of the kernel."""
    w = small_workload(hq)
    scheds = [
        workloads.SeqSchedule((1217, 300, 70), (130, 257, 64), 40),     # 19 pages behind the first unit, then more
        workloads.SeqSchedule((1230, 50, 5), (0, 200, 3), 0),           # second unit: last row in page 19 (20 pages)
        workloads.SeqSchedule((1152, 63, 129), (1, 300, 2), 17),        # second unit: 19 pages, third: 21
    ]
    flags = api.ST_CFG_PRECISE_P if variant == "two_term" else 0
    norm = None
    if variant == "qk_norm":
        rng = np.random.default_rng(5)
        norm = (rng.uniform(0.5, 1.5, size=(1, 128)).astype(np.float32), rng.uniform(0.5, 1.5, size=(1, 128)).astype(np.float32), 1e-6)
    # (two_streams: the chunk prefills on one stream, the spans on another; each side has its own merge workspace)
    ctx, plan, batches, flats = pu.run_plan(w, scheds, 0, mode="extend", lookahead=1, cfg_flags=flags, qk_norm=norm,
                                            two_streams=variant == "two_streams")
    norm0 = None if norm is None else (norm[0][0], norm[1][0], norm[2])
    worst = pu.check_against_oracle(w, scheds, plan, batches[0], flats[0], n_random=160, what=f"key split hq={hq} {variant}",
                                    qk_norm=norm0)
    assert pu.check_cache(ctx, w, scheds, plan, flats[0], seqs=(1,), k_norm=None if norm is None else (norm[1][0], norm[2])) <= 2
    print("key split", hq, variant, "worst (max_abs, rel_l2):", worst)


def test_ragged_edges_with_sentinel_filled_pages():
    """The ragged schedules on a debug context (ST_CFG_DEBUG_CHECKS): every free page, and so the unwritten tail of
    every sequence's last page, holds 9.95e29 instead of zeros. A kernel that reads a key or value one token, one
    tile or one page too far would no longer multiply it by zero quietly: the rows would leave the tolerance.
    A second pass after st_reset runs on released pages, which are filled with the sentinel again."""
    w = small_workload(40)
    scheds = [
        workloads.SeqSchedule((1, 7, 8, 63, 64, 65), (1, 0, 3, 2, 0, 5), 3),
        workloads.SeqSchedule((255, 256, 1), (4, 0, 1), 0),
        workloads.SeqSchedule((64, 64), (64, 1), 70),
        workloads.SeqSchedule((130,), (0,), 2),
    ]
    for mode in ("decode", "extend"):
        ctx, plan, batches, flats = pu.run_plan(w, scheds, 0, mode=mode, lookahead=2, cfg_flags=api.ST_CFG_DEBUG_CHECKS)
        pu.check_against_oracle(w, scheds, plan, batches[0], flats[0], what=f"sentinel pages {mode}")
        # the sentinel really is there: the token after the last one of sequence 3's source cache (130 tokens, so 62
        # unwritten slots in its third page) reads back as the sentinel through the page table
        ctx.reset()
        batch2 = runner.DeviceBatch(plan, *flats[0])
        runner.CompiledPlan(ctx, plan, [batch2]).replay()
        torch.cuda.synchronize()
        ctx.device_status()
        pu.check_against_oracle(w, scheds, plan, batch2, flats[0], what=f"sentinel pages after reset {mode}")
        ctx.close()


@pytest.mark.parametrize("hq", [8, 32, 40])
def test_two_term_probabilities_on_outlier_channels(hq):
    """ST_CFG_PRECISE_P (probabilities as two bf16 terms in chunk prefill and spans) on ragged schedules whose
    Q, K and V carry 2 % of their (head, channel) pairs multiplied by 8: unit lengths straddle pages and tiles,
    sequences end on odd page counts, and every row must stay within the tolerance."""
    w = workloads.Workload(0, f"outliers-{hq}q", hq, 8, 1, outlier_frac=0.02, outlier_mult=8.0)
    scheds = [
        workloads.SeqSchedule((1, 7, 8, 63, 64, 65), (1, 0, 3, 2, 0, 5), 3),
        workloads.SeqSchedule((255, 256, 1), (4, 0, 1), 0),
        workloads.SeqSchedule((300, 212), (64, 1), 70),
        workloads.SeqSchedule((130,), (0,), 2),
    ]
    for mode in ("decode", "extend"):
        ctx, plan, batches, flats = pu.run_plan(w, scheds, 0, mode=mode, lookahead=2, cfg_flags=api.ST_CFG_PRECISE_P)
        worst = pu.check_against_oracle(w, scheds, plan, batches[0], flats[0], what=f"two-term P hq={hq} {mode}")
        assert worst[0] <= 5e-3, f"two-term probabilities should leave a wide margin, got {worst}"
        assert pu.check_cache(ctx, w, scheds, plan, flats[0]) <= 2
        ctx.close()


def test_eq2_literal_lag_and_input_far_ahead():
    """Two visibility variants on the GPU. (1) Eq. 2 read literally lets reasoning unit u see source unit u + 1:
    every reasoning call names visible_units = N_EOT + 2 and the rows must equal the oracle's lag_units = 1
    schedule. (2) Algorithm 1's "input ahead" branch: the prefill side runs three units ahead of the reasoning
    side on workload 1, and the default visibility must still slice the source cache back to unit N_EOT + 1."""
    w = small_workload(32)
    scheds = [workloads.SeqSchedule((30, 70, 64, 5), (3, 2, 4, 2), 3), workloads.SeqSchedule((64, 1, 129), (2, 0, 3), 0)]
    for mode in ("decode", "extend"):
        _, plan, batches, flats = pu.run_plan(w, scheds, 0, mode=mode, lookahead=2, lag_units=1)
        assert any(c.vis is not None and c.unit >= 0 and (c.vis == c.unit + 2).all() for c in plan.calls)
        pu.check_against_oracle(w, scheds, plan, batches[0], flats[0], what=f"lag 1 {mode}", lag_units=1)
    w1 = workloads.WORKLOADS[1]
    s1 = workloads.schedules(1, batch=3)
    _, plan, batches, flats = pu.run_plan(w1, s1, 1, mode="decode", lookahead=3)
    pu.check_against_oracle(w1, s1, plan, batches[0], flats[0], n_random=64, full_seqs=(1,), what="cfg1 lookahead 3")


@pytest.mark.parametrize("position_mode", [api.ST_POS_CONCATENATED, api.ST_POS_UNIT_ALIGNED])
def test_other_position_modes(position_mode):
    """The original RoPE ids (reasoning token t at T + t, whole input appended first: the batch setting in which the
    paper compares the encodings) and the unit-aligned variant: rows and both caches against the oracle with the same
    ids, token by token (the decode kernel's fused append) and span by span (append kernel + tensor-core kernel)."""
    w = small_workload(32)
    scheds = [workloads.SeqSchedule((30, 70, 64, 5), (3, 2, 4, 2), 3), workloads.SeqSchedule((64, 1, 129), (2, 0, 3), 0),
              workloads.SeqSchedule((200, 56), (70, 9), 66)]
    lookahead = 4 if position_mode == api.ST_POS_CONCATENATED else 2
    for mode in ("decode", "extend"):
        ctx, plan, batches, flats = pu.run_plan(w, scheds, 0, mode=mode, lookahead=lookahead, position_mode=position_mode)
        pu.check_against_oracle(w, scheds, plan, batches[0], flats[0], what=f"position mode {position_mode} {mode}",
                                position_mode=position_mode)
        assert pu.check_cache(ctx, w, scheds, plan, flats[0], position_mode=position_mode) <= 2
        ctx.close()


@pytest.mark.parametrize("variant", ["plain", "lag1", "concatenated", "two_term", "simple_kernels"])
def test_packed_forward_matches_the_oracle_layout(variant):
    """st_forward_packed: one pass over [source ; reasoning] per sequence under the streaming mask -- the layout the
    oracle itself materialises -- for ragged schedules (empty units, a sequence without reasoning, several 128-row
    tiles per unit), every row against the oracle; then three more decode steps continue from the caches it left."""
    hq = 40 if variant == "two_term" else 32
    w = workloads.Workload(0, f"packed-{variant}", hq, 8, 1, outlier_frac=0.02 if variant == "two_term" else 0.0,
                           outlier_mult=8.0 if variant == "two_term" else 1.0)
    extra = 3
    scheds = [workloads.SeqSchedule((30, 70, 64, 5), (3, 2, 4, 2), 3), workloads.SeqSchedule((64, 1, 129), (2, 0, 3), 0),
              workloads.SeqSchedule((200, 56), (70, 9), 66), workloads.SeqSchedule((130,), (0,), 0)]
    longer = [workloads.SeqSchedule(s.src_unit_len, s.rsn_unit_len, s.final_len + extra) for s in scheds]
    lag = 1 if variant == "lag1" else 0
    pm = api.ST_POS_CONCATENATED if variant == "concatenated" else api.ST_POS_STREAMING
    total = sum(s.S + s.R for s in scheds)
    cfg = api.make_config(n_q_heads=hq, n_kv_heads=8, max_batch=len(scheds), n_pages_source=sum((s.S + 63) // 64 for s in scheds),
                          n_pages_reason=sum((s.R + extra + 63) // 64 for s in scheds), max_tokens_per_call=total,
                          flags=api.ST_CFG_PRECISE_P if variant == "two_term" else 0, position_mode=pm)
    ctx = api.Context(cfg)
    dev = torch.device("cuda", 0)
    tensors = [workloads.qkv(0, s, b, workload=w) for b, s in enumerate(longer)]
    q, k, v = (torch.cat([t[i][: s.S + s.R] for t, s in zip(tensors, scheds)]).to(dev) for i in range(3))
    out = torch.full((total, hq, 128), float("nan"), dtype=torch.float32, device=dev)
    ids = list(range(len(scheds)))
    ctx.forward_packed(0, ids, scheds, q, k, v, out, lag_units=lag,
                       flags=api.ST_REFERENCE_KERNELS if variant == "simple_kernels" else 0)
    steps = []
    for i in range(extra):
        qd, kd, vd = (torch.stack([t[j][s.S + s.R + i] for t, s in zip(tensors, scheds)]).to(dev) for j in range(3))
        o1 = torch.full((len(scheds), hq, 128), float("nan"), dtype=torch.float32, device=dev)
        ctx.reason_decode(0, ids, [api.ST_VIS_ALL] * len(scheds), qd, kd, vd, o1)
        steps.append(o1)
    torch.cuda.synchronize()
    ctx.device_status()
    row = 0
    for b, (s, sl) in enumerate(zip(scheds, longer)):
        n = s.S + s.R
        qb, kb, vb = tensors[b]
        want = pu.oracle_rows(w, sl, qb, kb, vb, np.arange(sl.S + sl.R), lag_units=lag, position_mode=pm)
        pu.compare(out[row:row + n].cpu().numpy(), want[:n], f"packed forward {variant} seq {b}")
        got_steps = torch.stack([o1[b] for o1 in steps]).cpu().numpy()
        pu.compare(got_steps, want[n:], f"decode steps after the packed forward {variant} seq {b}")
        row += n
    ctx.close()


@pytest.mark.parametrize("two_term", [False, True])
def test_qk_rmsnorm_fused_into_the_rotating_kernels(two_term):
    """Per-head RMS normalisation of q and k (Qwen3) in front of the rotation, in every kernel that rotates: the
    append kernel (keys of chunks and spans, queries of the two-term variant), the decode kernel's fused append (new
    key and the step's queries) and the attention kernel's query rotation. Two layers with different weights; rows
    of both layers and the caches (normalised, rotated, rounded once) against the oracle."""
    w = small_workload(40)
    rng = np.random.default_rng(33)
    wq = rng.uniform(0.5, 1.5, size=(2, 128)).astype(np.float32)
    wk = rng.uniform(0.5, 1.5, size=(2, 128)).astype(np.float32)
    eps = 1e-6
    scheds = [workloads.SeqSchedule((30, 70, 64, 5), (3, 2, 4, 2), 3), workloads.SeqSchedule((64, 1, 129), (2, 0, 3), 0),
              workloads.SeqSchedule((200, 56), (70, 9), 66)]
    flags = api.ST_CFG_PRECISE_P if two_term else 0
    for mode in ("decode", "extend"):
        ctx, plan, batches, flats = pu.run_plan(w, scheds, 0, mode=mode, lookahead=2, layer_seeds=(0, 1), cfg_flags=flags,
                                                qk_norm=(wq, wk, eps))
        for layer in range(2):
            norm = (wq[layer], wk[layer], eps)
            pu.check_against_oracle(w, scheds, plan, batches[layer], flats[layer], what=f"qk norm {mode} layer {layer}",
                                    qk_norm=norm)
            assert pu.check_cache(ctx, w, scheds, plan, flats[layer], layer=layer, k_norm=(wk[layer], eps)) <= 2
        ctx.close()


def test_page_id_outside_the_pool_is_reported_not_dereferenced():
    """The kernels compare every page id they read with the pool's page count before they build an address from it.
    The test overwrites one entry of the device page table with an id far outside the pool (a host-side test hook,
    nothing on the device is broken on purpose): the next decode step reports ST_ERR_DEVICE_CHECK through the status
    word, nothing faults, and after st_reset the context computes correct rows again."""
    w = workloads.WORKLOADS[0]
    scheds = workloads.schedules(0)
    plan = runner.make_plan(scheds, mode="decode")
    ctx = runner.make_context(w, scheds, plan)
    flat = runner.flatten_inputs(0, scheds, layer=0)
    dev = torch.device("cuda", 0)
    z = lambda n, H: torch.zeros((n, H, 128), dtype=torch.bfloat16, device=dev)
    Hq, Hkv = w.n_q_heads, w.n_kv_heads
    for which, call in ((0, "decode"), (1, "decode"), (0, "append")):
        # a short sound prefix: one source unit of 32 tokens and three decode steps
        ctx.append_source_chunk(0, [0], [0, 32], z(32, Hq), z(32, Hkv), z(32, Hkv), None, api.ST_END_OF_UNIT)
        out = torch.full((1, Hq, 128), float("nan"), dtype=torch.float32, device=dev)
        for _ in range(3):
            ctx.reason_decode(0, [0], None, z(1, Hq), z(1, Hkv), z(1, Hkv), out)
        ctx.device_status()
        ctx.debug_corrupt_page_table(0, which, 0, 1 << 20)
        if call == "decode":
            ctx.reason_decode(0, [0], None, z(1, Hq), z(1, Hkv), z(1, Hkv), out)
        else:
            ctx.append_source_chunk(0, [0], [0, 1], z(1, Hq), z(1, Hkv), z(1, Hkv), out)
        with pytest.raises(api.StError) as e:
            ctx.device_status()
        assert e.value.code == api.ST_ERR_DEVICE_CHECK
        ctx.device_status()                                   # cleared by the read
        ctx.reset()                                           # new appends rewrite the table entries
        batch = runner.DeviceBatch(plan, *flat)
        runner.CompiledPlan(ctx, plan, [batch]).replay()
        torch.cuda.synchronize()
        ctx.device_status()
        pu.check_against_oracle(w, scheds, plan, batch, flat, what=f"after a bad page id in table {which}")
        ctx.reset()
    ctx.close()


def test_more_sequences_than_one_launch_holds():
    """130 sequences in one call: a kernel launch carries at most 112, so every call is split into two launches."""
    w = small_workload(16)
    rng = np.random.default_rng(7)
    scheds = [workloads.SeqSchedule(tuple(int(x) for x in rng.integers(1, 40, size=2)),
                                    tuple(int(x) for x in rng.integers(0, 5, size=2)), int(rng.integers(0, 3)))
              for _ in range(130)]
    for mode in ("decode", "extend"):
        ctx, plan, batches, flats = pu.run_plan(w, scheds, 0, mode=mode)
        pu.check_against_oracle(w, scheds, plan, batches[0], flats[0], what=f"130 sequences {mode}")
        assert pu.check_cache(ctx, w, scheds, plan, flats[0], seqs=(0, 111, 112, 129)) <= 2


def test_two_streams_equal_serial_bitwise():
    w = workloads.WORKLOADS[1]
    scheds = workloads.schedules(1, batch=4)
    _, plan, b1, flats = pu.run_plan(w, scheds, 1, mode="decode")
    _, plan2, b2, _ = pu.run_plan(w, scheds, 1, mode="decode", two_streams=True, flat_inputs=flats)
    assert torch.equal(b1[0].out_src, b2[0].out_src)
    assert torch.equal(b1[0].out_rsn, b2[0].out_rsn)


def test_kernel_timers_sample_every_nth_decode_launch_and_leave_results_alone():
    """With a sampling period N the context brackets every N-th decode launch (and every launch of the tensor-core
    kernel) with events; a bracketed launch is serialised against its neighbours, the others overlap their
    prologue with the kernel in front, and both give the same rows bit for bit."""
    w = workloads.WORKLOADS[0]
    scheds = workloads.schedules(0)
    plan = runner.make_plan(scheds, mode="decode", lookahead=1)
    n_decode = sum(1 for c in plan.calls if c.kind == runner.DECODE)
    n_append = sum(1 for c in plan.calls if c.kind == runner.APPEND)
    outs = []
    for every in (0, 1, 5):
        ctx = runner.make_context(w, scheds, plan)
        batch = runner.DeviceBatch(plan, *runner.flatten_inputs(0, scheds, layer=0))
        ctx.kernel_timing_enable(every)
        runner.CompiledPlan(ctx, plan, [batch]).replay()
        torch.cuda.synchronize()
        ctx.device_status()
        n_dec, ms_dec = ctx.kernel_timing_read(0)
        n_tc, ms_tc = ctx.kernel_timing_read(1)
        if every == 0:
            assert (n_dec, n_tc) == (0, 0)
        else:
            assert n_dec == (n_decode + every - 1) // every and n_tc == n_append
            assert ms_dec > 0 and ms_tc > 0
        assert ctx.kernel_timing_read(0) == (0, 0.0)          # a read clears
        outs.append(batch.outputs_flat().clone())
        ctx.close()
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])


def test_decode_steps_at_large_positions():
    """Decode steps whose token sits at reasoning positions ~69,630 (across a multiple of 1024): the append that
    runs inside the decode kernel takes cos/sin from two tables by an angle addition, and the rotated keys it
    writes must still be the oracle's bf16(RoPE_fp64(k)) bit for bit. Everything expected comes from the oracle on
    the raw inputs: the whole reasoning cache (the 69,629 keys the span append wrote and the 6 of the decode steps)
    against expected_cache, and the decode rows against attention_rows."""
    import time
    from oracle import streaming_attention as osa
    Hq, Hkv = 4, 2
    S, R0, steps, theta = 64, 69_629, 6, 1.0e6
    R = R0 + steps
    cfg = api.make_config(n_q_heads=Hq, n_kv_heads=Hkv, max_batch=1, n_pages_source=2, n_pages_reason=R // 64 + 2,
                          max_source_len=128, max_reason_len=R + 64, max_tokens_per_call=8192, rope_theta=theta)
    ctx = api.Context(cfg)
    dev = torch.device("cuda", 0)
    g = torch.Generator().manual_seed(7)
    draw = lambda n, H: torch.randn((n, H, 128), generator=g).to(torch.bfloat16)
    stream = torch.cuda.current_stream().cuda_stream
    q_all, k_all, v_all = draw(S + R, Hq), draw(S + R, Hkv), draw(S + R, Hkv)     # layout [source ; reasoning]
    ctx.append_source_chunk(0, [0], [0, S], q_all[:S].to(dev), k_all[:S].to(dev), v_all[:S].to(dev), None,
                            api.ST_END_OF_UNIT, stream)
    done = 0
    while done < R0:                                            # cache-only spans (no attention) up to position R0
        n = min(8192, R0 - done)
        sl = slice(S + done, S + done + n)
        ctx.reason_extend(0, [0], [0, n], [api.ST_VIS_ALL], q_all[sl].to(dev), k_all[sl].to(dev), v_all[sl].to(dev), None, 0, stream)
        done += n
    outs = []
    for i in range(steps):
        sl = slice(S + R0 + i, S + R0 + i + 1)
        out = torch.full((1, Hq, 128), float("nan"), dtype=torch.float32, device=dev)
        ctx.reason_decode(0, [0], [api.ST_VIS_ALL], q_all[sl].to(dev), k_all[sl].to(dev), v_all[sl].to(dev), out, 0, stream)
        outs.append(out)
    torch.cuda.synchronize()
    ctx.device_status()
    as_f64 = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).double().numpy()

    t0 = time.perf_counter()
    sched = osa.build_schedule([S], [0], R)                     # one source unit, every reasoning token final-depth
    kd, vd = k_all.double().numpy(), v_all.double().numpy()
    (ks_want, vs_want), (kr_want, vr_want) = osa.expected_cache(sched, kd, vd, theta)
    # both caches as stored against the oracle's definition (at most a couple of one-ulp rounding disagreements)
    for which, kw, vw, n in ((0, ks_want, vs_want, S), (1, kr_want, vr_want, R)):
        kg, vg = (as_f64(a) for a in ctx.debug_read_cache(0, 0, which, 0, n))
        assert np.array_equal(vg, vw)
        diff = kg != kw
        assert int(diff.sum()) <= 4, f"cache {which}: {int(diff.sum())} rotated keys differ from the oracle's"
        assert (np.abs(kg[diff] - kw[diff]) <= np.abs(kw[diff]) * 2.0 ** -7).all()
        if which == 1:
            assert int(diff[R0:].sum()) <= 1                      # the six keys the decode kernel appended
    rows = S + R0 + np.arange(steps)
    want = osa.attention_rows(sched, q_all.double().numpy(), kd, vd, rows, theta=theta)
    print(f"oracle: {time.perf_counter() - t0:.1f} s for both caches and {steps} rows over {S + R} keys")
    for i in range(steps):
        pu.compare(outs[i][0].cpu().numpy(), want[i], f"decode step at position {R0 + i}")
    ctx.close()


def test_bounded_wait_expires_into_a_status_and_leaves_the_context_usable():
    """A device-side wait that nothing satisfies ends after its limit with ST_ERR_DEVICE_TIMEOUT in the status word
    (read once, then cleared); the kernel returns, nothing hangs, and the context computes correct rows afterwards."""
    import time
    w = workloads.WORKLOADS[0]
    scheds = workloads.schedules(0)
    plan = runner.make_plan(scheds, mode="decode")
    ctx = runner.make_context(w, scheds, plan)
    assert ctx.debug_wait_expiry(0, check=False) == api.ST_ERR_INVALID_ARG
    assert ctx.debug_wait_expiry(5000, check=False) == api.ST_ERR_INVALID_ARG
    t0 = time.perf_counter()
    ctx.debug_wait_expiry(150)
    with pytest.raises(api.StError) as e:
        ctx.device_status()
    dt = time.perf_counter() - t0
    assert e.value.code == api.ST_ERR_DEVICE_TIMEOUT
    assert 0.1 < dt < 1.5, f"the wait took {dt:.3f} s for a limit of 0.15 s"
    ctx.device_status()                                      # cleared by the read above
    flat = runner.flatten_inputs(0, scheds, layer=0)
    batch = runner.DeviceBatch(plan, *flat)
    runner.CompiledPlan(ctx, plan, [batch]).replay()
    torch.cuda.synchronize()
    ctx.device_status()
    pu.check_against_oracle(w, scheds, plan, batch, flat, what="after an expired wait")
    ctx.close()


def test_multi_layer_pools_are_independent():
    w = small_workload(32)
    scheds = [workloads.scaled_schedule(3, 70, 5, 9), workloads.scaled_schedule(3, 33, 2, 1)]
    ctx, plan, batches, flats = pu.run_plan(w, scheds, 0, mode="decode", layer_seeds=(0, 1, 2))
    for layer in range(3):
        pu.check_against_oracle(w, scheds, plan, batches[layer], flats[layer], what=f"layer {layer}")
        assert pu.check_cache(ctx, w, scheds, plan, flats[layer], layer=layer) <= 2


@pytest.mark.parametrize("index,memory", [(0, "pinned"), (1, "pinned"), (1, "pageable")])
def test_host_io_flag_matches_device_io(index, memory):
    """ST_IO_HOST gives the rows of device buffers bit for bit on each of its routes: page-locked buffers of a
    small call are read and written in place by the kernels (every call of workload 0, the decode steps of
    workload 1), large calls (workload 1's appends of 512 tokens = 4 MiB) and ordinary pageable memory go through
    the staging copies."""
    w = workloads.WORKLOADS[index]
    scheds = workloads.schedules(index)
    _, plan, b_dev, flats = pu.run_plan(w, scheds, index, mode="decode")
    plan_h = runner.make_plan(scheds, mode="decode")
    ctx = runner.make_context(w, scheds, plan_h)
    b_host = runner.DeviceBatch(plan_h, *flats[0], pinned_host=memory == "pinned", pageable_host=memory == "pageable")
    b_host.out_src.fill_(float("nan"))
    b_host.out_rsn.fill_(float("nan"))
    runner.CompiledPlan(ctx, plan_h, [b_host]).replay()
    torch.cuda.synchronize()
    ctx.device_status()
    assert torch.equal(b_host.out_src[: plan.n_src_tokens], b_dev[0].out_src[: plan.n_src_tokens].cpu())
    assert torch.equal(b_host.out_rsn[: plan.n_rsn_tokens], b_dev[0].out_rsn[: plan.n_rsn_tokens].cpu())
    ctx.close()


def test_reset_and_reuse_of_pages():
    w = workloads.WORKLOADS[0]
    scheds = workloads.schedules(0)
    plan = runner.make_plan(scheds, mode="decode")
    ctx = runner.make_context(w, scheds, plan)
    flat = runner.flatten_inputs(0, scheds)
    outs = []
    for _ in range(2):
        batch = runner.DeviceBatch(plan, *flat)
        runner.CompiledPlan(ctx, plan, [batch]).replay()
        torch.cuda.synchronize()
        outs.append(batch.outputs_flat())
        ctx.reset()
    assert torch.equal(outs[0], outs[1])
    assert ctx.launch_count() > 0
