"""Shared helpers of the GPU parity tests: run a plan through the C ABI, compare with the oracle."""
import numpy as np
import torch

from oracle import streaming_attention as osa
from paper_2510_17238_b200 import api, runner, workloads

MAX_ABS_TOL = 1e-2      # bf16 inputs, fp32 accumulation (stated tolerance of the method's contract)
REL_L2_TOL = 5e-3


POSITION_MODE_NAMES = {0: "streaming", 1: "concatenated", 2: "unit_aligned"}


def oracle_rows(workload, sched, q, k, v, rows, lag_units=0, position_mode=0, qk_norm=None):
    """fp64 oracle outputs for the listed rows of one sequence (q/k/v: CPU bf16 [S+R, H, 128])."""
    o = osa.build_schedule(sched.src_unit_len, sched.rsn_unit_len, sched.final_len, lag_units=lag_units,
                           position_mode=POSITION_MODE_NAMES[position_mode])
    return osa.attention_rows(o, q.double().numpy(), k.double().numpy(), v.double().numpy(), rows,
                              theta=workload.rope_theta, qk_norm=qk_norm)


def sample_rows(sched, n_random, seed):
    """First and last row of every unit (both streams) plus n_random seeded rows."""
    S, R = sched.S, sched.R
    rows = set()
    p = 0
    for n in sched.src_unit_len:
        if n:
            rows.update((p, p + n - 1))
        p += n
    r = 0
    for m in sched.rsn_unit_len:
        if m:
            rows.update((S + r, S + r + m - 1))
        r += m
    if sched.final_len:
        rows.update((S + r, S + R - 1))
    rng = np.random.default_rng([seed, S, R])
    rows.update(int(x) for x in rng.integers(0, S + R, size=min(n_random, S + R)))
    return np.array(sorted(rows), dtype=np.int64)


def compare(got, want, what=""):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert not np.isnan(got).any(), f"{what}: NaN in the GPU output (row never written?)"
    err = np.abs(got - want)
    max_abs = float(err.max())
    rel_l2 = float(np.linalg.norm(got - want) / np.linalg.norm(want))
    at = tuple(int(i) for i in np.unravel_index(int(err.argmax()), err.shape))
    assert max_abs <= MAX_ABS_TOL and rel_l2 <= REL_L2_TOL, (
        f"{what}: max_abs={max_abs:.3e} rel_l2={rel_l2:.3e}; worst element at index {at}: got {got[at]:.6f}, "
        f"want {want[at]:.6f}")
    return max_abs, rel_l2


def run_plan(workload, scheds, index, mode="decode", lookahead=1, two_streams=False, extra_flags=0, layer_seeds=(0,),
             flat_inputs=None, n_layers=None, lag_units=0, cfg_flags=0, position_mode=0, qk_norm=None):
    """Runs a whole plan on the GPU. Returns (ctx, plan, batches, flats) with outputs synchronised."""
    plan = runner.make_plan(scheds, mode=mode, lookahead=lookahead, lag_units=lag_units)
    L = len(layer_seeds) if n_layers is None else n_layers
    ctx = runner.make_context(workload, scheds, plan, n_layers=L, flags=cfg_flags, position_mode=position_mode,
                              qk_norm=qk_norm)
    flats, batches = [], []
    for layer in range(L):
        fl = flat_inputs[layer] if flat_inputs is not None else runner.flatten_inputs(
            index, scheds, layer=layer_seeds[layer % len(layer_seeds)], workload=workload)
        flats.append(fl)
        batches.append(runner.DeviceBatch(plan, *fl))
    if two_streams:
        sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
        torch.cuda.synchronize()
        cp = runner.CompiledPlan(ctx, plan, batches, sa, sb, extra_flags=extra_flags)
    else:
        cp = runner.CompiledPlan(ctx, plan, batches, extra_flags=extra_flags)
    cp.replay()
    torch.cuda.synchronize()
    ctx.device_status()
    return ctx, plan, batches, flats


def check_against_oracle(workload, scheds, plan, batch, flat, n_random=None, full_seqs=(), what="", lag_units=0,
                         position_mode=0, qk_norm=None):
    """Compares a layer's GPU outputs with the oracle: all rows for `full_seqs` (or every sequence when
    n_random is None), unit-boundary rows plus n_random seeded rows otherwise."""
    out = batch.outputs_flat()
    worst = (0.0, 0.0)
    fq, fk, fv = flat
    for b, s in enumerate(scheds):
        lo, hi = int(plan.seq_offset[b]), int(plan.seq_offset[b + 1])
        if hi == lo:
            continue
        rows = np.arange(hi - lo) if (n_random is None or b in full_seqs) else sample_rows(s, n_random, b)
        want = oracle_rows(workload, s, fq[lo:hi], fk[lo:hi], fv[lo:hi], rows, lag_units=lag_units,
                           position_mode=position_mode, qk_norm=qk_norm)
        got = out[lo:hi][torch.from_numpy(rows)].numpy()
        r = compare(got, want, f"{what} seq {b}")
        worst = (max(worst[0], r[0]), max(worst[1], r[1]))
    # every row must have been produced
    assert not torch.isnan(out).any(), f"{what}: some rows were never written"
    return worst


def check_cache(ctx, workload, scheds, plan, flat, layer=0, seqs=None, position_mode=0, k_norm=None):
    """Cache contents vs the oracle's definition bf16(RoPE_fp64(k)), v. Returns mismatching key elements."""
    fq, fk, fv = flat
    bad = 0
    for b, s in enumerate(scheds):
        if seqs is not None and b not in seqs:
            continue
        lo, hi = int(plan.seq_offset[b]), int(plan.seq_offset[b + 1])
        o = osa.build_schedule(s.src_unit_len, s.rsn_unit_len, s.final_len, position_mode=POSITION_MODE_NAMES[position_mode])
        (ks, vs), (kr, vr) = osa.expected_cache(o, fk[lo:hi].double().numpy(), fv[lo:hi].double().numpy(),
                                                workload.rope_theta, k_norm=k_norm)
        for which, (kw, vw, n) in enumerate(((ks, vs, s.S), (kr, vr, s.R))):
            if n == 0:
                continue
            kg, vg = ctx.debug_read_cache(layer, b, which, 0, n)
            kg = torch.from_numpy(kg.view(np.int16)).view(torch.bfloat16).double().numpy()
            vg = torch.from_numpy(vg.view(np.int16)).view(torch.bfloat16).double().numpy()
            assert np.array_equal(vg, vw), "values must be stored unchanged"
            diff = kg != kw
            if diff.any():
                # a double-rounding style disagreement may move a key by one bf16 ulp at most
                ulp = np.abs(kw[diff]) * 2.0 ** -7
                assert (np.abs(kg[diff] - kw[diff]) <= ulp).all(), "rotated key off by more than one bf16 ulp"
            bad += int(diff.sum())
    return bad
