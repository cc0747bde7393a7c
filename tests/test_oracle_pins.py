"""Pins for the fp64 oracle: every check here is independent of oracle code.

What is compared against what:
* a scalar triple-loop attention over one concatenated cache with an explicit
  mask built from Eq. 1's conditioning sets (written here, shares nothing),
* torch's scaled_dot_product_attention (library routine) for the cases that
  reduce to ordinary causal attention, with RoPE done as a complex rotation,
* closed forms / invariants: softmax rows, position ids, RoPE properties,
  invariance of source rows to reasoning tokens, Eq. 2's indicator.
"""
import cmath
import math

import os

import numpy as np
import pytest
import torch

from oracle import streaming_attention as osa

THETA = 1.0e6


# ----------------------------------------------------------------------------- helpers (independent)

def conditioning_sets(n, m, final_len, lag=0):
    """Eq. 1: reasoning unit u conditions on C_{<=u} and on all earlier reasoning; the final
    stage conditions on everything. Returned as {row index: set(column indices)} over
    the layout [source ; reasoning]."""
    U = len(n)
    S = sum(n)
    src_cols_of_unit = []
    j = 0
    for u in range(U):
        src_cols_of_unit.append(list(range(j, j + n[u])))
        j += n[u]
    allowed = {}
    for i in range(S):
        allowed[i] = set(range(0, i + 1))
    r = 0
    for u in range(U):
        for _ in range(m[u]):
            cols = set()
            for uu in range(min(u + 1 + lag, U)):
                cols.update(src_cols_of_unit[uu])
            cols.update(S + rr for rr in range(r + 1))
            allowed[S + r] = cols
            r += 1
    for _ in range(final_len):
        allowed[S + r] = set(range(S)) | {S + rr for rr in range(r + 1)}
        r += 1
    return allowed


def scalar_rope(vec, pos, theta):
    d = len(vec)
    out = [0.0] * d
    for c in range(d // 2):
        ang = pos * theta ** (-2.0 * c / d)
        cs, sn = math.cos(ang), math.sin(ang)
        out[c] = vec[c] * cs - vec[c + d // 2] * sn
        out[c + d // 2] = vec[c + d // 2] * cs + vec[c] * sn
    return out


def brute_force(n, m, final_len, q, k, v, Hq, Hkv, theta, round_fn=None):
    """Scalar loops; returns O[S+R][Hq][d] as nested lists."""
    allowed = conditioning_sets(n, m, final_len)
    S = sum(n)
    T = S + sum(m) + final_len
    d = q.shape[-1]
    G = Hq // Hkv
    pos = [i if i < S else i - S for i in range(T)]
    qr = [[scalar_rope(list(q[i, h]), pos[i], theta) for h in range(Hq)] for i in range(T)]
    kr = [[scalar_rope(list(k[i, h]), pos[i], theta) for h in range(Hkv)] for i in range(T)]
    if round_fn is not None:
        qr = [[[round_fn(x) for x in hv] for hv in row] for row in qr]
        kr = [[[round_fn(x) for x in hv] for hv in row] for row in kr]
    out = np.zeros((T, Hq, d))
    for i in range(T):
        for h in range(Hq):
            cols = sorted(allowed[i])
            logits = []
            for j in cols:
                acc = 0.0
                for c in range(d):
                    acc += qr[i][h][c] * kr[j][h // G][c]
                logits.append(acc / math.sqrt(d))
            mx = max(logits)
            w = [math.exp(z - mx) for z in logits]
            tot = sum(w)
            for c in range(d):
                acc = 0.0
                for a, j in enumerate(cols):
                    acc += w[a] * float(v[j, h // G, c])
                out[i, h, c] = acc / tot
    return out


def complex_rope(x, pos, theta):
    """RoPE as multiplication by e^{i pos w_c} of the complex number x[c] + i x[c + d/2]."""
    T, H, d = x.shape
    out = np.empty_like(x, dtype=np.float64)
    for t in range(T):
        for c in range(d // 2):
            rot = cmath.exp(1j * float(pos[t]) * theta ** (-2.0 * c / d))
            for h in range(H):
                z = complex(x[t, h, c], x[t, h, c + d // 2]) * rot
                out[t, h, c] = z.real
                out[t, h, c + d // 2] = z.imag
    return out


def bf16_via_torch(x):
    return float(torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64))


def rand_qkv(rng, T, Hq, Hkv, d, bf16=True):
    def mk(H):
        x = rng.standard_normal((T, H, d))
        if bf16:
            x = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
        return x
    return mk(Hq), mk(Hkv), mk(Hkv)


# ----------------------------------------------------------------------------- tests

@pytest.mark.parametrize("n,m,f,Hq,Hkv,d,row_block", [
    ([2, 3, 1], [1, 2, 2], 2, 2, 1, 4, 256),
    ([1, 1, 1, 1], [1, 1, 1, 1], 0, 2, 2, 8, 256),
    ([3, 2], [0, 2], 1, 4, 2, 4, 256),
    ([4], [3], 0, 1, 1, 8, 256),
    # the oracle's loop over blocks of rows, with several blocks and a ragged last one: 11 rows in blocks of 3,
    # 8 rows in blocks of 1 and 7 rows in blocks of 4
    ([2, 3, 1], [1, 2, 2], 2, 2, 1, 4, 3),
    ([1, 1, 1, 1], [1, 1, 1, 1], 0, 2, 2, 8, 1),
    ([4], [3], 0, 1, 1, 8, 4),
])
def test_brute_force_tiny(n, m, f, Hq, Hkv, d, row_block):
    rng = np.random.default_rng(11)
    sched = osa.build_schedule(n, m, f)
    q, k, v = rand_qkv(rng, sched.S + sched.R, Hq, Hkv, d)
    want = brute_force(n, m, f, q, k, v, Hq, Hkv, THETA)
    got = osa.attention_rows(sched, q, k, v, np.arange(sched.S + sched.R), theta=THETA, round_rotated=False,
                             row_block=row_block)
    assert np.abs(got - want).max() < 1e-12
    # with the two bf16 rounding points (rounded through torch, not the oracle's routine)
    want_r = brute_force(n, m, f, q, k, v, Hq, Hkv, THETA, round_fn=bf16_via_torch)
    got_r = osa.attention_rows(sched, q, k, v, np.arange(sched.S + sched.R), theta=THETA, round_rotated=True,
                               row_block=row_block)
    assert np.abs(got_r - want_r).max() < 1e-12
    assert np.abs(got_r - got).max() > 1e-6      # the rounding is really applied


def test_row_subsets_in_any_order_across_blocks():
    """Rows may be listed in any order, repeated, and spread over several row blocks: every listed row equals the
    scalar loops' row (the GPU parity tests hand the oracle sampled row lists longer than one block)."""
    rng = np.random.default_rng(12)
    n, m, f, Hq, Hkv, d = [3, 1, 4], [2, 0, 3], 2, 4, 2, 8
    sched = osa.build_schedule(n, m, f)
    T = sched.S + sched.R
    q, k, v = rand_qkv(rng, T, Hq, Hkv, d)
    want = brute_force(n, m, f, q, k, v, Hq, Hkv, THETA)
    rows = np.array([T - 1, 0, 9, 9, 3, 12, 1, 8, 14, 2, 5])
    for blk in (2, 5, 256):
        got, probs = osa.attention_rows(sched, q, k, v, rows, theta=THETA, round_rotated=False, row_block=blk,
                                        return_probs=True)
        assert np.abs(got - want[rows]).max() < 1e-12
        assert np.abs(probs.sum(-1) - 1).max() < 1e-12


def sdpa_causal(qr, kr, v, G, scale):
    """Ordinary causal attention with torch's library routine, fp64."""
    qt = torch.from_numpy(qr).permute(1, 0, 2)                       # [Hq, T, d]
    kt = torch.from_numpy(np.repeat(kr, G, axis=1)).permute(1, 0, 2)
    vt = torch.from_numpy(np.repeat(v, G, axis=1)).permute(1, 0, 2)
    o = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True, scale=scale)
    return o.permute(1, 0, 2).numpy()


def test_single_unit_is_causal_attention():
    """One unit, no final tokens: the source rows are plain causal attention."""
    rng = np.random.default_rng(5)
    S, Hq, Hkv, d = 37, 4, 2, 16
    sched = osa.build_schedule([S], [0], 0)
    q, k, v = rand_qkv(rng, S, Hq, Hkv, d)
    got = osa.attention_rows(sched, q, k, v, np.arange(S), theta=THETA, round_rotated=False)
    pos = np.arange(S)
    want = sdpa_causal(complex_rope(q, pos, THETA), complex_rope(k, pos, THETA), v, Hq // Hkv, 1 / math.sqrt(d))
    assert np.abs(got - want).max() < 1e-12


def test_everything_visible_is_causal_over_concatenation():
    """The 'batch' route: if every reasoning token sees the whole source, the streaming mask is
    the ordinary causal mask over [source ; reasoning]; only the position ids stay streaming."""
    rng = np.random.default_rng(6)
    n, m, f = [5, 7, 3], [4, 0, 6], 5
    Hq, Hkv, d = 4, 2, 16
    sched = osa.build_schedule(n, m, f, lag_units=len(n))
    T = sched.S + sched.R
    q, k, v = rand_qkv(rng, T, Hq, Hkv, d)
    got = osa.attention_rows(sched, q, k, v, np.arange(T), theta=THETA, round_rotated=False)
    pos = np.concatenate([np.arange(sched.S), np.arange(sched.R)])
    want = sdpa_causal(complex_rope(q, pos, THETA), complex_rope(k, pos, THETA), v, Hq // Hkv, 1 / math.sqrt(d))
    assert np.abs(got - want).max() < 1e-12
    # and with the default lag the reasoning rows of early units must differ from it
    sched0 = osa.build_schedule(n, m, f)
    got0 = osa.attention_rows(sched0, q, k, v, np.arange(T), theta=THETA, round_rotated=False)
    assert np.abs(got0[sched.S] - want[sched.S]).max() > 1e-4
    assert np.abs(got0[: sched.S] - want[: sched.S]).max() < 1e-12     # source rows agree
    assert np.abs(got0[-f:] - want[-f:]).max() < 1e-12                # final-depth rows agree


def test_concatenated_ids_with_everything_visible_is_the_batch_route():
    """Original RoPE ids (reasoning token t at T + t, Section 3.2) with every reasoning token seeing the whole
    input is ordinary causal attention over [input ; reasoning] with ordinary position ids 0 .. T+R-1: the single
    cache "batch" route, computed here by torch's library routine."""
    rng = np.random.default_rng(16)
    n, m, f = [4, 6, 2], [3, 1, 5], 4
    Hq, Hkv, d = 4, 2, 16
    sched = osa.build_schedule(n, m, f, lag_units=len(n), position_mode="concatenated")
    T = sched.S + sched.R
    assert sched.pos_ids.tolist() == list(range(T))
    q, k, v = rand_qkv(rng, T, Hq, Hkv, d)
    got = osa.attention_rows(sched, q, k, v, np.arange(T), theta=THETA, round_rotated=False)
    pos = np.arange(T)
    want = sdpa_causal(complex_rope(q, pos, THETA), complex_rope(k, pos, THETA), v, Hq // Hkv, 1 / math.sqrt(d))
    assert np.abs(got - want).max() < 1e-12
    # the streaming ids give different reasoning rows on the same mask, and the same source rows
    got_s = osa.attention_rows(osa.build_schedule(n, m, f, lag_units=len(n)), q, k, v, np.arange(T), theta=THETA,
                               round_rotated=False)
    assert np.abs(got_s[: sched.S] - want[: sched.S]).max() < 1e-12
    assert np.abs(got_s[sched.S :] - want[sched.S :]).max() > 1e-4


def test_position_modes_closed_form():
    n, m, f = [3, 1, 4], [2, 0, 3], 2
    S = sum(n)
    s0 = osa.build_schedule(n, m, f)
    s1 = osa.build_schedule(n, m, f, position_mode="concatenated")
    s2 = osa.build_schedule(n, m, f, position_mode="unit_aligned")
    for s in (s0, s1, s2):
        assert s.pos_ids[:S].tolist() == list(range(S))                 # the input always counts from zero
        assert np.array_equal(s.vis_len, s0.vis_len)                    # positions do not touch visibility
    assert s0.pos_ids[S:].tolist() == [0, 1, 2, 3, 4, 5, 6]
    assert s1.pos_ids[S:].tolist() == [8, 9, 10, 11, 12, 13, 14]        # T + t
    # unit 1 starts at P_0 = 0, unit 3 at P_2 = 4, the final stage at S = 8
    assert s2.pos_ids[S:].tolist() == [0, 1, 4, 5, 6, 8, 9]
    with pytest.raises(ValueError):
        osa.build_schedule(n, m, f, position_mode="other")


def test_qk_rmsnorm_pins():
    """The q/k normalisation against scalar loops and torch's rms_norm; with eps = 0 a token's scale cancels, so
    attention with the normalisation is invariant to rescaling any query or key token; and the whole path with
    the normalisation equals the scalar brute force fed with rows normalised by the scalar loop."""
    rng = np.random.default_rng(21)
    T, H, d = 9, 3, 8
    x = rng.standard_normal((T, H, d))
    w = rng.uniform(0.5, 1.5, size=d)
    eps = 1e-6
    got = osa.qk_rmsnorm(x, w, eps)
    want = np.empty_like(x)
    for t in range(T):
        for h in range(H):
            ms = sum(float(x[t, h, c]) ** 2 for c in range(d)) / d
            for c in range(d):
                want[t, h, c] = float(x[t, h, c]) / math.sqrt(ms + eps) * float(w[c])
    assert np.abs(got - want).max() < 1e-14
    lib = torch.nn.functional.rms_norm(torch.from_numpy(x), (d,), torch.from_numpy(w), eps).numpy()
    assert np.abs(got - lib).max() < 1e-13
    ones = osa.qk_rmsnorm(x, np.ones(d), 0.0)
    assert np.abs((ones ** 2).mean(-1) - 1).max() < 1e-13            # unit weight: every head has RMS 1
    # scale invariance of the attention rows (eps = 0)
    n, m, f, Hq, Hkv = [3, 2], [2, 1], 1, 4, 2
    sched = osa.build_schedule(n, m, f)
    Tt = sched.S + sched.R
    q, k, v = rand_qkv(rng, Tt, Hq, Hkv, d, bf16=False)
    wq, wk = rng.uniform(0.5, 1.5, size=d), rng.uniform(0.5, 1.5, size=d)
    base = osa.attention_rows(sched, q, k, v, np.arange(Tt), theta=THETA, round_rotated=False, qk_norm=(wq, wk, 0.0))
    scale = rng.uniform(0.2, 5.0, size=(Tt, 1, 1))
    scaled = osa.attention_rows(sched, q * scale, k * scale[::-1], v, np.arange(Tt), theta=THETA, round_rotated=False,
                                qk_norm=(wq, wk, 0.0))
    assert np.abs(base - scaled).max() < 1e-12
    plain = osa.attention_rows(sched, q, k, v, np.arange(Tt), theta=THETA, round_rotated=False)
    assert np.abs(base - plain).max() > 1e-3                         # and it is really applied
    # brute force on rows normalised by scalar loops (and the cache definition with it)
    def scalar_norm(a, wv, e):
        out = np.empty_like(a)
        for t in range(a.shape[0]):
            for h in range(a.shape[1]):
                ms = sum(float(z) ** 2 for z in a[t, h]) / a.shape[2]
                out[t, h] = [float(z) / math.sqrt(ms + e) * float(g) for z, g in zip(a[t, h], wv)]
        return out
    want_rows = brute_force(n, m, f, scalar_norm(q, wq, eps), scalar_norm(k, wk, eps), v, Hq, Hkv, THETA,
                            round_fn=bf16_via_torch)
    got_rows = osa.attention_rows(sched, q, k, v, np.arange(Tt), theta=THETA, qk_norm=(wq, wk, eps))
    assert np.abs(got_rows - want_rows).max() < 1e-12
    (ks, _), (kr, _) = osa.expected_cache(sched, k, v, THETA, k_norm=(wk, eps))
    kn = scalar_norm(k, wk, eps)
    pos = [i if i < sched.S else i - sched.S for i in range(Tt)]
    want_k = np.array([[[bf16_via_torch(z) for z in scalar_rope(list(kn[i, h]), pos[i], THETA)] for h in range(Hkv)]
                       for i in range(Tt)])
    assert np.array_equal(np.concatenate([ks, kr]), want_k)


def test_linear_pins():
    """The projection against a triple loop, against an identity and a selection matrix, and its bf16 rounding
    against torch's conversion."""
    rng = np.random.default_rng(41)
    T, K, N = 5, 7, 4
    x, w = rng.standard_normal((T, K)), rng.standard_normal((N, K))
    want = np.zeros((T, N))
    for t in range(T):
        for n in range(N):
            acc = 0.0
            for k in range(K):
                acc += float(x[t, k]) * float(w[n, k])
            want[t, n] = acc
    got = osa.linear(x, w)
    assert np.abs(got - want).max() < 1e-13
    assert np.array_equal(osa.linear(x, np.eye(K)), x)
    sel = np.zeros((2, K)); sel[0, 3] = 1.0; sel[1, 0] = -2.0
    assert np.array_equal(osa.linear(x, sel), np.stack([x[:, 3], -2.0 * x[:, 0]], axis=1))
    rounded = osa.linear(x, w, round_out=True)
    via_torch = torch.from_numpy(want).to(torch.float32).to(torch.bfloat16).double().numpy()
    assert np.abs(rounded - via_torch).max() <= np.abs(want).max() * 2.0 ** -8   # (torch rounds fp32, a double rounding)
    assert (rounded == via_torch).mean() > 0.9 and np.abs(rounded - want).max() <= np.abs(want).max() * 2.0 ** -8
    with pytest.raises(ValueError):
        osa.linear(x, w.T)


def test_softmax_rows():
    rng = np.random.default_rng(7)
    n, m, f = [3, 4, 2], [2, 3, 1], 3
    sched = osa.build_schedule(n, m, f)
    T = sched.S + sched.R
    q, k, v = rand_qkv(rng, T, 2, 1, 8)
    _, P = osa.attention_rows(sched, q, k, v, np.arange(T), return_probs=True)
    A = osa.dense_mask(sched)
    assert np.abs(P.sum(-1) - 1.0).max() < 1e-12
    assert (P[:, 0, :][A == 0] == 0.0).all() and (P[:, 1, :][A == 0] == 0.0).all()
    assert (P[:, 0, :][A == 1] > 0.0).all()


def test_source_rows_ignore_reasoning_and_reasoning_ignores_future():
    rng = np.random.default_rng(8)
    n, m, f = [6, 5, 7], [3, 4, 2], 4
    Hq, Hkv, d = 4, 2, 16
    sched = osa.build_schedule(n, m, f)
    S, R = sched.S, sched.R
    q, k, v = rand_qkv(rng, S + R, Hq, Hkv, d)
    full = osa.attention_rows(sched, q, k, v, np.arange(S + R))
    # (a) no reasoning tokens at all: same source rows (the matrix products run over a shorter
    #     key axis, so the summation order inside BLAS may differ in the last bits)
    sched_src = osa.build_schedule(n, [0, 0, 0], 0)
    only = osa.attention_rows(sched_src, q[:S], k[:S], v[:S], np.arange(S))
    assert np.abs(only - full[:S]).max() < 1e-14
    # (b) different reasoning tokens: source rows bit-identical
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[S:], k2[S:], v2[S:] = q2[S:] * 3 + 1, k2[S:] * -2, v2[S:] + 5
    assert np.array_equal(osa.attention_rows(sched, q2, k2, v2, np.arange(S)), full[:S])
    # (c) rows of reasoning unit u do not change when source tokens >= P_u change,
    #     nor when later reasoning tokens change
    for u in (1, 2):
        Pu = int(sched.src_prefix[u])
        rows_u = [S + r for r in range(R) if sched.rsn_unit[r] == u]
        last = max(rows_u)
        q3, k3, v3 = q.copy(), k.copy(), v.copy()
        k3[Pu:S] += 7.0
        v3[Pu:S] -= 3.0
        k3[last + 1:] *= 5.0
        v3[last + 1:] *= -1.0
        got = osa.attention_rows(sched, q3, k3, v3, rows_u)
        assert np.array_equal(got, full[rows_u])
        # ... and does change when a visible source token changes
        k4 = k.copy()
        k4[Pu - 1] += 7.0
        assert np.abs(osa.attention_rows(sched, q, k4, v, rows_u) - full[rows_u]).max() > 1e-6


@pytest.mark.parametrize("n,m,f", [([2, 3, 1], [1, 2, 2], 2), ([5], [0], 3), ([1, 1, 1], [2, 0, 1], 0), ([4, 4], [4, 4], 4)])
@pytest.mark.parametrize("lag", [0, 1])
def test_mask_equals_eq1_conditioning_sets(n, m, f, lag):
    sched = osa.build_schedule(n, m, f, lag_units=lag)
    A = osa.dense_mask(sched)
    allowed = conditioning_sets(n, m, f, lag=lag)
    T = sched.S + sched.R
    assert A.shape == (T, T) and A.dtype == np.uint8
    for i in range(T):
        assert set(np.nonzero(A[i])[0].tolist()) == allowed[i]


def _worked_examples():
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "streaming_mask_worked_examples.txt")
    blocks, cur = [], None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("example"):
            n, m, f = (part.strip() for part in line[len("example"):].split(";"))
            cur = dict(n=[int(x) for x in n.split(",")], m=[int(x) for x in m.split(",")], f=int(f), rows=[])
            blocks.append(cur)
        elif line.startswith("pos"):
            cur["pos"] = [int(x) for x in line.split()[1:]]
        elif line.startswith("vis"):
            cur["vis"] = [int(x) for x in line.split()[1:]]
        else:
            cur["rows"].append([int(ch) for ch in line])
    return blocks


def test_hand_written_worked_examples():
    """Masks, position ids and visibility typed by hand from Eq. 1, the streaming mask and the streaming position
    encoding (tests/golden): the oracle's schedule and dense mask reproduce them entry by entry."""
    blocks = _worked_examples()
    assert len(blocks) == 3
    for b in blocks:
        sched = osa.build_schedule(b["n"], b["m"], b["f"])
        assert sched.pos_ids.tolist() == b["pos"]
        assert sched.vis_len.tolist() == b["vis"]
        assert osa.dense_mask(sched).tolist() == b["rows"]


def test_mask_eq2_indicator_token_level():
    """One token per unit. Eq. 2 blocks, for row i >= T and column j < T, the entries with
    j > (i - T) + 1 (0-based), i.e. reasoning step r sees inputs 0..r+1: one more than Eq. 1
    grants. lag_units=1 reproduces the indicator; the default is one unit stricter."""
    T = L = 6
    causal = np.tril(np.ones((T + L, T + L), dtype=np.uint8))
    eq2 = causal.copy()
    for i in range(T + L):
        for j in range(T + L):
            if i >= T and j < T and j > i - T + 1:
                eq2[i, j] = 0
    lit = osa.dense_mask(osa.build_schedule([1] * T, [1] * L, 0, lag_units=1))
    assert np.array_equal(lit, eq2)
    ours = osa.dense_mask(osa.build_schedule([1] * T, [1] * L, 0))
    for r in range(L):
        assert ours[T + r, :T].sum() == r + 1          # inputs 0..r, as Eq. 1 states
        assert lit[T + r, :T].sum() == min(r + 2, T)


def test_position_ids_closed_form():
    n, m, f = [3, 9, 4, 1], [2, 0, 5, 3], 6
    sched = osa.build_schedule(n, m, f)
    S, R = sum(n), sum(m) + f
    assert sched.S == S and sched.R == R
    assert sched.pos_ids.dtype == np.int32 and sched.vis_len.dtype == np.int32
    assert sched.pos_ids[:S].tolist() == list(range(S))
    assert sched.pos_ids[S:].tolist() == list(range(R))
    assert int(sched.pos_ids[:S].max()) == S - 1 and int(sched.pos_ids[S:].max()) == R - 1
    want_vis = [3, 3] + [16] * 5 + [17] * 3 + [17] * 6
    assert sched.vis_len.tolist() == want_vis
    assert sched.src_prefix.tolist() == [0, 3, 12, 16, 17]


def test_rope_properties():
    rng = np.random.default_rng(9)
    d = 16
    x = rng.standard_normal((5, 3, d))
    pos = np.array([0, 1, 7, 1000, 32767])
    y = osa.rope(x, pos, THETA)
    assert np.array_equal(y[0], x[0])                                     # pos 0 is the identity
    n_in = x[..., : d // 2] ** 2 + x[..., d // 2:] ** 2
    n_out = y[..., : d // 2] ** 2 + y[..., d // 2:] ** 2
    assert np.abs(n_in - n_out).max() < 1e-12                             # rotation per pair
    assert np.abs(y - complex_rope(x, pos, THETA)).max() < 1e-9           # independent formula
    # relative-position property: <R(a) q, R(b) k> depends on a - b only
    q = rng.standard_normal((1, 1, d))
    k = rng.standard_normal((1, 1, d))
    for a, b, shift in [(5, 2, 100), (3, 40, 999), (0, 0, 12345)]:
        z0 = (osa.rope(q, [a], THETA) * osa.rope(k, [b], THETA)).sum()
        z1 = (osa.rope(q, [a + shift], THETA) * osa.rope(k, [b + shift], THETA)).sum()
        assert abs(z0 - z1) < 1e-9
    # a sign error in the rotation direction would break this: q at a, k at b equals rotating q by a-b
    z = (osa.rope(q, [9], THETA) * osa.rope(k, [4], THETA)).sum()
    z_rel = (osa.rope(q, [5], THETA) * k).sum()
    assert abs(z - z_rel) < 1e-9
    w = osa.rope_inv_freq(128, THETA)
    assert w[0] == 1.0 and abs(w[32] - 1e-3) < 1e-15 and abs(w[63] - THETA ** (-126 / 128)) < 1e-18


def test_round_to_bf16_matches_torch():
    rng = np.random.default_rng(10)
    x32 = (rng.standard_normal(200000) * np.exp(rng.uniform(-20, 20, 200000))).astype(np.float32)
    want = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    got = osa.round_to_bf16(x32.astype(np.float64))
    assert np.array_equal(got, want)
    # exact ties go to even; zero stays zero; already-representable values are unchanged
    ties = np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -(2.0 + 2 ** -7), 0.0, 1.5, -0.375])
    assert osa.round_to_bf16(ties).tolist() == [1.0, 1.0 + 2 ** -6, -2.0, 0.0, 1.5, -0.375]
    # an fp64 value just above a tie must round up even though its fp32 rounding is the tie itself
    x = 1.0 + 2 ** -8 + 2 ** -40
    assert osa.round_to_bf16(np.array([x]))[0] == 1.0 + 2 ** -7


def test_expected_cache_split():
    rng = np.random.default_rng(12)
    sched = osa.build_schedule([3, 2], [2, 1], 1)
    T = sched.S + sched.R
    _, k, v = rand_qkv(rng, T, 2, 2, 8)
    (ks, vs), (kr, vr) = osa.expected_cache(sched, k, v, THETA)
    assert ks.shape[0] == 5 and kr.shape[0] == 4
    assert np.array_equal(kr[0], osa.round_to_bf16(k[5]))        # reasoning position 0: identity rotation
    assert np.array_equal(vs, v[:5]) and np.array_equal(vr, v[5:])
    for t in range(T):
        p = t if t < 5 else t - 5
        want = np.array([[bf16_via_torch(x) for x in scalar_rope(list(k[t, h]), p, THETA)] for h in range(2)])
        got = (ks if t < 5 else kr)[p]
        assert np.array_equal(got, want)


def lse_merge(parts):
    """Exact combination of partial softmax states (m, l, O) over disjoint key sets."""
    m = max(p[0] for p in parts)
    l = sum(p[1] * math.exp(p[0] - m) for p in parts)
    o = sum(p[2] * (p[1] * math.exp(p[0] - m)) for p in parts) / l
    return o


def test_split_and_merge_equals_unsplit():
    rng = np.random.default_rng(13)
    nk, d = 50, 8
    z = rng.standard_normal(nk) * 4
    v = rng.standard_normal((nk, d))
    ref = osa.softmax_rows(z[None, :])[0] @ v
    for cuts in ([17], [1, 2, 49], [10, 20, 30, 40]):
        parts = []
        for lo, hi in zip([0] + cuts, cuts + [nk]):
            mm = z[lo:hi].max()
            w = np.exp(z[lo:hi] - mm)
            parts.append((mm, w.sum(), (w @ v[lo:hi]) / w.sum()))
        assert np.abs(lse_merge(parts) - ref).max() < 1e-12
