"""fp64 oracle: attention under the streaming mask and streaming position ids.

TEST INFRASTRUCTURE ONLY (see the package docstring). Plain numpy, fp64.

Layout used throughout is the paper's *training* layout (Section 3.2): one
sequence is the concatenation ``[all source tokens ; all reasoning tokens]`` of
length ``S + R``; the dense ``(S+R) x (S+R)`` mask and the position ids are
materialised and ordinary masked softmax attention is evaluated on them. The
two-cache inference procedure (Section 3.3, Algorithm 1) must produce exactly
these rows: source rows when a chunk is appended, reasoning rows when reasoning
tokens are decoded.

Readings taken where the paper is silent or ambiguous (each is also exercised by
a test):

* Visibility is unit-level (Eq. 1 and the ``N_EOS == N_EOT + 1`` rule of
  Algorithm 1): every token of reasoning unit ``u`` (1-based) may attend to the
  source tokens of units ``1..u`` and to nothing later. Eq. 2 is the
  one-token-per-unit special case and, read literally, is shifted by one unit;
  ``lag_units=1`` reproduces that literal reading.
* Final-depth reasoning tokens (the last factor of Eq. 1) see the whole source.
* Position ids (Section 3.2, streaming position encoding): two running
  counters, one per stream, both starting at zero and never reset; final-depth
  tokens continue the reasoning counter.
* The diagonal is visible (a token attends to itself), as in the ordinary
  causal mask that Eq. 2 starts from.
* RoPE uses the half-split pairing (channel ``c`` with ``c + d/2``) and
  ``inv_freq[c] = theta ** (-2c/d)``.
* Optional (outside the paper's method, part of its Qwen3 backbones): queries and keys
  are RMS-normalised per head before the rotation.
* The caches hold bf16 values, so rotated keys are rounded to bf16
  (round-to-nearest-even) after the fp64 rotation, and rotated queries enter
  the contraction as bf16 too. ``round_rotated=False`` disables both roundings.
  Nothing else is rounded.

Pins (tests/test_oracle_*.py): a scalar triple-loop attention written apart from
this file, reduction to ordinary causal attention, softmax row sums, invariance
of source rows to reasoning tokens, Eq. 1's conditioning sets, Eq. 2's
indicator, closed-form position ids, RoPE's relative-position property and
torch's bf16 conversion for ``round_to_bf16``.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


# --------------------------------------------------------------------------- schedule


@dataclass(frozen=True)
class Schedule:
    """Streaming-unit schedule of one sequence and everything derived from it."""

    src_unit_len: np.ndarray  # [U] tokens of source unit u (u = 1..U)
    rsn_unit_len: np.ndarray  # [U] tokens of reasoning unit u
    final_len: int            # final-depth reasoning tokens after the last unit
    lag_units: int            # extra source units visible to a reasoning unit
    S: int                    # total source tokens
    R: int                    # total reasoning tokens
    src_prefix: np.ndarray    # [U+1] P_u = sum_{u' <= u} n_{u'}, P_0 = 0
    pos_ids: np.ndarray       # [S+R] int32, streaming position ids
    vis_len: np.ndarray       # [R] int32, visible source prefix of reasoning token r
    rsn_unit: np.ndarray      # [R] int32, unit of reasoning token r (U+1 = final depth)


POSITION_MODES = ("streaming", "concatenated", "unit_aligned")


def build_schedule(src_unit_len, rsn_unit_len, final_len=0, lag_units=0, position_mode="streaming") -> Schedule:
    """Eq. 1 / Algorithm 1 (visibility) and the position ids (Section 3.2).

    Reasoning unit ``u`` is produced while ``N_EOS == N_EOT + 1 == u``, i.e. when
    exactly the first ``u`` source units are in the (sliced) source cache, so its
    tokens see the source prefix ``P_u``. ``lag_units`` shifts that to
    ``P_{min(u + lag, U)}``.

    ``position_mode`` (source tokens always count from zero):

    * ``"streaming"``: the streaming position encoding -- reasoning tokens count from
      zero on a counter of their own (the method's encoding);
    * ``"concatenated"``: the original RoPE ids that Section 3.2 starts from -- the
      reasoning token with index ``t`` gets ``T + t``, ``T`` the input length (the
      "RoPE" rows of the batch-setting comparison);
    * ``"unit_aligned"``: a variant of this build, not the paper's: the ``i``-th token
      of reasoning unit ``u`` gets ``P_{u-1} + i``, i.e. every reasoning unit restarts at
      the position where its source unit starts; final-depth tokens get ``S + i``.
    """
    if position_mode not in POSITION_MODES:
        raise ValueError(f"position_mode must be one of {POSITION_MODES}")
    n = np.asarray(src_unit_len, dtype=np.int64).reshape(-1)
    m = np.asarray(rsn_unit_len, dtype=np.int64).reshape(-1)
    if n.shape != m.shape:
        raise ValueError("one reasoning-unit length per source unit is required")
    if (n < 0).any() or (m < 0).any() or final_len < 0:
        raise ValueError("lengths must be non-negative")
    U = n.shape[0]
    P = np.zeros(U + 1, dtype=np.int64)
    for u in range(1, U + 1):
        P[u] = P[u - 1] + n[u - 1]
    S = int(P[U])
    R = int(m.sum() + final_len)

    pos = np.empty(S + R, dtype=np.int32)
    for j in range(S):          # source counter starts at zero
        pos[j] = j
    if position_mode == "streaming":
        for r in range(R):      # reasoning counter starts at zero too
            pos[S + r] = r
    elif position_mode == "concatenated":
        for r in range(R):      # one counter over [input ; reasoning]
            pos[S + r] = S + r
    else:
        r = 0
        for u in range(1, U + 1):
            for i in range(int(m[u - 1])):
                pos[S + r] = P[u - 1] + i
                r += 1
        for i in range(int(final_len)):
            pos[S + r] = S + i
            r += 1

    vis = np.empty(R, dtype=np.int32)
    unit = np.empty(R, dtype=np.int32)
    r = 0
    for u in range(1, U + 1):
        seen = min(u + lag_units, U)
        for _ in range(int(m[u - 1])):
            vis[r] = P[seen]
            unit[r] = u
            r += 1
    for _ in range(int(final_len)):
        vis[r] = S
        unit[r] = U + 1
        r += 1
    assert r == R
    return Schedule(n, m, int(final_len), int(lag_units), S, R, P, pos, vis, unit)


def mask_rows(sched: Schedule, rows) -> np.ndarray:
    """Rows of the dense streaming mask, 1 = may attend (Eq. 2 on top of causal).

    Row/column index ``i < S`` is source token ``i``; index ``S + r`` is
    reasoning token ``r``.
    """
    S, R = sched.S, sched.R
    rows = np.asarray(rows, dtype=np.int64).reshape(-1)
    A = np.zeros((rows.shape[0], S + R), dtype=np.uint8)
    for a, i in enumerate(rows):
        if i < S:
            # source row: the ordinary causal mask; every reasoning column lies
            # after every source column in the layout, so none is reachable.
            A[a, : i + 1] = 1
        else:
            r = i - S
            A[a, : sched.vis_len[r]] = 1          # streaming mask region
            A[a, S : S + r + 1] = 1               # causal over reasoning tokens
    return A


def dense_mask(sched: Schedule) -> np.ndarray:
    return mask_rows(sched, np.arange(sched.S + sched.R))


# --------------------------------------------------------------------------- arithmetic


def rope_inv_freq(d: int, theta: float) -> np.ndarray:
    c = np.arange(d // 2, dtype=np.float64)
    return np.float64(theta) ** (-2.0 * c / d)


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding of ``x[..., d]`` at integer positions ``pos`` (half-split pairs).

    ``x`` has shape ``[T, H, d]`` and ``pos`` shape ``[T]``.
    """
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    ang = np.asarray(pos, dtype=np.float64)[:, None] * rope_inv_freq(d, theta)[None, :]
    cos = np.cos(ang)[:, None, :]
    sin = np.sin(ang)[:, None, :]
    lo, hi = x[..., : d // 2], x[..., d // 2 :]
    return np.concatenate([lo * cos - hi * sin, hi * cos + lo * sin], axis=-1)


def qk_rmsnorm(x: np.ndarray, weight: np.ndarray, eps: float) -> np.ndarray:
    """Per-head RMS normalisation of queries or keys over the head dimension, as the Qwen3
    backbones of Section 4.1 apply it before the rotary embedding:
    ``x / sqrt(mean(x**2) + eps) * weight`` with ``x [T, H, d]`` and ``weight [d]``."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(weight, dtype=np.float64).reshape(-1)
    if w.shape[0] != x.shape[-1]:
        raise ValueError("one weight per channel of a head is required")
    ms = (x * x).mean(axis=-1, keepdims=True)
    return x / np.sqrt(ms + float(eps)) * w


def linear(x: np.ndarray, weight: np.ndarray, round_out: bool = False) -> np.ndarray:
    """Projection ``y = x W^T`` of the attention block around the path (Q, K, V and output
    projections of the Qwen3 backbones; not part of the paper's method): ``x [T, K]``,
    ``weight [N, K]`` (one row per output feature), fp64. ``round_out`` rounds the result to
    bf16, which is what feeds the attention calls (their q/k/v are bf16)."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(weight, dtype=np.float64)
    if x.ndim != 2 or w.ndim != 2 or x.shape[1] != w.shape[1]:
        raise ValueError("x [T, K] and weight [N, K] are required")
    y = x @ w.T
    return round_to_bf16(y) if round_out else y


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest bf16 value (ties to even) of each fp64 element, returned as fp64.

    bf16 keeps 8 significant bits. Values are assumed to lie in bf16's normal
    range or to be zero (true for every workload here).
    """
    x = np.asarray(x, dtype=np.float64)
    mant, expo = np.frexp(x)                 # x = mant * 2**expo, 0.5 <= |mant| < 1
    return np.ldexp(np.rint(mant * 256.0), expo - 8)   # rint rounds ties to even


def softmax_rows(z: np.ndarray) -> np.ndarray:
    zmax = z.max(axis=-1, keepdims=True)
    e = np.exp(z - zmax)
    return e / e.sum(axis=-1, keepdims=True)


# --------------------------------------------------------------------------- attention


def rotate_and_round(sched: Schedule, q, k, theta: float, round_rotated: bool = True, qk_norm=None):
    """Steps 1 and 3: (optional q/k normalisation ->) position ids -> RoPE -> the two bf16 rounding points.

    ``qk_norm = (weight_q, weight_k, eps)`` applies ``qk_rmsnorm`` to q and k first; there is no rounding
    between the normalisation and the rotation (the fused form: one rounding, after the rotation)."""
    if qk_norm is not None:
        wq, wk, eps = qk_norm
        q = qk_rmsnorm(q, wq, eps)
        k = qk_rmsnorm(k, wk, eps)
    qh = rope(q, sched.pos_ids, theta)
    kh = rope(k, sched.pos_ids, theta)
    if round_rotated:
        qh = round_to_bf16(qh)
        kh = round_to_bf16(kh)
    return qh, kh


def attention_rows(sched: Schedule, q, k, v, rows, theta: float = 1.0e6, scale=None,
                   round_rotated: bool = True, row_block: int = 256,
                   return_probs: bool = False, rotated=None, qk_norm=None):
    """Masked softmax attention for the listed rows of ``[source ; reasoning]``.

    q: ``[S+R, Hq, d]``; k, v: ``[S+R, Hkv, d]`` (un-rotated, any float dtype).
    Returns ``O[len(rows), Hq, d]`` in fp64 (and the probabilities
    ``[len(rows), Hq, S+R]`` when asked). ``rotated`` may carry the result of
    ``rotate_and_round`` so that several row sets share one rotation.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    if T != sched.S + sched.R or k.shape[0] != T or v.shape != k.shape:
        raise ValueError("tensor lengths do not match the schedule")
    if Hq % Hkv:
        raise ValueError("n_q_heads must be a multiple of n_kv_heads")
    G = Hq // Hkv
    s = (1.0 / np.sqrt(d)) if scale is None else float(scale)
    rows = np.asarray(rows, dtype=np.int64).reshape(-1)

    qh, kh = rotated if rotated is not None else rotate_and_round(sched, q, k, theta, round_rotated, qk_norm)

    O = np.empty((rows.shape[0], Hq, d), dtype=np.float64)
    probs = np.empty((rows.shape[0], Hq, T), dtype=np.float64) if return_probs else None
    for b0 in range(0, rows.shape[0], row_block):
        blk = rows[b0 : b0 + row_block]
        A = mask_rows(sched, blk)                              # [nb, T]
        for h in range(Hq):
            Z = s * (qh[blk, h, :] @ kh[:, h // G, :].T)       # [nb, T]
            Z = np.where(A != 0, Z, -np.inf)
            Pm = softmax_rows(Z)
            O[b0 : b0 + blk.shape[0], h, :] = Pm @ v[:, h // G, :]
            if return_probs:
                probs[b0 : b0 + blk.shape[0], h, :] = Pm
    return (O, probs) if return_probs else O


def expected_cache(sched: Schedule, k, v, theta: float = 1.0e6, k_norm=None):
    """What the two caches must hold: ``bf16(RoPE(k, pos))`` and ``v``, split by stream
    (``k_norm = (weight_k, eps)``: keys normalised first)."""
    if k_norm is not None:
        k = qk_rmsnorm(k, k_norm[0], k_norm[1])
    kh = round_to_bf16(rope(k, sched.pos_ids, theta))
    v = np.asarray(v, dtype=np.float64)
    S = sched.S
    return (kh[:S], v[:S]), (kh[S:], v[S:])
