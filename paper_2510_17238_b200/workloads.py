"""Seeded synthetic workloads: streaming-unit schedules and bf16 Q/K/V tensors.

This module holds no attention arithmetic. It only draws unit lengths and
random tensors, so both the CUDA path and the CPU oracle can be fed the same
inputs without sharing any of the method's code. It needs numpy and torch (CPU)
and never touches the CUDA library.

Five workloads ("configs") are defined, indexed 0..4:

0. 16 q / 8 kv heads, batch 1: 4 units of (32 source, 16 reasoning) tokens, 64 final-depth tokens.
1. 16 / 8, batch 8: 16 units of (64, 48), 256 final-depth tokens.
2. 32 / 8, batch 32: 32 units of (128, 64), 6144 final-depth tokens (4096 source, 8192 reasoning).
3. 32 / 8, batch 64, 36 layers, ragged: 32 units per sequence, source unit length
   ``clip(round(LogNormal(ln 48 - 0.18, 0.6)), 8, 256)``, reasoning unit length uniform on 0..128.
4. 40 / 8, batch 16, long context: source units drawn as in 3 with mean 96 until 32768
   tokens (last unit truncated), reasoning unit ``floor(3 n / 8)``, the remainder of 16384
   reasoning tokens as final depth; 1 % of the (head, channel) pairs of each of Q, K, V
   are multiplied by 8 before rounding to bf16.

All tensors are i.i.d. N(0,1) rounded to bf16, head_dim 128, RoPE theta 1e6, page size 64.
Every tensor is drawn from ``numpy.random.default_rng([seed, config, layer, seq, tensor])`` so any
(layer, sequence) slice can be regenerated alone.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch

HEAD_DIM = 128
PAGE_SIZE = 64
ROPE_THETA = 1.0e6


@dataclass(frozen=True)
class Workload:
    index: int
    name: str
    n_q_heads: int
    n_kv_heads: int
    batch: int
    n_layers: int = 1
    head_dim: int = HEAD_DIM
    page_size: int = PAGE_SIZE
    rope_theta: float = ROPE_THETA
    outlier_frac: float = 0.0
    outlier_mult: float = 1.0
    two_streams: bool = False


WORKLOADS = (
    Workload(0, "cfg0-qwen3-0.6b-b1-4x(32,16)+64", 16, 8, 1),
    Workload(1, "cfg1-qwen3-1.7b-b8-16x(64,48)+256", 16, 8, 8),
    Workload(2, "cfg2-qwen3-4b-b32-32x(128,64)+6144", 32, 8, 32, two_streams=True),
    Workload(3, "cfg3-qwen3-8b-b64-36layers-ragged", 32, 8, 64, n_layers=36),
    Workload(4, "cfg4-qwen3-14b-b16-32k-source-16k-reasoning-outliers", 40, 8, 16,
             outlier_frac=0.01, outlier_mult=8.0),
)


@dataclass(frozen=True)
class SeqSchedule:
    """Unit lengths of one sequence: source unit u, reasoning unit u, final-depth tokens."""
    src_unit_len: tuple
    rsn_unit_len: tuple
    final_len: int

    @property
    def S(self) -> int:
        return int(sum(self.src_unit_len))

    @property
    def R(self) -> int:
        return int(sum(self.rsn_unit_len)) + int(self.final_len)


def _lognormal_units(rng, mean: float, sigma: float = 0.6, lo: int = 8, hi: int = 256, count=None, total=None):
    mu = math.log(mean) - 0.5 * sigma * sigma
    out = []
    if count is not None:
        draws = rng.lognormal(mu, sigma, size=count)
        return [int(min(max(round(float(x)), lo), hi)) for x in draws]
    acc = 0
    while acc < total:
        n = int(min(max(round(float(rng.lognormal(mu, sigma))), lo), hi))
        n = min(n, total - acc)
        out.append(n)
        acc += n
    return out


def schedules(index: int, seed: int = 0, batch=None) -> list:
    """One ``SeqSchedule`` per sequence of workload ``index``."""
    w = WORKLOADS[index]
    B = w.batch if batch is None else batch
    out = []
    for b in range(B):
        if index == 0:
            out.append(SeqSchedule((32,) * 4, (16,) * 4, 64))
        elif index == 1:
            out.append(SeqSchedule((64,) * 16, (48,) * 16, 256))
        elif index == 2:
            out.append(SeqSchedule((128,) * 32, (64,) * 32, 6144))
        elif index == 3:
            rng = np.random.default_rng([seed, index, b, 1000])
            n = _lognormal_units(rng, 48.0, count=32)
            m = [int(x) for x in rng.integers(0, 129, size=32)]
            out.append(SeqSchedule(tuple(n), tuple(m), 0))
        elif index == 4:
            rng = np.random.default_rng([seed, index, b, 1000])
            n = _lognormal_units(rng, 96.0, total=32768)
            m = [(3 * x) // 8 for x in n]
            out.append(SeqSchedule(tuple(n), tuple(m), 16384 - sum(m)))
        else:
            raise IndexError(index)
    return out


def scaled_schedule(n_units: int, n_src: int, n_rsn: int, final_len: int) -> SeqSchedule:
    """A uniform schedule of arbitrary size (used by small parity cases)."""
    return SeqSchedule((n_src,) * n_units, (n_rsn,) * n_units, final_len)


_TENSOR_ID = {"q": 0, "k": 1, "v": 2}


def _draw(seed, index, layer, seq, name, T, H, d, w: Workload) -> torch.Tensor:
    rng = np.random.default_rng([seed, index, layer, seq, _TENSOR_ID[name]])
    x = rng.standard_normal((T, H, d), dtype=np.float32)
    if w.outlier_frac > 0.0:
        # the outlier (head, channel) pairs are fixed per sequence and tensor kind
        orng = np.random.default_rng([seed, index, 0, seq, 100 + _TENSOR_ID[name]])
        n_out = int(math.ceil(w.outlier_frac * H * d))
        flat = orng.choice(H * d, size=n_out, replace=False)
        x.reshape(T, H * d)[:, flat] *= np.float32(w.outlier_mult)
    return torch.from_numpy(x).to(torch.bfloat16)


def qkv(index: int, sched: SeqSchedule, seq: int, layer: int = 0, seed: int = 0, workload=None):
    """bf16 tensors of one (layer, sequence) in the ``[source ; reasoning]`` layout.

    Returns ``q [S+R, Hq, d]``, ``k [S+R, Hkv, d]``, ``v [S+R, Hkv, d]`` (torch, CPU, bf16).
    """
    w = WORKLOADS[index] if workload is None else workload
    T = sched.S + sched.R
    q = _draw(seed, index, layer, seq, "q", T, w.n_q_heads, w.head_dim, w)
    k = _draw(seed, index, layer, seq, "k", T, w.n_kv_heads, w.head_dim, w)
    v = _draw(seed, index, layer, seq, "v", T, w.n_kv_heads, w.head_dim, w)
    return q, k, v
