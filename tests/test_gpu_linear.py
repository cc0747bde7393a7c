"""GPU parity of the projection kernel (st_linear) against the oracle's linear, and of a whole attention block
(Q/K/V projections -> source append with chunk prefill -> output projection) against the oracle's composition.

Tolerances. st_linear multiplies bf16 operands exactly and accumulates in fp32: against the fp64 product the fp32
output must agree to 1e-5 of the largest |y| of the case (K <= 2560 terms of order 1/sqrt(K)); the bf16 output adds
one rounding, so every element must be within 2^-8 of its own magnitude plus that slack. The block ends in attention
rows, which keep the tolerance of the other parity tests (max abs <= 1e-2, relative L2 <= 5e-3)."""
import numpy as np
import pytest
import torch

from oracle import streaming_attention as osa
from paper_2510_17238_b200 import api, workloads

import parity_util as pu

pytestmark = pytest.mark.gpu


def bf16_tensor(rng, shape, scale):
    return torch.from_numpy((rng.standard_normal(shape) * scale).astype(np.float32)).to(torch.bfloat16)


@pytest.mark.parametrize("m,n,k,pad", [(128, 256, 64, 0), (1, 8, 8, 0), (300, 1000, 520, 8), (4096, 1024, 2560, 0),
                                       (129, 264, 72, 16), (777, 4096, 1024, 0)])
def test_linear_matches_the_oracle(m, n, k, pad):
    rng = np.random.default_rng([m, n, k])
    dev = torch.device("cuda", 0)
    ldx, ldw = k + pad, k + pad
    x = torch.zeros((m, ldx), dtype=torch.bfloat16)
    w = torch.zeros((n, ldw), dtype=torch.bfloat16)
    x[:, :k] = bf16_tensor(rng, (m, k), 1.0)
    w[:, :k] = bf16_tensor(rng, (n, k), 1.0 / np.sqrt(k))
    if pad:                                                     # what lies beyond a row's end must not be read into the product
        x[:, k:] = 1000.0
        w[:, k:] = 1000.0
    want = osa.linear(x[:, :k].double().numpy(), w[:, :k].double().numpy())
    xd, wd = x.to(dev), w.to(dev)
    stream = torch.cuda.current_stream().cuda_stream
    for out_fp32 in (True, False):
        ldy = n + (8 if pad else 0)
        y = torch.full((m, ldy), float("nan"), dtype=torch.float32 if out_fp32 else torch.bfloat16, device=dev)
        api.linear(0, xd, m, k, ldx, wd, n, ldw, y, ldy, out_fp32=out_fp32, stream=stream)
        assert api.linear_status(0, stream) == api.ST_OK
        got = y[:, :n].double().cpu().numpy()
        assert not np.isnan(got).any()
        if pad:
            assert torch.isnan(y[:, n:].float()).all(), "columns beyond n must not be written"
        slack = 1e-5 * np.abs(want).max()
        if out_fp32:
            assert np.abs(got - want).max() <= slack
        else:
            assert (np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + slack).all()


def test_attention_block_projections_prefill_output_projection():
    """x -> (Wq, Wk, Wv) -> st_append_source_chunk (two chunks) -> cast -> Wo, every step in the library's kernels,
    against the oracle: linear with bf16-rounded outputs, attention_rows, linear."""
    rng = np.random.default_rng(77)
    dev = torch.device("cuda", 0)
    hidden, Hq, Hkv, T = 512, 16, 8, 200
    chunks = (137, 63)
    x = bf16_tensor(rng, (T, hidden), 1.0)
    wq = bf16_tensor(rng, (Hq * 128, hidden), 1.0 / np.sqrt(hidden))
    wk = bf16_tensor(rng, (Hkv * 128, hidden), 1.0 / np.sqrt(hidden))
    wv = bf16_tensor(rng, (Hkv * 128, hidden), 1.0 / np.sqrt(hidden))
    wo = bf16_tensor(rng, (hidden, Hq * 128), 1.0 / np.sqrt(Hq * 128))
    stream = torch.cuda.current_stream().cuda_stream
    xd = x.to(dev)
    q = torch.empty((T, Hq, 128), dtype=torch.bfloat16, device=dev)
    k = torch.empty((T, Hkv, 128), dtype=torch.bfloat16, device=dev)
    v = torch.empty((T, Hkv, 128), dtype=torch.bfloat16, device=dev)
    for wt, dst, H in ((wq, q, Hq), (wk, k, Hkv), (wv, v, Hkv)):
        api.linear(0, xd, T, hidden, hidden, wt.to(dev), H * 128, hidden, dst, H * 128, stream=stream)
    cfg = api.make_config(n_q_heads=Hq, n_kv_heads=Hkv, max_batch=1, n_pages_source=4, n_pages_reason=1, max_tokens_per_call=T)
    ctx = api.Context(cfg)
    attn = torch.full((T, Hq, 128), float("nan"), dtype=torch.float32, device=dev)
    t0 = 0
    for n in chunks:
        sl = slice(t0, t0 + n)
        ctx.append_source_chunk(0, [0], [0, n], q[sl], k[sl], v[sl], attn[sl], api.ST_END_OF_UNIT, stream)
        t0 += n
    attn_bf16 = torch.empty((T, Hq * 128), dtype=torch.bfloat16, device=dev)
    assert api.cast_to_bf16(0, attn, attn_bf16, T * Hq * 128, stream) == api.ST_OK
    y = torch.empty((T, hidden), dtype=torch.float32, device=dev)
    api.linear(0, attn_bf16, T, Hq * 128, Hq * 128, wo.to(dev), hidden, Hq * 128, y, hidden, out_fp32=True, stream=stream)
    assert api.linear_status(0, stream) == api.ST_OK
    ctx.device_status()

    xf = x.double().numpy()
    qo = osa.linear(xf, wq.double().numpy(), round_out=True).reshape(T, Hq, 128)
    ko = osa.linear(xf, wk.double().numpy(), round_out=True).reshape(T, Hkv, 128)
    vo = osa.linear(xf, wv.double().numpy(), round_out=True).reshape(T, Hkv, 128)
    sched = osa.build_schedule(list(chunks), [0, 0], 0)
    rows = osa.attention_rows(sched, qo, ko, vo, np.arange(T))
    want_attn = rows.reshape(T, Hq * 128)
    pu.compare(attn.reshape(T, Hq * 128).cpu().numpy(), want_attn, "attention rows of the block")
    want = osa.linear(osa.round_to_bf16(want_attn), wo.double().numpy())
    pu.compare(y.cpu().numpy(), want, "output projection of the block")
    ctx.close()
