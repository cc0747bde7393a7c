"""ctypes binding over the C-ABI CUDA library (same names as include/streaming_thinker.h).

Argument marshalling only: every step of the path runs inside the library's kernels. Importing this
module fails loudly if the library has not been built (``python -m paper_2510_17238_b200.build``);
there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libstreaming_thinker.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build the CUDA library first (python -m paper_2510_17238_b200.build). "
        "This package has no CPU or PyTorch fallback.")
lib = C.CDLL(_LIB_PATH)

ST_OK, ST_ERR_INVALID_ARG, ST_ERR_OOM_PAGES, ST_ERR_NOT_READY = 0, -1, -2, -3
ST_ERR_STATE, ST_ERR_CUDA, ST_ERR_DEVICE_TIMEOUT, ST_ERR_DEVICE_CHECK = -4, -5, -6, -7
ST_CFG_HOST_ONLY, ST_CFG_DEBUG_CHECKS, ST_CFG_PRECISE_P = 1, 2, 4
ST_END_OF_UNIT, ST_REFERENCE_KERNELS, ST_IO_HOST = 1, 2, 4
ST_VIS_DEFAULT, ST_VIS_ALL = -1, -2
ST_POS_STREAMING, ST_POS_CONCATENATED, ST_POS_UNIT_ALIGNED = 0, 1, 2

ERROR_NAMES = {0: "ST_OK", -1: "ST_ERR_INVALID_ARG", -2: "ST_ERR_OOM_PAGES", -3: "ST_ERR_NOT_READY",
               -4: "ST_ERR_STATE", -5: "ST_ERR_CUDA", -6: "ST_ERR_DEVICE_TIMEOUT", -7: "ST_ERR_DEVICE_CHECK"}


class st_config(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("max_batch", C.c_int32), ("page_size", C.c_int32),
        ("n_pages_source", C.c_int64), ("n_pages_reason", C.c_int64),
        ("max_source_len", C.c_int32), ("max_reason_len", C.c_int32),
        ("max_tokens_per_call", C.c_int32), ("device", C.c_int32),
        ("pool_base", C.c_void_p), ("pool_bytes", C.c_uint64),
        ("rope_theta", C.c_double), ("softmax_scale", C.c_float), ("flags", C.c_uint32),
        ("position_mode", C.c_int32), ("reserved", C.c_int32),
        ("q_norm_weight", C.c_void_p), ("k_norm_weight", C.c_void_p), ("qk_norm_eps", C.c_float), ("reserved2", C.c_int32),
    ]


_i32p = C.POINTER(C.c_int32)
_i64p = C.POINTER(C.c_int64)
_vp = C.c_void_p

_SIGS = {
    "st_pool_bytes": (C.c_uint64, [C.POINTER(st_config)]),
    "st_create": (C.c_int, [C.POINTER(st_config), C.POINTER(_vp)]),
    "st_destroy": (C.c_int, [_vp]),
    "st_reset": (C.c_int, [_vp, _i32p, C.c_int32]),
    "st_append_source_chunk": (C.c_int, [_vp, C.c_int32, _i32p, _i32p, C.c_int32, _vp, _vp, _vp, _vp, C.c_uint32, _vp]),
    "st_reason_decode": (C.c_int, [_vp, C.c_int32, _i32p, C.c_int32, _i32p, _vp, _vp, _vp, _vp, C.c_uint32, _vp]),
    "st_reason_extend": (C.c_int, [_vp, C.c_int32, _i32p, _i32p, C.c_int32, _i32p, _vp, _vp, _vp, _vp, C.c_uint32, _vp]),
    "st_forward_packed": (C.c_int, [_vp, C.c_int32, _i32p, C.c_int32, _i32p, _i32p, _i32p, _i32p, C.c_int32, _vp, _vp, _vp, _vp,
                                    C.c_uint32, _vp]),
    "st_schedule_build": (C.c_int, [_i32p, _i32p, C.c_int32, C.c_int32, C.c_int32, _i32p, _i32p, _i64p, _i64p]),
    "st_schedule_dense_mask": (C.c_int, [_i32p, _i32p, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_uint8)]),
    "st_seq_state": (C.c_int, [_vp, C.c_int32, _i32p, _i32p, _i32p, _i32p]),
    "st_pages_free": (C.c_int, [_vp, _i64p, _i64p]),
    "st_debug_last_call_meta": (C.c_int, [_vp, _i32p, _i32p, _i32p, C.c_int32, _i32p]),
    "st_debug_read_cache": (C.c_int, [_vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _vp, _vp]),
    "st_debug_page_table": (C.c_int, [_vp, C.c_int32, C.c_int32, _i32p, C.c_int32, _i32p]),
    "st_device_status": (C.c_int, [_vp]),
    "st_debug_wait_expiry": (C.c_int, [_vp, C.c_int32, _vp]),
    "st_kernel_timing_enable": (C.c_int, [_vp, C.c_int32]),
    "st_kernel_timing_read": (C.c_int, [_vp, C.c_int32, _i64p, C.POINTER(C.c_double)]),
    "st_launch_count": (C.c_int64, [_vp]),
    "st_last_error_string": (C.c_char_p, [_vp]),
    "st_debug_fail_after": (C.c_int, [_vp, C.c_int32]),
    "st_debug_corrupt_page_table": (C.c_int, [_vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _vp]),
    "st_decode_attention_static": (C.c_int, [C.c_int32, _vp, C.c_int64, _vp, C.c_int64, _vp, C.c_int32, _vp, C.c_int32,
                                             _i32p, _i32p, _i32p, C.c_int32, _vp, _vp, C.c_int32, C.c_int32, C.c_float,
                                             _vp, C.c_char_p, C.c_int32]),
    "st_decode_static_status": (C.c_int, [C.c_int32, _vp]),
    "st_linear": (C.c_int, [C.c_int32, _vp, C.c_int64, C.c_int64, C.c_int64, _vp, C.c_int64, C.c_int64, _vp, C.c_int64,
                            C.c_int32, _vp, C.c_char_p, C.c_int32]),
    "st_linear_status": (C.c_int, [C.c_int32, _vp]),
    "st_cast_to_bf16": (C.c_int, [C.c_int32, _vp, _vp, C.c_int64, _vp]),
}
EXPORTED = tuple(_SIGS)
for _name, (_res, _args) in _SIGS.items():
    _fn = getattr(lib, _name)          # AttributeError here = the library does not export the symbol
    _fn.restype = _res
    _fn.argtypes = _args


class StError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"{ERROR_NAMES.get(code, code)}: {msg}")
        self.code = code


def _i32(a):
    """int32 ctypes pointer (and a keep-alive object) for a list / array, or NULL."""
    if a is None:
        return None, None
    arr = np.ascontiguousarray(a, dtype=np.int32)
    return arr.ctypes.data_as(_i32p), arr


def _ptr(x):
    """Raw address of a torch tensor / numpy array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    return x.ctypes.data


def st_pool_bytes(cfg: st_config) -> int:
    return int(lib.st_pool_bytes(C.byref(cfg)))


def make_config(n_layers=1, n_q_heads=16, n_kv_heads=8, max_batch=1, n_pages_source=0, n_pages_reason=0,
                max_source_len=0, max_reason_len=0, max_tokens_per_call=1, device=0, pool_base=None, pool_bytes=0,
                rope_theta=1.0e6, softmax_scale=0.0, flags=0, position_mode=0, qk_norm=None) -> st_config:
    """qk_norm: (weight_q, weight_k, eps) with float32 numpy arrays [n_layers, 128] (host), or None."""
    cfg = st_config(n_layers, n_q_heads, n_kv_heads, 128, max_batch, 64, n_pages_source, n_pages_reason,
                    max_source_len, max_reason_len, max_tokens_per_call, device, pool_base, pool_bytes,
                    rope_theta, softmax_scale, flags, position_mode, 0, None, None, 0.0, 0)
    if qk_norm is not None:
        wq = np.ascontiguousarray(qk_norm[0], dtype=np.float32).reshape(n_layers, 128)
        wk = np.ascontiguousarray(qk_norm[1], dtype=np.float32).reshape(n_layers, 128)
        cfg._keep = (wq, wk)                       # the library copies them in st_create; keep them alive until then
        cfg.q_norm_weight, cfg.k_norm_weight, cfg.qk_norm_eps = wq.ctypes.data, wk.ctypes.data, float(qk_norm[2])
    return cfg


class Context:
    """Thin owner of one ``st_ctx*``; methods mirror the C entry points one to one."""

    def __init__(self, cfg: st_config):
        self.cfg = cfg
        self._h = _vp()
        rc = lib.st_create(C.byref(cfg), C.byref(self._h))
        if rc != ST_OK:
            raise StError(rc, lib.st_last_error_string(None).decode())

    # -- helpers
    def _check(self, rc):
        if rc != ST_OK:
            raise StError(rc, lib.st_last_error_string(self._h).decode())
        return rc

    def close(self):
        if self._h:
            lib.st_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- C entry points
    def reset(self, seq_ids=None):
        p, keep = _i32(seq_ids)
        return self._check(lib.st_reset(self._h, p, 0 if seq_ids is None else len(keep)))

    def append_source_chunk(self, layer, seq_ids, cu_tokens, q, k, v, out, flags=0, stream=None, check=True):
        ps, ks = _i32(seq_ids)
        pc, kc = _i32(cu_tokens)
        rc = lib.st_append_source_chunk(self._h, layer, ps, pc, len(ks), _ptr(q), _ptr(k), _ptr(v), _ptr(out), flags,
                                        _ptr(stream))
        return self._check(rc) if check else rc

    def reason_decode(self, layer, seq_ids, visible_units, q, k, v, out, flags=0, stream=None, check=True):
        ps, ks = _i32(seq_ids)
        pv, kv = _i32(visible_units)
        rc = lib.st_reason_decode(self._h, layer, ps, len(ks), pv, _ptr(q), _ptr(k), _ptr(v), _ptr(out), flags,
                                  _ptr(stream))
        return self._check(rc) if check else rc

    def reason_extend(self, layer, seq_ids, cu_tokens, visible_units, q, k, v, out, flags=0, stream=None, check=True):
        ps, ks = _i32(seq_ids)
        pc, kc = _i32(cu_tokens)
        pv, kv = _i32(visible_units)
        rc = lib.st_reason_extend(self._h, layer, ps, pc, len(ks), pv, _ptr(q), _ptr(k), _ptr(v), _ptr(out), flags,
                                  _ptr(stream))
        return self._check(rc) if check else rc

    def forward_packed(self, layer, seq_ids, scheds, q, k, v, out, lag_units=0, flags=0, stream=None, check=True):
        """st_forward_packed for a list of schedules (objects with src_unit_len, rsn_unit_len, final_len)."""
        ps, ks = _i32(seq_ids)
        pn, kn = _i32([len(s.src_unit_len) for s in scheds])
        pa, ka = _i32([x for s in scheds for x in s.src_unit_len] or [0])
        pb, kb = _i32([x for s in scheds for x in s.rsn_unit_len] or [0])
        pf, kf = _i32([s.final_len for s in scheds])
        rc = lib.st_forward_packed(self._h, layer, ps, len(ks), pn, pa, pb, pf, lag_units, _ptr(q), _ptr(k), _ptr(v),
                                   _ptr(out), flags, _ptr(stream))
        return self._check(rc) if check else rc

    def seq_state(self, seq_id):
        a, b, c, d = C.c_int32(), C.c_int32(), C.c_int32(), C.c_int32()
        self._check(lib.st_seq_state(self._h, seq_id, C.byref(a), C.byref(b), C.byref(c), C.byref(d)))
        return {"source_len": a.value, "reason_len": b.value, "n_eos": c.value, "n_eot": d.value}

    def pages_free(self):
        a, b = C.c_int64(), C.c_int64()
        self._check(lib.st_pages_free(self._h, C.byref(a), C.byref(b)))
        return a.value, b.value

    def debug_last_call_meta(self):
        n = C.c_int32()
        self._check(lib.st_debug_last_call_meta(self._h, None, None, None, 0, C.byref(n)))
        pos = np.zeros(max(n.value, 1), np.int32)
        vs = np.zeros_like(pos)
        vr = np.zeros_like(pos)
        self._check(lib.st_debug_last_call_meta(self._h, pos.ctypes.data_as(_i32p), vs.ctypes.data_as(_i32p),
                                                vr.ctypes.data_as(_i32p), n.value, C.byref(n)))
        return pos[: n.value], vs[: n.value], vr[: n.value]

    def debug_read_cache(self, layer, seq_id, which, tok0, ntok):
        """Returns (k, v) as uint16 numpy arrays [ntok, n_kv_heads, 128] holding bf16 bit patterns."""
        k = np.zeros((ntok, self.cfg.n_kv_heads, 128), np.uint16)
        v = np.zeros_like(k)
        self._check(lib.st_debug_read_cache(self._h, layer, seq_id, which, tok0, ntok, k.ctypes.data, v.ctypes.data))
        return k, v

    def debug_page_table(self, seq_id, which):
        n = C.c_int32()
        self._check(lib.st_debug_page_table(self._h, seq_id, which, None, 0, C.byref(n)))
        pages = np.zeros(max(n.value, 1), np.int32)
        self._check(lib.st_debug_page_table(self._h, seq_id, which, pages.ctypes.data_as(_i32p), n.value, C.byref(n)))
        return pages[: n.value]

    def device_status(self, check=True):
        rc = lib.st_device_status(self._h)
        return self._check(rc) if check else rc

    def debug_wait_expiry(self, limit_ms, stream=None, check=True):
        rc = lib.st_debug_wait_expiry(self._h, int(limit_ms), _ptr(stream))
        return self._check(rc) if check else rc

    def debug_fail_after(self, n_steps):
        return self._check(lib.st_debug_fail_after(self._h, int(n_steps)))

    def debug_corrupt_page_table(self, seq_id, which, index, page, stream=None):
        return self._check(lib.st_debug_corrupt_page_table(self._h, seq_id, which, index, page, _ptr(stream)))

    def kernel_timing_enable(self, every=1):
        """Bracket every `every`-th launch of the two dominant kernels with CUDA events (0 / False = off)."""
        return self._check(lib.st_kernel_timing_enable(self._h, int(every)))

    def kernel_timing_read(self, which):
        """(launches, total milliseconds) of the decode kernel (0) or the tensor-core attention kernel (1)."""
        n, ms = C.c_int64(), C.c_double()
        self._check(lib.st_kernel_timing_read(self._h, which, C.byref(n), C.byref(ms)))
        return n.value, ms.value

    def launch_count(self) -> int:
        return int(lib.st_launch_count(self._h))

    def last_error(self) -> str:
        return lib.st_last_error_string(self._h).decode()

    @property
    def handle(self):
        return self._h


def schedule_build(src_unit_len, rsn_unit_len, final_len=0, lag_units=0):
    ps, ks = _i32(src_unit_len)
    pr, kr = _i32(rsn_unit_len)
    S, R = C.c_int64(), C.c_int64()
    rc = lib.st_schedule_build(ps, pr, len(ks), final_len, lag_units, None, None, C.byref(S), C.byref(R))
    if rc != ST_OK:
        raise StError(rc, "st_schedule_build")
    pos = np.zeros(max(S.value + R.value, 1), np.int32)
    vis = np.zeros(max(R.value, 1), np.int32)
    rc = lib.st_schedule_build(ps, pr, len(ks), final_len, lag_units, pos.ctypes.data_as(_i32p),
                               vis.ctypes.data_as(_i32p), None, None)
    if rc != ST_OK:
        raise StError(rc, "st_schedule_build")
    return pos[: S.value + R.value], vis[: R.value], S.value, R.value


def schedule_dense_mask(src_unit_len, rsn_unit_len, final_len=0, lag_units=0):
    ps, ks = _i32(src_unit_len)
    pr, kr = _i32(rsn_unit_len)
    S, R = C.c_int64(), C.c_int64()
    rc = lib.st_schedule_build(ps, pr, len(ks), final_len, lag_units, None, None, C.byref(S), C.byref(R))
    if rc != ST_OK:
        raise StError(rc, "st_schedule_build")
    T = S.value + R.value
    mask = np.zeros((max(T, 1), max(T, 1)), np.uint8)
    rc = lib.st_schedule_dense_mask(ps, pr, len(ks), final_len, lag_units, mask.ctypes.data_as(C.POINTER(C.c_uint8)))
    if rc != ST_OK:
        raise StError(rc, "st_schedule_dense_mask")
    return mask[:T, :T]


def decode_attention_static(device, pool_source, n_pages_source, pool_reason, n_pages_reason, page_table_source,
                            table_stride_source, page_table_reason, table_stride_reason, slots, source_len, reason_len,
                            q_rotated, out, n_q_heads, n_kv_heads, softmax_scale=0.0, stream=None, check=True):
    """st_decode_attention_static: decode attention on the workspace built into the library (no allocation).

    Pointers may be torch tensors, numpy arrays or raw addresses; slots / source_len / reason_len are host
    int sequences. Returns the status code (raises StError with the library's message when check is set)."""
    ps, ks = _i32(slots)
    pa, ka = _i32(source_len)
    pr, kr = _i32(reason_len)
    err = C.create_string_buffer(256)
    rc = lib.st_decode_attention_static(device, _ptr(pool_source), n_pages_source, _ptr(pool_reason), n_pages_reason,
                                        _ptr(page_table_source), table_stride_source, _ptr(page_table_reason),
                                        table_stride_reason, ps, pa, pr, len(ks), _ptr(q_rotated), _ptr(out), n_q_heads,
                                        n_kv_heads, softmax_scale, _ptr(stream), err, 256)
    if rc != ST_OK and check:
        raise StError(rc, err.value.decode())
    return rc, err.value.decode()


def decode_static_status(device, stream=None) -> int:
    """st_decode_static_status: status code of the most recent allocation-free decode call on the device."""
    return int(lib.st_decode_static_status(device, _ptr(stream)))


def linear(device, x, m, k, ldx, w, n, ldw, y, ldy, out_fp32=False, stream=None, check=True):
    """st_linear: y[m, n] = x[m, k] w[n, k]^T on the tensor cores (pointers: torch tensors, arrays or addresses)."""
    err = C.create_string_buffer(256)
    rc = lib.st_linear(device, _ptr(x), m, k, ldx, _ptr(w), n, ldw, _ptr(y), ldy, 1 if out_fp32 else 0, _ptr(stream), err, 256)
    if rc != ST_OK and check:
        raise StError(rc, err.value.decode())
    return rc, err.value.decode()


def linear_status(device, stream=None) -> int:
    return int(lib.st_linear_status(device, _ptr(stream)))


def cast_to_bf16(device, src, dst, n, stream=None) -> int:
    return int(lib.st_cast_to_bf16(device, _ptr(src), _ptr(dst), n, _ptr(stream)))
