"""ctypes binding of ``libisv.so`` (declared in ``include/isv.h``).

Argument marshalling only: every function here forwards to the C entry point
of the same name; all computation happens in the library's CUDA kernels.
Pointers may be given as torch tensors (``data_ptr()``), numpy arrays or ints.
Loading fails loudly if the library has not been built
(``python -m paper_2504_11816_b200.build``); there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libisv.so")

ISV_OK = 0
ISV_EINVAL = -1
ISV_ENOMEM_DEVICE = -2
ISV_ENOMEM_PINNED = -3
ISV_ECAPACITY = -4
ISV_ECUDA = -5
ISV_ETIMEOUT = -6
ISV_EDEVICE_STATUS = -7
ISV_ENODEVICE = -8
ISV_F16 = 0
ISV_BF16 = 1
ISV_BLOCK_NONE = -1
ISV_BLOCK_HOST_BIT = 1 << 30
ISV_STATUS_BAD_BLOCK_ID = 1
ISV_STATUS_WAIT_EXPIRED = 2
ISV_STATUS_BAD_LENGTH = 4

EXPORTS = [
    "isv_kv_alloc", "isv_kv_free", "isv_kv_reset", "isv_kv_info", "isv_kv_fill", "isv_kv_fill_async",
    "isv_fill_timing", "isv_kv_append",
    "isv_attn_decode", "isv_decode_layer", "isv_decode_step", "isv_decode_step_host", "isv_kv_gather",
    "isv_block_table_dev", "isv_seq_lens_dev", "isv_block_table_host", "isv_seq_lens_host",
    "isv_plan_bytes", "isv_set_zero_copy", "isv_set_timing", "isv_step_timing", "isv_sync", "isv_link_probe",
    "isv_set_host_timeout", "isv_set_wait_limit", "isv_inject_lost_copy",
    "isv_attn_decode_static", "isv_linear_create", "isv_linear_forward", "isv_linear_status", "isv_linear_free",
    "isv_last_error",
]


class IsvError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"isv error {code}: {message}")
        self.code = code
        self.message = message


class KvDesc(ctypes.Structure):
    _fields_ = [
        ("layers", ctypes.c_int32), ("phys_layers", ctypes.c_int32),
        ("q_heads", ctypes.c_int32), ("kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("block_tokens", ctypes.c_int32), ("dtype", ctypes.c_int32), ("offload_frac", ctypes.c_float),
        ("max_seqs", ctypes.c_int32), ("max_tokens_per_seq", ctypes.c_int32),
        ("perm_seed", ctypes.c_uint64), ("chunk_bytes", ctypes.c_uint64),
        ("ring_depth", ctypes.c_int32), ("max_ctas", ctypes.c_int32), ("plan_only", ctypes.c_int32),
        ("compute_stream", ctypes.c_void_p),
    ]


class KvInfo(ctypes.Structure):
    _fields_ = [
        ("block_bytes", ctypes.c_uint64), ("kv_bytes_per_token", ctypes.c_uint64),
        ("max_blocks_per_seq", ctypes.c_int32), ("hbm_blocks", ctypes.c_int32),
        ("host_blocks", ctypes.c_int32), ("hbm_blocks_used", ctypes.c_int32),
        ("host_blocks_used", ctypes.c_int32),
        ("hbm_pool_bytes", ctypes.c_uint64), ("host_pool_bytes", ctypes.c_uint64),
        ("scratch_bytes", ctypes.c_uint64),
        ("phys_layers", ctypes.c_int32), ("max_ctas", ctypes.c_int32),
        ("ring_depth", ctypes.c_int32), ("sm_count", ctypes.c_int32),
        ("chunk_bytes", ctypes.c_uint64), ("kernel_launches", ctypes.c_uint64),
    ]


class StepTimes(ctypes.Structure):
    _fields_ = [
        ("append_ms", ctypes.c_float), ("h2d_ms", ctypes.c_float),
        ("attn_resident_ms", ctypes.c_float), ("attn_offloaded_ms", ctypes.c_float),
        ("merge_ms", ctypes.c_float), ("total_ms", ctypes.c_float),
        ("bytes_resident", ctypes.c_uint64), ("bytes_offloaded", ctypes.c_uint64),
        ("bytes_staged", ctypes.c_uint64), ("bytes_appended", ctypes.c_uint64),
        ("n_chunks", ctypes.c_int32), ("status", ctypes.c_uint32),
    ]

    def as_dict(self):
        return {name: getattr(self, name) for name, _ in self._fields_}


class FillTimes(ctypes.Structure):
    _fields_ = [
        ("pack_ms", ctypes.c_float), ("store_ms", ctypes.c_float), ("total_ms", ctypes.c_float),
        ("bytes_stored", ctypes.c_uint64), ("bytes_resident", ctypes.c_uint64), ("n_copies", ctypes.c_int32),
    ]


_lib = None


def lib():
    """The loaded library; raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2504_11816_b200.build` "
            "(this package has no fallback implementation)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, u64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint64
    P = ctypes.POINTER
    L.isv_kv_alloc.argtypes = [P(vp), P(KvDesc)]
    L.isv_kv_free.argtypes = [vp]
    L.isv_kv_reset.argtypes = [vp]
    L.isv_kv_info.argtypes = [vp, P(KvInfo)]
    L.isv_kv_fill.argtypes = [vp, i32, vp, vp, vp, i32, i32]
    L.isv_kv_fill_async.argtypes = [vp, i32, vp, vp, vp, i32, i32]
    L.isv_fill_timing.argtypes = [vp, P(FillTimes)]
    L.isv_kv_append.argtypes = [vp, i32, vp, vp, i32]
    L.isv_attn_decode.argtypes = [vp, i32, vp, vp, vp, vp, vp, i32]
    L.isv_decode_layer.argtypes = [vp, i32, vp, vp, vp, vp, vp, i32]
    L.isv_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, i32]
    L.isv_decode_step_host.argtypes = [vp, vp, vp, vp, vp, i32]
    L.isv_kv_gather.argtypes = [vp, i32, i32, vp, vp, P(i32)]
    L.isv_block_table_dev.argtypes = [vp, P(i32)]
    L.isv_block_table_dev.restype = vp
    L.isv_seq_lens_dev.argtypes = [vp, i32]
    L.isv_seq_lens_dev.restype = vp
    L.isv_block_table_host.argtypes = [vp, vp, i32, i32]
    L.isv_seq_lens_host.argtypes = [vp, i32, vp, i32]
    L.isv_plan_bytes.argtypes = [vp, i32, i32, P(u64), P(u64), P(u64), P(i32)]
    L.isv_set_zero_copy.argtypes = [vp, i32]
    L.isv_set_timing.argtypes = [vp, i32]
    L.isv_set_host_timeout.argtypes = [vp, ctypes.c_double]
    L.isv_set_wait_limit.argtypes = [vp, ctypes.c_uint32]
    L.isv_inject_lost_copy.argtypes = [vp, i32]
    L.isv_step_timing.argtypes = [vp, i32, P(StepTimes)]
    L.isv_sync.argtypes = [vp, P(ctypes.c_uint32)]
    L.isv_link_probe.argtypes = [u64, i32, P(ctypes.c_double), P(ctypes.c_double)]
    L.isv_attn_decode_static.argtypes = [vp, i32, vp, i32, vp, i32, i32, i32, i32, i32, i32, i32, i32, vp, vp, vp,
                                         vp, vp]
    L.isv_linear_create.argtypes = [P(vp), vp, i32, i32, i32, i32, vp]
    L.isv_linear_forward.argtypes = [vp, vp, vp, vp, i32]
    L.isv_linear_status.argtypes = [vp, P(ctypes.c_uint32)]
    L.isv_linear_free.argtypes = [vp]
    L.isv_last_error.argtypes = []
    L.isv_last_error.restype = ctypes.c_char_p
    for name in EXPORTS:
        fn = getattr(L, name)
        if name not in ("isv_block_table_dev", "isv_seq_lens_dev", "isv_last_error"):
            fn.restype = ctypes.c_int
    _lib = L
    return L


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    raise TypeError(f"cannot take a pointer from {type(x)!r}")


def isv_last_error() -> str:
    return lib().isv_last_error().decode()


def _check(rc: int):
    if rc != ISV_OK:
        raise IsvError(rc, isv_last_error())


# ---------------------------------------------------------------- entry points, same names as the C ABI

def isv_kv_alloc(**kw) -> int:
    """Fields of ``isv_kv_desc`` as keyword arguments; returns the handle."""
    d = KvDesc()
    for k, v in kw.items():
        if k == "compute_stream":
            v = ctypes.c_void_p(v) if v else None
        setattr(d, k, v)
    h = ctypes.c_void_p()
    _check(lib().isv_kv_alloc(ctypes.byref(h), ctypes.byref(d)))
    return h.value


def isv_kv_free(h: int):
    _check(lib().isv_kv_free(h))


def isv_kv_reset(h: int):
    _check(lib().isv_kv_reset(h))


def isv_kv_info(h: int) -> KvInfo:
    o = KvInfo()
    _check(lib().isv_kv_info(h, ctypes.byref(o)))
    return o


def isv_kv_fill(h: int, layer: int, k, v, lens_host, n_seqs: int, T: int):
    lens = np.ascontiguousarray(lens_host, dtype=np.int32)
    _check(lib().isv_kv_fill(h, layer, _ptr(k), _ptr(v), lens.ctypes.data, n_seqs, T))


def isv_kv_fill_async(h: int, layer: int, k, v, lens_host, n_seqs: int, T: int):
    lens = np.ascontiguousarray(lens_host, dtype=np.int32)
    _check(lib().isv_kv_fill_async(h, layer, _ptr(k), _ptr(v), lens.ctypes.data, n_seqs, T))


def isv_fill_timing(h: int) -> FillTimes:
    o = FillTimes()
    _check(lib().isv_fill_timing(h, ctypes.byref(o)))
    return o


def isv_kv_append(h: int, layer: int, k, v, n_seqs: int):
    _check(lib().isv_kv_append(h, layer, _ptr(k), _ptr(v), n_seqs))


def isv_attn_decode(h: int, layer: int, q, out, out_f32, block_table, seq_lens, n_seqs: int):
    _check(lib().isv_attn_decode(h, layer, _ptr(q), _ptr(out), _ptr(out_f32), _ptr(block_table),
                                 _ptr(seq_lens), n_seqs))


def isv_decode_layer(h: int, layer: int, q, k, v, out, out_f32, n_seqs: int):
    _check(lib().isv_decode_layer(h, layer, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(out_f32), n_seqs))


def isv_decode_step(h: int, q, k, v, out, out_f32, n_seqs: int):
    _check(lib().isv_decode_step(h, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(out_f32), n_seqs))


def isv_decode_step_host(h: int, q, k, v, out, n_seqs: int):
    _check(lib().isv_decode_step_host(h, _ptr(q), _ptr(k), _ptr(v), _ptr(out), n_seqs))


def isv_kv_gather(h: int, layer: int, seq: int, k_host: np.ndarray, v_host: np.ndarray) -> int:
    n = ctypes.c_int32(0)
    _check(lib().isv_kv_gather(h, layer, seq, k_host.ctypes.data, v_host.ctypes.data, ctypes.byref(n)))
    return n.value


def isv_block_table_dev(h: int):
    stride = ctypes.c_int32(0)
    p = lib().isv_block_table_dev(h, ctypes.byref(stride))
    return p, stride.value


def isv_seq_lens_dev(h: int, layer: int):
    return lib().isv_seq_lens_dev(h, layer)


def isv_block_table_host(h: int, n_seqs: int) -> np.ndarray:
    stride = isv_kv_info(h).max_blocks_per_seq
    out = np.empty((n_seqs, stride), dtype=np.int32)
    _check(lib().isv_block_table_host(h, out.ctypes.data, n_seqs, stride))
    return out


def isv_seq_lens_host(h: int, layer: int, n_seqs: int) -> np.ndarray:
    out = np.empty(n_seqs, dtype=np.int32)
    _check(lib().isv_seq_lens_host(h, layer, out.ctypes.data, n_seqs))
    return out


def isv_plan_bytes(h: int, layer: int, n_seqs: int):
    """(bytes_resident, bytes_offloaded, bytes_staged, n_chunks)."""
    r, o, s = ctypes.c_uint64(0), ctypes.c_uint64(0), ctypes.c_uint64(0)
    n = ctypes.c_int32(0)
    _check(lib().isv_plan_bytes(h, layer, n_seqs, ctypes.byref(r), ctypes.byref(o), ctypes.byref(s),
                                ctypes.byref(n)))
    return r.value, o.value, s.value, n.value


def isv_set_zero_copy(h: int, on: bool):
    _check(lib().isv_set_zero_copy(h, 1 if on else 0))


def isv_set_host_timeout(h: int, seconds: float):
    _check(lib().isv_set_host_timeout(h, float(seconds)))


def isv_set_wait_limit(h: int, polls: int):
    _check(lib().isv_set_wait_limit(h, polls))


def isv_inject_lost_copy(h: int, launches: int):
    _check(lib().isv_inject_lost_copy(h, launches))


def isv_set_timing(h: int, on: bool):
    _check(lib().isv_set_timing(h, 1 if on else 0))


def isv_step_timing(h: int, layer: int = -1) -> StepTimes:
    o = StepTimes()
    _check(lib().isv_step_timing(h, layer, ctypes.byref(o)))
    return o


def isv_sync(h: int) -> int:
    st = ctypes.c_uint32(0)
    _check(lib().isv_sync(h, ctypes.byref(st)))
    return st.value


def isv_link_probe(nbytes: int = 1 << 30, reps: int = 10):
    """(h2d_GBps, d2h_GBps) of pinned copies on the current device."""
    a, b = ctypes.c_double(0), ctypes.c_double(0)
    _check(lib().isv_link_probe(nbytes, reps, ctypes.byref(a), ctypes.byref(b)))
    return a.value, b.value


ISV_STATIC_SCRATCH_BYTES = 8 << 20


def isv_attn_decode_static(kv_pool, n_pool_blocks: int, block_table, table_stride: int, seq_lens, n_seqs: int,
                           max_blocks_per_seq: int, q_heads: int, kv_heads: int, head_dim: int, block_tokens: int,
                           dtype: int, max_ctas: int, q, out, out_f32, status=None, stream: int = 0):
    """Decode attention over a caller-owned, all-resident paged KV pool without any
    allocation by the library (for callers that may not call cudaMalloc: see
    ``include/isv.h``).  Scratch is a fixed 8 MiB device array shared by all calls;
    shapes that need more raise ``IsvError`` with code ``ISV_ECAPACITY``."""
    _check(lib().isv_attn_decode_static(_ptr(kv_pool), n_pool_blocks, _ptr(block_table), table_stride,
                                        _ptr(seq_lens), n_seqs, max_blocks_per_seq, q_heads, kv_heads, head_dim,
                                        block_tokens, dtype, max_ctas, _ptr(q), _ptr(out), _ptr(out_f32),
                                        _ptr(status), stream or None))


def isv_linear_create(w, N: int, K: int, dtype: int, max_M: int, stream: int = 0) -> int:
    h = ctypes.c_void_p()
    _check(lib().isv_linear_create(ctypes.byref(h), _ptr(w), N, K, dtype, max_M, stream or None))
    return h.value


def isv_linear_forward(l: int, x, y, y_f32, M: int):
    _check(lib().isv_linear_forward(l, _ptr(x), _ptr(y), _ptr(y_f32), M))


def isv_linear_status(l: int) -> int:
    st = ctypes.c_uint32(0)
    _check(lib().isv_linear_status(l, ctypes.byref(st)))
    return st.value


def isv_linear_free(l: int):
    _check(lib().isv_linear_free(l))


def desc_from_workload(w, **overrides) -> dict:
    """Keyword arguments for :func:`isv_kv_alloc` from a ``workloads.Workload``."""
    d = dict(layers=w.layers, phys_layers=0, q_heads=w.q_heads, kv_heads=w.kv_heads,
             head_dim=w.head_dim, block_tokens=w.block_tokens,
             dtype=ISV_F16 if w.dtype == "f16" else ISV_BF16, offload_frac=w.offload_frac,
             max_seqs=w.batch, max_tokens_per_seq=w.max_tokens, perm_seed=w.perm_seed)
    d.update(overrides)
    return d
