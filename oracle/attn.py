"""Python face of the fp64 attention oracle (``attn_oracle.c``) plus the
log-sum-exp merge rule written out in numpy.

TEST INFRASTRUCTURE ONLY: nothing on the product path imports this module, and
this module imports nothing from the product package.

The attention definition follows the decode self-attention that the paper's
T_compute^d formula counts (Section IV-C, "Decode Stage Processing Time"):
``out = softmax(q K^T / sqrt(d)) V`` per sequence and query head, over the
sequence's tokens in logical order.
"""
from __future__ import annotations

import ctypes
import math
from typing import List, Sequence, Tuple

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        lib.oracle_attn_decode.restype = ctypes.c_int
        lib.oracle_attn_decode.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
        lib.oracle_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def max_threads() -> int:
    """Threads the C oracle uses when ``n_threads`` is left at 0."""
    return int(_load().oracle_max_threads())


def to_f64(x) -> np.ndarray:
    """Exact widening of an fp16 / bf16 / fp32 array (numpy or torch CPU) to
    a contiguous numpy float64 array.  Every fp16 and bf16 value is exactly
    representable in fp64, so no rounding happens here."""
    if isinstance(x, np.ndarray):
        return np.ascontiguousarray(x.astype(np.float64))
    import torch  # torch is only needed for bf16, which numpy lacks
    if isinstance(x, torch.Tensor):
        return np.ascontiguousarray(x.detach().cpu().to(torch.float64).numpy())
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def attn_decode(q, K_list: Sequence, V_list: Sequence, return_weights: bool = False,
                n_threads: int = 0):
    """Decode attention for a batch.

    q        [n_seqs, Hq, d]
    K_list   per sequence an array [n_s, Hkv, d] (logical token order), n_s >= 1
    V_list   same shapes as K_list
    Returns out [n_seqs, Hq, d] float64, and with ``return_weights`` also a list
    of per-sequence arrays [Hq, n_s] holding the normalised softmax weights.
    """
    q64 = to_f64(q)
    n_seqs, Hq, d = q64.shape
    assert len(K_list) == n_seqs and len(V_list) == n_seqs
    K64 = [to_f64(k) for k in K_list]
    V64 = [to_f64(v) for v in V_list]
    Hkv = K64[0].shape[1] if n_seqs else 1
    lens = np.array([k.shape[0] for k in K64], dtype=np.int32)
    for k, v in zip(K64, V64):
        assert k.shape == v.shape and k.shape[1] == Hkv and k.shape[2] == d
    row_off = np.zeros(n_seqs, dtype=np.int64)
    if n_seqs:
        row_off[1:] = np.cumsum(lens[:-1], dtype=np.int64)
    Kc = np.ascontiguousarray(np.concatenate(K64, axis=0)) if n_seqs else np.zeros((0, Hkv, d))
    Vc = np.ascontiguousarray(np.concatenate(V64, axis=0)) if n_seqs else np.zeros((0, Hkv, d))
    out = np.empty((n_seqs, Hq, d), dtype=np.float64)
    wbuf = np.empty(int(lens.sum()) * Hq, dtype=np.float64) if return_weights else None
    rc = _load().oracle_attn_decode(
        q64.ctypes.data, Kc.ctypes.data, Vc.ctypes.data,
        row_off.ctypes.data, lens.ctypes.data,
        n_seqs, Hq, Hkv, d, out.ctypes.data,
        wbuf.ctypes.data if wbuf is not None else None, int(n_threads))
    if rc != 0:
        raise ValueError(f"oracle_attn_decode failed with code {rc}")
    if not return_weights:
        return out
    weights: List[np.ndarray] = []
    for s in range(n_seqs):
        a = int(row_off[s]) * Hq
        weights.append(wbuf[a:a + Hq * int(lens[s])].reshape(Hq, int(lens[s])).copy())
    return out, weights


# --------------------------------------------------------------------------
# The split / merge rule that the library's merge step implements, in fp64.
# A partial over a subset P of one (sequence, head)'s tokens is the triple
#   m = max_{i in P} score_i,  l = sum_{i in P} exp(score_i - m),
#   o = sum_{i in P} exp(score_i - m) V_i            (not normalised)
# and partials combine as
#   m* = max_p m_p;  l* = sum_p l_p e^{m_p - m*};  o* = sum_p o_p e^{m_p - m*};  out = o*/l*.
# --------------------------------------------------------------------------

Partial = Tuple[float, float, np.ndarray]


def attn_partial(q_row, K_rows, V_rows) -> Partial:
    """(m, l, o) of one query row over the given token rows ([n, d] each)."""
    qv = to_f64(q_row)
    Kr = to_f64(K_rows)
    Vr = to_f64(V_rows)
    d = qv.shape[0]
    scores = np.array([float(np.dot(qv, Kr[i])) / math.sqrt(d) for i in range(Kr.shape[0])])
    m = float(scores.max())
    w = np.exp(scores - m)
    return m, float(w.sum()), (w[:, None] * Vr).sum(axis=0)


def merge_partials(parts: Sequence[Partial]) -> np.ndarray:
    """Normalised output from any number of non-empty partials."""
    m_star = max(p[0] for p in parts)
    l_star = 0.0
    o_star = np.zeros_like(parts[0][2], dtype=np.float64)
    for m, l, o in parts:
        a = math.exp(m - m_star)
        l_star += l * a
        o_star = o_star + o * a
    return o_star / l_star
