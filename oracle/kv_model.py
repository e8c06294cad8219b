"""Plain model of what the paged, partly offloaded KV cache must contain and
how many of its bytes sit on each side of the host link.

TEST INFRASTRUCTURE ONLY: the product library never imports this.

* ``ShadowCache`` is the definition of the cache's logical content: per layer
  and sequence, the K and V rows in the order they were loaded and appended
  (the paper's KV cache grows by one token per decode step, Section II-A).
  The library's gather must return exactly these bits.
* ``is_host_block`` is the residency rule that turns the paper's offload ratio
  C_off (Section IV-B, ``C_off = 1 - Mem_avail / Mem_KVcache``) into a per-block
  decision: of every prefix of j blocks, floor(j * C_off) are host-resident.
* ``layer_step_bytes`` counts, for one layer and one decode step, the KV bytes
  read from GPU memory and the KV bytes that must cross the host link; its
  offloaded part reduces to the first term of the paper's T_trans^d numerator
  (Section IV-C), ``C_off * 2 * L * h1 * Precision_bytes * BS``.
"""
from __future__ import annotations

import math
from typing import Dict, List, Sequence, Tuple

import numpy as np


def f32(x: float) -> float:
    """The value a C ``float`` holds for x, as a Python float (double)."""
    return float(np.float32(x))


def is_host_block(j: int, offload_frac: float) -> bool:
    """Logical block j of a sequence is host-resident iff
    floor((j+1) f) > floor(j f), f being the float32 offload fraction widened
    to double.  The products are exact in double for j < 2^28."""
    f = f32(offload_frac)
    return math.floor((j + 1) * f) > math.floor(j * f)


def n_blocks(n_tokens: int, block_tokens: int) -> int:
    return (n_tokens + block_tokens - 1) // block_tokens


def kv_bytes_per_token(kv_heads: int, head_dim: int, elem_bytes: int) -> int:
    """K and V of one token in one layer (Table II's per-layer KV size divided
    by BS * tokens, with h1 read as kv_heads * head_dim)."""
    return 2 * kv_heads * head_dim * elem_bytes


def layer_step_bytes(lens: Sequence[int], offload_frac: float, block_tokens: int,
                     kappa: int) -> Tuple[int, int]:
    """(resident bytes, offloaded bytes) that one layer's decode attention
    reads when sequence s attends to lens[s] tokens.

    A host-resident block counts as offloaded only once it is complete and is
    no longer the sequence's newest block: the block that holds the newest
    token is always kept in GPU memory (it is still being written)."""
    res = 0
    off = 0
    for n in lens:
        if n <= 0:
            continue
        nb = n_blocks(n, block_tokens)
        host_tokens = 0
        for j in range(nb - 1):
            if is_host_block(j, offload_frac):
                host_tokens += block_tokens
        off += host_tokens * kappa
        res += (n - host_tokens) * kappa
    return res, off


class ShadowCache:
    """Logical content of the cache: rows of raw 16-bit patterns.

    ``fill`` and ``append`` take arrays of dtype uint16 (the bit patterns of
    fp16 or bf16 values); ``gathered`` returns [n, Hkv, d] uint16 arrays.
    Rows are kept as a list of [rows, Hkv, d] pieces in arrival order."""

    def __init__(self, layers: int, kv_heads: int, head_dim: int):
        self.layers = layers
        self.kv_heads = kv_heads
        self.head_dim = head_dim
        self._k: Dict[Tuple[int, int], List[np.ndarray]] = {}
        self._v: Dict[Tuple[int, int], List[np.ndarray]] = {}

    def fill(self, layer: int, k_bits: np.ndarray, v_bits: np.ndarray, lens: Sequence[int]):
        """k_bits, v_bits: [n_seqs, T, Hkv, d] uint16; sequence s keeps its
        first lens[s] tokens and forgets anything it held before."""
        assert k_bits.dtype == np.uint16 and v_bits.dtype == np.uint16
        for s, n in enumerate(lens):
            self._k[(layer, s)] = [k_bits[s, :n].copy()]
            self._v[(layer, s)] = [v_bits[s, :n].copy()]

    def append(self, layer: int, k_bits: np.ndarray, v_bits: np.ndarray):
        """k_bits, v_bits: [n_seqs, Hkv, d] uint16, one new token per sequence."""
        assert k_bits.dtype == np.uint16 and v_bits.dtype == np.uint16
        for s in range(k_bits.shape[0]):
            self._k.setdefault((layer, s), []).append(k_bits[s][None].copy())
            self._v.setdefault((layer, s), []).append(v_bits[s][None].copy())

    def store_at(self, layer: int, k_bits: np.ndarray, v_bits: np.ndarray, positions: Sequence[int]):
        """Writes one token per sequence at explicit positions (overwriting what is there, or extending by
        one).  This is what happens when several logical layers share one physical slab: each of them
        writes its token of the step into the same slot, and the last writer's rows stay."""
        assert k_bits.dtype == np.uint16 and v_bits.dtype == np.uint16
        for s, pos in enumerate(positions):
            k, v = self.gathered(layer, s)
            assert 0 <= pos <= k.shape[0], "positions must overwrite or extend by one"
            if pos == k.shape[0]:
                k = np.concatenate([k, k_bits[s][None]])
                v = np.concatenate([v, v_bits[s][None]])
            else:
                k = k.copy(); v = v.copy()
                k[pos] = k_bits[s]
                v[pos] = v_bits[s]
            self._k[(layer, s)] = [k]
            self._v[(layer, s)] = [v]

    def length(self, layer: int, s: int) -> int:
        return sum(c.shape[0] for c in self._k.get((layer, s), []))

    def gathered(self, layer: int, s: int) -> Tuple[np.ndarray, np.ndarray]:
        k = self._k.get((layer, s), [])
        v = self._v.get((layer, s), [])
        shape = (0, self.kv_heads, self.head_dim)
        if not k:
            return np.zeros(shape, np.uint16), np.zeros(shape, np.uint16)
        return np.concatenate(k, axis=0), np.concatenate(v, axis=0)
