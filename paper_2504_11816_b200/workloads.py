"""Seeded synthetic workloads: shapes, lengths and random tensors only.

This module holds no attention arithmetic.  It serves both the CUDA library's
callers and the CPU reference used in tests, so it imports neither.

The five presets mirror the decode workloads this library is measured on.
They stand in for the paper's OPT-1.3B/2.7B/6.7B runs (Section V-A: 128-in /
512-out online and 1024-in / 128-out offline requests, batch sizes 1-64):
trained weights are not needed because the cost of decode attention depends
only on batch size, context length, KV width, dtype and offload ratio, so
Llama-shaped random tensors of those shapes are used instead.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Tuple

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    layers: int
    q_heads: int
    kv_heads: int
    head_dim: int
    dtype: str              # "f16" or "bf16"
    batch: int
    ctx_min: int            # prompt length range, inclusive; equal = fixed length
    ctx_max: int
    steps: int              # decode steps after the prompt
    block_tokens: int
    offload_frac: float
    perm_seed: int          # 0 = physical block ids handed out in order
    seed: int
    outlier_prob: float = 0.0
    outlier_scale: float = 1.0

    @property
    def elem_bytes(self) -> int:
        return 2

    @property
    def kv_bytes_per_token(self) -> int:
        """K and V of one token in one layer."""
        return 2 * self.kv_heads * self.head_dim * self.elem_bytes

    @property
    def max_tokens(self) -> int:
        return self.ctx_max + self.steps

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


CONFIGS: Dict[str, Workload] = {
    # 1 layer, batch 4, 8 q / 8 KV heads, d 64, fp16, context 256, every other block on the host
    "tiny": Workload("tiny", 1, 8, 8, 64, "f16", 4, 256, 256, 1, 16, 0.5, 0, 0),
    # Llama-2-7B-shaped decode, everything in HBM
    "c2": Workload("c2", 32, 32, 32, 128, "f16", 32, 1024, 1024, 128, 16, 0.0, 0, 1),
    # Llama-2-7B-shaped offline batch, half of each sequence's blocks on the host
    "c3": Workload("c3", 32, 32, 32, 128, "f16", 128, 2048, 2048, 64, 16, 0.5, 2, 2),
    # Llama-3-8B-shaped GQA, bf16, three quarters on the host
    "c4": Workload("c4", 32, 32, 8, 128, "bf16", 256, 4096, 4096, 32, 16, 0.75, 3, 3),
    # the paper's own offline workload (Section V-A): OPT-2.7B (32 layers, 32 heads x 80), batch 32, 1024 input
    # and 128 output tokens, fp16; offload fraction 0 / 0.6 / 1 in its Table VI (set with --offload)
    "opt2.7b": Workload("opt2.7b", 32, 32, 32, 80, "f16", 32, 1024, 1024, 128, 16, 0.0, 0, 5),
    # 13B-shaped, ragged contexts, 1 % of K/V entries scaled by 8; offload fraction is swept
    "c5": Workload("c5", 40, 40, 40, 128, "f16", 64, 512, 8192, 32, 16, 0.0, 4, 4,
                   outlier_prob=0.01, outlier_scale=8.0),
}


def prompt_lens(w: Workload) -> np.ndarray:
    """Per-sequence prompt lengths: integers uniform in [ctx_min, ctx_max],
    independent per sequence, not rounded to block multiples.  Drawn from their
    own stream so they do not depend on how many tensor values were drawn."""
    if w.ctx_min == w.ctx_max:
        return np.full(w.batch, w.ctx_min, dtype=np.int32)
    rng = np.random.default_rng([w.seed, 0x1E45])
    return rng.integers(w.ctx_min, w.ctx_max + 1, size=w.batch).astype(np.int32)


# ---------------------------------------------------------------- host (numpy)

def _round_to_bits(x32: np.ndarray, dtype: str) -> np.ndarray:
    """float32 values -> the uint16 bit patterns of their fp16 / bf16 rounding
    (round to nearest even, done by numpy / torch)."""
    if dtype == "f16":
        return np.ascontiguousarray(x32.astype(np.float16)).view(np.uint16)
    if dtype == "bf16":
        import torch
        t = torch.from_numpy(np.ascontiguousarray(x32)).to(torch.bfloat16)
        return t.view(torch.int16).numpy().view(np.uint16)
    raise ValueError(f"unknown dtype {dtype!r}")


def normal_bits(rng: np.random.Generator, shape: Tuple[int, ...], dtype: str,
                outlier_prob: float = 0.0, outlier_scale: float = 1.0) -> np.ndarray:
    """N(0,1) draws rounded to ``dtype`` and returned as uint16 bit patterns.
    With ``outlier_prob`` > 0 each entry is, independently, multiplied by
    ``outlier_scale`` (the uniform draw follows the normal draw on the same
    stream)."""
    x = rng.standard_normal(shape, dtype=np.float32)
    if outlier_prob > 0.0:
        mask = rng.random(shape, dtype=np.float32) < outlier_prob
        x = np.where(mask, x * np.float32(outlier_scale), x)
    return _round_to_bits(x, dtype)


def bits_to_values(bits: np.ndarray, dtype: str):
    """uint16 bit patterns -> numpy float16 array, or a torch bfloat16 CPU
    tensor for "bf16" (numpy has no bfloat16)."""
    if dtype == "f16":
        return bits.view(np.float16)
    import torch
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)


def host_rng(w: Workload) -> np.random.Generator:
    """Tensor stream of a workload.  Order of use: prompt K, prompt V (per
    layer), then per decode step and layer: k, v, q."""
    return np.random.default_rng(w.seed)


def host_prompt(w: Workload, rng: np.random.Generator, T: int | None = None):
    """One layer's prompt K and V, [batch, T, kv_heads, head_dim] uint16 each."""
    T = w.ctx_max if T is None else T
    shape = (w.batch, T, w.kv_heads, w.head_dim)
    k = normal_bits(rng, shape, w.dtype, w.outlier_prob, w.outlier_scale)
    v = normal_bits(rng, shape, w.dtype, w.outlier_prob, w.outlier_scale)
    return k, v


def host_step(w: Workload, rng: np.random.Generator):
    """One layer's decode-step inputs: k, v [batch, kv_heads, head_dim] and
    q [batch, q_heads, head_dim], uint16 bit patterns.  q has no outliers."""
    k = normal_bits(rng, (w.batch, w.kv_heads, w.head_dim), w.dtype, w.outlier_prob, w.outlier_scale)
    v = normal_bits(rng, (w.batch, w.kv_heads, w.head_dim), w.dtype, w.outlier_prob, w.outlier_scale)
    q = normal_bits(rng, (w.batch, w.q_heads, w.head_dim), w.dtype)
    return k, v, q


# ---------------------------------------------------------------- device (torch)

def torch_dtype(dtype: str):
    import torch
    return {"f16": torch.float16, "bf16": torch.bfloat16}[dtype]


def device_generator(w: Workload, stream_id: int = 0, device: str = "cuda"):
    """Seeded torch generator on the device, for tensors too large to draw on
    the host in reasonable time."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed((w.seed << 20) + stream_id)
    return g


def device_normal(gen, shape, dtype: str, outlier_prob: float = 0.0, outlier_scale: float = 1.0,
                  device: str = "cuda"):
    """N(0,1) tensor of ``dtype`` drawn on ``device`` with the same outlier
    recipe as :func:`normal_bits`."""
    import torch
    x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    if outlier_prob > 0.0:
        mask = torch.rand(shape, generator=gen, device=device, dtype=torch.float32) < outlier_prob
        x = torch.where(mask, x * outlier_scale, x)
    return x.to(torch_dtype(dtype))
