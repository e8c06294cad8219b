"""Test harness: drives the CUDA library and the CPU reference side by side on
the same seeded inputs.  The reference never sees library memory: it reads the
harness's own record (ShadowCache) of what was loaded and appended."""
from __future__ import annotations

import numpy as np
import torch

from oracle import attn as oa
from oracle import kv_model as km
from paper_2504_11816_b200 import binding as B
from paper_2504_11816_b200 import workloads as W

TOL = 2e-3   # max-abs bound on fp32 outputs against the fp64 reference


def bits_to_dev(bits: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()
    return t.view(W.torch_dtype(dtype))


def dev_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def values(bits: np.ndarray, dtype: str):
    return W.bits_to_values(np.ascontiguousarray(bits), dtype)


def round_to(x64: np.ndarray, dtype: str) -> np.ndarray:
    """fp64 -> values of the 16-bit dtype, as fp64 (round to nearest even)."""
    t = torch.from_numpy(np.ascontiguousarray(x64)).to(W.torch_dtype(dtype))
    return t.to(torch.float64).numpy()


class Harness:
    def __init__(self, w: W.Workload, lens=None, **desc):
        self.w = w
        self.lens = np.array(W.prompt_lens(w) if lens is None else lens, dtype=np.int32)
        assert len(self.lens) == w.batch
        kw = B.desc_from_workload(w, **desc)
        kw["max_tokens_per_seq"] = max(kw["max_tokens_per_seq"], int(self.lens.max()) + w.steps)
        self.h = B.isv_kv_alloc(**kw)
        # layers that share a physical slab share their record too (same order of writes)
        self.phys = kw.get("phys_layers", 0) or w.layers
        self.shadow = km.ShadowCache(w.layers, w.kv_heads, w.head_dim)
        self.rng = W.host_rng(w)
        self.cur = self.lens.copy()

    def close(self):
        if self.h:
            B.isv_kv_free(self.h)
            self.h = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    # ---- loading
    def fill(self):
        w = self.w
        T = max(1, int(self.lens.max()))
        for layer in range(w.layers):
            k, v = W.host_prompt(w, self.rng, T)
            kd, vd = bits_to_dev(k, w.dtype), bits_to_dev(v, w.dtype)
            torch.cuda.synchronize()
            B.isv_kv_fill(self.h, layer, kd, vd, self.lens, w.batch, T)
            self.shadow.fill(layer % self.phys, k, v, self.lens.tolist())

    # ---- one decode step through separate append / attention calls
    def step(self, f32=True, out16=True, fused=False):
        """One decode step, layer by layer, through isv_kv_append + isv_attn_decode or (fused) through
        isv_decode_layer.  Returns per layer (q_bits, out_f32 ndarray or None, out16 bits or None)."""
        w = self.w
        res = []
        for layer in range(w.layers):
            k, v, q = W.host_step(w, self.rng)
            kd, vd, qd = (bits_to_dev(x, w.dtype) for x in (k, v, q))
            of = torch.full((w.batch, w.q_heads, w.head_dim), float("nan"), device="cuda") if f32 else None
            o16 = torch.zeros((w.batch, w.q_heads, w.head_dim), device="cuda",
                              dtype=W.torch_dtype(w.dtype)) if out16 else None
            torch.cuda.synchronize()
            if fused:
                B.isv_decode_layer(self.h, layer, qd, kd, vd, o16, of, w.batch)
            else:
                B.isv_kv_append(self.h, layer, kd, vd, w.batch)
                B.isv_attn_decode(self.h, layer, qd, o16, of, None, None, w.batch)
            B.isv_sync(self.h)
            if self.phys < w.layers:
                # shared slabs: this layer's token lands at its own position, over a sharer's if one wrote first;
                # the reference must be taken now, before the next sharer overwrites the slot again
                self.shadow.store_at(layer % self.phys, k, v, self.cur.tolist())
                ref = self.reference(layer, q, lens=(self.cur + 1))
            else:
                self.shadow.append(layer, k, v)
                ref = None
            res.append((q, of.cpu().numpy() if f32 else None, dev_to_bits(o16) if out16 else None, ref))
        self.cur += 1
        return res

    # ---- reference
    def reference(self, layer: int, q_bits: np.ndarray, seqs=None, lens=None) -> np.ndarray:
        w = self.w
        seqs = list(range(w.batch)) if seqs is None else list(seqs)
        K, V = [], []
        for s in seqs:
            kb, vb = self.shadow.gathered(layer % self.phys, s)
            if lens is not None:
                kb, vb = kb[: int(lens[s])], vb[: int(lens[s])]
            K.append(values(kb, w.dtype))
            V.append(values(vb, w.dtype))
        q = values(q_bits[seqs], w.dtype)
        return oa.attn_decode(q, K, V)

    def check_step(self, res, tol=TOL):
        """Element-by-element comparison of one step's outputs with the reference."""
        w = self.w
        worst = 0.0
        for layer, (q, of, o16, ref_now) in enumerate(res):
            ref = ref_now if ref_now is not None else self.reference(layer, q)
            if of is not None:
                assert np.all(np.isfinite(of)), f"layer {layer}: non-finite output"
                err = float(np.max(np.abs(of.astype(np.float64) - ref)))
                assert err <= tol, f"layer {layer}: max-abs error {err}"
                worst = max(worst, err)
            if o16 is not None:
                # the 16-bit output is the fp32 result rounded once more: half a unit in the last place of
                # the stored value (2^-11 relative for fp16, 2^-8 for bf16) comes on top of the bound
                got = oa.to_f64(values(o16, w.dtype))
                half_ulp = np.abs(ref) * (2.0 ** -8 if w.dtype == "bf16" else 2.0 ** -11)
                excess = float(np.max(np.abs(got - ref) - half_ulp))
                assert excess <= tol, f"layer {layer}: 16-bit output error exceeds its rounding by {excess}"
        return worst

    def check_gather(self, layers=None, seqs=None):
        """The library's logical-order copy equals the record bit for bit."""
        w = self.w
        cap = B.isv_kv_info(self.h)
        for layer in (range(w.layers) if layers is None else layers):
            for s in (range(w.batch) if seqs is None else seqs):
                kb, vb = self.shadow.gathered(layer % self.phys, s)
                rows = max(1, kb.shape[0])
                kh = np.zeros((rows, w.kv_heads, w.head_dim), np.uint16)
                vh = np.zeros_like(kh)
                n = B.isv_kv_gather(self.h, layer, s, kh, vh)
                assert n == kb.shape[0], (layer, s, n, kb.shape)
                assert np.array_equal(kh[:n], kb), f"K mismatch layer {layer} seq {s}"
                assert np.array_equal(vh[:n], vb), f"V mismatch layer {layer} seq {s}"
        return cap
