"""Calibrates the paper's time model against this library on the GPU at hand.

    python -m paper_2504_11816_b200.calibrate [--ctx 512] [--out-len 128] [--offload 0.5]

Follows the paper's procedure (Section IV-E): run the workload at several
batch sizes, take the measured per-layer time from ``isv_step_timing``, and
fit CTCF(T) = alpha * T + beta by least squares against the model's
T_compute^d attention term (4 * BS * ctx * h1 / FLOPS).  A second run with part
of the cache offloaded compares the measured host-link time with the model's
T_trans^d for the measured link bandwidth, and the measured step time with
Eq. 6 (sum) and with the overlapped alternative (max).  Prints one JSON
object.  Needs a CUDA device; every number comes from the CUDA path.
"""
from __future__ import annotations

import argparse
import json

import numpy as np


def measure(w, steps: int, warmup: int):
    """Mean per-layer times (seconds) and byte counters of `steps` decode steps."""
    import torch
    from . import binding as B
    from . import workloads as W
    lens = W.prompt_lens(w)
    T = int(lens.max())
    h = B.isv_kv_alloc(**B.desc_from_workload(w, max_tokens_per_seq=w.ctx_max + steps + warmup + 1))
    try:
        gen = W.device_generator(w)
        for layer in range(w.layers):
            k = W.device_normal(gen, (w.batch, T, w.kv_heads, w.head_dim), w.dtype)
            v = W.device_normal(gen, (w.batch, T, w.kv_heads, w.head_dim), w.dtype)
            torch.cuda.synchronize()
            B.isv_kv_fill(h, layer, k, v, lens, w.batch, T)
            del k, v
        q = W.device_normal(gen, (w.layers, w.batch, w.q_heads, w.head_dim), w.dtype)
        k = W.device_normal(gen, (w.layers, w.batch, w.kv_heads, w.head_dim), w.dtype)
        v = W.device_normal(gen, (w.layers, w.batch, w.kv_heads, w.head_dim), w.dtype)
        out = torch.zeros_like(q)
        torch.cuda.synchronize()
        B.isv_set_timing(h, True)
        for _ in range(warmup):
            B.isv_decode_step(h, q, k, v, out, w.batch)
        B.isv_sync(h)
        acc = {"attn": 0.0, "h2d": 0.0, "total": 0.0, "bytes_res": 0, "bytes_off": 0}
        for _ in range(steps):
            B.isv_decode_step(h, q, k, v, out, w.batch)
            st = B.isv_step_timing(h, -1)
            acc["attn"] += (st.attn_resident_ms + st.merge_ms) * 1e-3
            acc["h2d"] += st.h2d_ms * 1e-3
            acc["total"] += st.total_ms * 1e-3
            acc["bytes_res"] += st.bytes_resident
            acc["bytes_off"] += st.bytes_offloaded
        n = steps * w.layers
        return {k_: v_ / n for k_, v_ in acc.items()}
    finally:
        B.isv_kv_free(h)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--ctx", type=int, default=512)
    ap.add_argument("--out-len", type=int, default=128)
    ap.add_argument("--offload", type=float, default=0.5)
    ap.add_argument("--layers", type=int, default=8)
    ap.add_argument("--flops", type=float, default=2.25e15, help="FLOP/s the model divides by (dense fp16 peak)")
    args = ap.parse_args()
    import torch
    from . import binding as B
    from . import cost_model as cm
    from . import workloads as W
    assert torch.cuda.is_available(), "calibration needs a CUDA device"
    h2d, d2h = B.isv_link_probe(1 << 30, 10)
    hw = cm.Machine(flops=args.flops, bw_h2d=h2d * 1e9, bw_d2h=d2h * 1e9)
    base = W.Workload("cal", args.layers, 32, 32, 128, "f16", 1, args.ctx, args.ctx, args.out_len, 16, 0.0, 0, 7)
    shape = cm.ModelShape(h1=base.kv_heads * base.head_dim, h2=4 * base.kv_heads * base.head_dim,
                          n_layers=base.layers, prec_bytes=2)
    steps, warmup = 8, 3
    rows, t_model, t_meas = [], [], []
    for bs in (1, 2, 4, 8, 16, 32, 64):
        m = measure(base.with_(batch=bs), steps, warmup)
        ctx_mean = args.ctx + warmup + (steps + 1) / 2.0
        model_attn = 4.0 * bs * ctx_mean * shape.h1 / hw.flops          # attention term of T_compute^d
        rows.append({"batch": bs, "model_attn_s": model_attn, "measured_attn_s": m["attn"],
                     "hbm_GBps": m["bytes_res"] / m["attn"] / 1e9})
        t_model.append(model_attn)
        t_meas.append(m["attn"])
    alpha, beta, err = cm.fit_ctcf(t_model, t_meas)
    for r in rows:
        r["ctcf_s"] = cm.ctcf(r["model_attn_s"], alpha, beta)
        r["error_pct"] = abs(r["ctcf_s"] - r["measured_attn_s"]) / r["measured_attn_s"] * 100
    # offloaded run: transfer term and the sum-vs-max question
    bs = 32
    off = measure(base.with_(batch=bs, offload_frac=args.offload), 4, 3)
    model_trans = off["bytes_off"] / hw.bw_h2d            # first term of T_trans^d with the measured byte count
    compute = cm.ctcf(4.0 * bs * (args.ctx + 5) * (1 - args.offload) * shape.h1 / hw.flops, alpha, beta)
    result = {
        "device": torch.cuda.get_device_name(0), "link_GBps": {"h2d": h2d, "d2h": d2h},
        "shape": {"h1": shape.h1, "layers": base.layers, "ctx": args.ctx, "out_len": args.out_len},
        "flops_used": hw.flops, "ctcf": {"alpha": alpha, "beta_s": beta, "avg_error_pct": err}, "rows": rows,
        "offloaded": {"batch": bs, "offload_frac": args.offload, "bytes_off_per_layer": off["bytes_off"],
                      "t_trans_model_s": model_trans, "t_trans_measured_s": off["h2d"],
                      "t_layer_measured_s": off["total"],
                      "eq6_sum_s": compute + model_trans, "overlapped_max_s": max(compute, model_trans)},
    }
    print(json.dumps(result))


if __name__ == "__main__":
    main()
