#!/usr/bin/env python
"""Benchmark of the offloaded-KV decode path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload c2|c3|c4|c5|tiny] [--offload F] [--phys-layers P]

A step is one decode step of the whole batch through all layers (KV append +
attention per layer).  One JSON line is printed by rank 0:
tokens/s = sequences x steps / time, with the roofline of the dominant kernel,
the combined HBM / host-link roofline, an end-to-end figure measured through
the host-buffer entry point, and the CPU reference timed on the host cores.

With N > 1 (torchrun) every rank runs an independent replica of the workload
on its own GPU (the path has no exchange step); times are the maximum over
ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "offloaded-KV decode attn tokens/s; fraction of HBM+host-link roofline"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of the resident decode kernel from one ncu capture (bytes per KV byte
# processed), valid only for the kernel source it was taken from.
NCU_TRAFFIC = {"kernels_sha1": "315a5d0284e8aa65b79e1e1cba0d9bbe00020e71",
               # multi-head shapes (CUDA-core arithmetic): (546.94 MB read + 4.85 MB written) / 539.23 MB
               # algorithmic, 2-layer case of the default shape
               "dram_bytes_per_kv_byte": (546.935296 + 4.850688) / 539.230208,
               "source": "profiles/decode_kernel_c2_2layers.md",
               # grouped-query shapes (tensor-core arithmetic): (540.00 MB + 5.09 MB) / 537.46 MB, 32 sequences
               # and 2 layers of the 8B-GQA shape
               "dram_bytes_per_kv_byte_gqa": (539.998464 + 5.091072) / 537.460736,
               "source_gqa": "profiles/decode_kernel_gqa_c4shape_batch32_2layers.md"}


def kernels_sha1() -> str:
    h = hashlib.sha1()
    for f in ("isv_kernels.cu", "isv_kernels.cuh"):
        h.update(open(os.path.join(ROOT, "paper_2504_11816_b200", "csrc", f), "rb").read())
    return h.hexdigest()


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while a region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---------------------------------------------------------------- reference arm (CPU)

def reference_sample(w, ctx_lens, n_sample, rng):
    """Host tensors for one layer-step of `n_sample` sequences of the workload."""
    from paper_2504_11816_b200 import workloads as W
    K, V = [], []
    for s in range(n_sample):
        n = int(ctx_lens[s])
        K.append(W.bits_to_values(W.normal_bits(rng, (n, w.kv_heads, w.head_dim), w.dtype, w.outlier_prob,
                                                w.outlier_scale), w.dtype))
        V.append(W.bits_to_values(W.normal_bits(rng, (n, w.kv_heads, w.head_dim), w.dtype, w.outlier_prob,
                                                w.outlier_scale), w.dtype))
    q = W.bits_to_values(W.normal_bits(rng, (n_sample, w.q_heads, w.head_dim), w.dtype), w.dtype)
    return q, K, V


def time_reference(w, n_sample, reps, warmup=0, n_threads=0):
    """Times the CPU reference, as it stands, on a bounded sample: `n_sample`
    sequences (all heads) of one layer-step, on `n_threads` threads (0 = all the
    process may use).  Returns (tokens/s extrapolated to the whole batch and all
    layers, seconds per sampled call, threads, description of the sample)."""
    from oracle import attn as oa
    from paper_2504_11816_b200 import workloads as W
    lens = W.prompt_lens(w) + 1
    order = np.argsort(-lens)                      # longest and shortest both present when ragged
    pick = np.concatenate([order[: (n_sample + 1) // 2], order[::-1][: n_sample // 2]])[:n_sample]
    ctx = lens[pick]
    rng = np.random.default_rng([w.seed, 77])
    q, K, V = reference_sample(w, ctx, n_sample, rng)
    times = []
    for i in range(warmup + reps):
        t0 = time.perf_counter()
        oa.attn_decode(q, K, V, n_threads=n_threads)
        t1 = time.perf_counter()
        if i >= warmup:
            times.append(t1 - t0)
    t = float(np.mean(times))
    # scale by tokens attended: whole batch / sample
    scale = float(lens.sum()) / float(ctx.sum())
    t_layer_step = t * scale
    tps = w.batch / (w.layers * t_layer_step)
    return tps, t, (n_threads or oa.max_threads()), f"{n_sample} of {w.batch} sequences x {w.q_heads} heads, one layer-step " \
        f"(contexts {int(ctx.min())}..{int(ctx.max())}), scaled by attended tokens to the batch and x{w.layers} layers"


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_sample = min(w.batch, 8 if w.name == "c2" else 4)
    tps, t, threads, what = time_reference(w, n_sample, args.steps, args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, args, None),
        "cpu_baseline": {"value": tps, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": what},
        "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------- our arm

def workload_config(w, args, info):
    c = {"workload": f"{w.name}: {w.layers} layers, {w.q_heads} q / {w.kv_heads} kv heads x {w.head_dim}, "
                     f"{w.dtype}, batch {w.batch}, prompt {w.ctx_min}"
                     + (f"..{w.ctx_max}" if w.ctx_max != w.ctx_min else "")
                     + f" tokens, KV block {w.block_tokens}, offload {w.offload_frac:g}",
         "offload_frac": w.offload_frac, "batch": w.batch, "layers": w.layers, "accumulate": "f32",
         "l2": "KV read per layer-step exceeds L2 (inputs larger than L2)", "parallelism": "replicas",
         "offloaded_path": "zero-copy reads" if getattr(args, "zero_copy", False) else "staged through the ring"}
    if info is not None:
        c.update({"phys_layers": info.phys_layers, "max_ctas": info.max_ctas,
                  "chunk_bytes": info.chunk_bytes, "ring_depth": info.ring_depth})
    return c


def choose_phys_layers(w, max_tokens, requested):
    if requested:
        return requested
    import torch
    nb = (max_tokens + w.block_tokens - 1) // w.block_tokens
    host_per_seq = int(np.floor(nb * np.float32(w.offload_frac)))
    block = w.block_tokens * w.kv_bytes_per_token
    hbm_layer = w.batch * (nb - host_per_seq + (1 if host_per_seq else 0)) * block
    host_layer = w.batch * host_per_seq * block
    free, _ = torch.cuda.mem_get_info()
    hbm_budget = 0.70 * free
    avail = 64 << 30
    try:
        for ln in open("/proc/meminfo"):
            if ln.startswith("MemAvailable"):
                avail = int(ln.split()[1]) * 1024
    except OSError:
        pass
    host_budget = min(0.35 * avail, 48 << 30)
    p = w.layers
    if hbm_layer:
        p = min(p, int(hbm_budget // hbm_layer))
    if host_layer:
        p = min(p, int(host_budget // host_layer))
    return max(1, p)


def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2504_11816_b200 import binding as B
    from paper_2504_11816_b200 import replicas as R
    from paper_2504_11816_b200 import workloads as W

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU path exists)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    B.lib()

    K, Wm = args.steps, args.warmup
    passes_steps = Wm + K
    max_tokens = w.ctx_max + passes_steps
    lens = W.prompt_lens(w)
    phys = choose_phys_layers(w, max_tokens, args.phys_layers)
    stream = torch.cuda.Stream()
    desc = B.desc_from_workload(w, phys_layers=phys, max_tokens_per_seq=max_tokens,
                                compute_stream=stream.cuda_stream)
    h = B.isv_kv_alloc(**desc)
    info = B.isv_kv_info(h)
    td = W.torch_dtype(w.dtype)
    if args.zero_copy:
        B.isv_set_zero_copy(h, True)

    store = {"bytes": 0, "ms": 0.0, "copies": 0, "layers": 0}

    def fill(measure_store=False):
        """Seeded prompt K/V, drawn on the device one layer at a time and loaded with isv_kv_fill; with
        `measure_store` the device-to-host write-back of the offloaded share is timed per layer."""
        T = int(lens.max())
        for layer in range(w.layers):
            gen = W.device_generator(w, stream_id=layer % phys)
            k = W.device_normal(gen, (w.batch, T, w.kv_heads, w.head_dim), w.dtype, w.outlier_prob, w.outlier_scale)
            v = W.device_normal(gen, (w.batch, T, w.kv_heads, w.head_dim), w.dtype, w.outlier_prob, w.outlier_scale)
            torch.cuda.synchronize()
            B.isv_kv_fill(h, layer, k, v, lens, w.batch, T)
            if measure_store:
                ft = B.isv_fill_timing(h)
                store["bytes"] += ft.bytes_stored
                store["ms"] += ft.store_ms
                store["copies"] += ft.n_copies
                store["layers"] += 1
            del k, v

    # a few distinct step inputs, resident in HBM, cycled through
    n_in = 4
    gen = W.device_generator(w, stream_id=1000)
    qs = [W.device_normal(gen, (w.layers, w.batch, w.q_heads, w.head_dim), w.dtype) for _ in range(n_in)]
    ks = [W.device_normal(gen, (w.layers, w.batch, w.kv_heads, w.head_dim), w.dtype, w.outlier_prob, w.outlier_scale)
          for _ in range(n_in)]
    vs = [W.device_normal(gen, (w.layers, w.batch, w.kv_heads, w.head_dim), w.dtype, w.outlier_prob, w.outlier_scale)
          for _ in range(n_in)]
    out = torch.zeros((w.layers, w.batch, w.q_heads, w.head_dim), device="cuda", dtype=td)

    def barrier():
        torch.cuda.synchronize()
        R.barrier(dist)
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        return R.max_over_ranks(x, dist, device="cuda")

    # -------- pass 1: device-resident inputs, no per-layer events -> `value`
    fill(measure_store=w.offload_frac > 0)
    for i in range(Wm):
        B.isv_decode_step(h, qs[i % n_in], ks[i % n_in], vs[i % n_in], out, None, w.batch)
    B.isv_sync(h)
    probe_before = B.isv_link_probe(1 << 30, 10) if w.offload_frac > 0 else None
    h2d_before = probe_before[0] if probe_before else None
    launches0 = B.isv_kv_info(h).kernel_launches
    bytes_res = bytes_off = 0
    sampler = ClockSampler(local_rank)
    sampler.start()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(K):
        B.isv_decode_step(h, qs[i % n_in], ks[i % n_in], vs[i % n_in], out, None, w.batch)
    e1.record(stream)
    barrier()
    clocks = sampler.stop()
    ms = max_over_ranks(e0.elapsed_time(e1))
    launches = B.isv_kv_info(h).kernel_launches - launches0
    status = B.isv_sync(h)
    h2d_after = B.isv_link_probe(1 << 30, 10)[0] if w.offload_frac > 0 else None
    value = R.aggregate_tokens_per_s(w.batch, K, ms, world)

    # -------- pass 2: same K steps with per-layer events -> kernel durations and byte counters
    B.isv_kv_reset(h)
    fill()
    B.isv_set_timing(h, True)
    for i in range(Wm):
        B.isv_decode_step(h, qs[i % n_in], ks[i % n_in], vs[i % n_in], out, None, w.batch)
    B.isv_sync(h)
    t_res = t_h2d = t_off = t_merge = t_app = t_tot = 0.0
    staged = 0
    for i in range(K):
        B.isv_decode_step(h, qs[i % n_in], ks[i % n_in], vs[i % n_in], out, None, w.batch)
        st = B.isv_step_timing(h, -1)
        t_res += st.attn_resident_ms
        t_h2d += st.h2d_ms
        t_off += st.attn_offloaded_ms
        t_merge += st.merge_ms
        t_app += st.append_ms
        t_tot += st.total_ms
        bytes_res += st.bytes_resident
        bytes_off += st.bytes_offloaded
        staged += st.bytes_staged
    B.isv_set_timing(h, False)

    hbm_gbs, peak_kind = measured_peaks()
    n_launch = K * w.layers
    ev_ms = t_res / n_launch                    # pass 2: events around every launch (they add gaps of their own)
    ev_achieved = (bytes_res / n_launch) / (ev_ms * 1e-3) / 1e9 if ev_ms > 0 else 0.0
    if w.offload_frac == 0:
        # Nothing is offloaded: the timed region of pass 1 holds one decode_kernel launch per layer-step and
        # nothing else (bar a table update every 16 steps), so its two events give the kernel's average
        # duration directly, launch gaps included, without per-launch events perturbing the stream.
        avg_ms = ms / n_launch
        timed = ("CUDA events around the timed region / launches in it (one decode_kernel launch per layer-step; "
                 "includes the gaps between launches)")
    else:
        avg_ms = ev_ms
        timed = "separate pass of the same K steps with CUDA events around every launch"
    achieved = (bytes_res / n_launch) / (avg_ms * 1e-3) / 1e9 if avg_ms > 0 else 0.0
    traffic = None
    if NCU_TRAFFIC["kernels_sha1"] == kernels_sha1():   # counters taken from this very kernel source
        gqa = w.q_heads // w.kv_heads >= 2               # those shapes run the tensor-core variant
        traffic = NCU_TRAFFIC["dram_bytes_per_kv_byte_gqa" if gqa else "dram_bytes_per_kv_byte"] * bytes_res / n_launch
    roofline = {"bound": "hbm", "kernel": "decode_kernel (resident, split flash-decoding)",
                "achieved": achieved, "peak": hbm_gbs, "unit": "GB/s", "frac": achieved / hbm_gbs,
                "peak_kind": f"of {peak_kind}", "traffic": traffic,
                "bytes_per_launch": bytes_res / n_launch, "avg_launch_ms": avg_ms, "timed": timed,
                "per_launch_events": {"avg_launch_ms": ev_ms, "achieved": ev_achieved, "frac": ev_achieved / hbm_gbs}}

    # combined roofline of the whole step: per layer-step max(resident bytes / HBM peak, offloaded bytes / link)
    h2d = None
    if h2d_before:
        h2d = 0.5 * (h2d_before + h2d_after)
    t_star = 0.0
    per_ls_res = bytes_res / n_launch
    per_ls_off = bytes_off / n_launch
    t_star = max(per_ls_res / (hbm_gbs * 1e9), per_ls_off / (h2d * 1e9) if h2d else 0.0)
    roof_tps = w.batch / (w.layers * t_star) * world if t_star > 0 else None
    combined = {"hbm_gbs": hbm_gbs, "h2d_gbs": h2d, "h2d_gbs_before_after": [h2d_before, h2d_after],
                "resident_bytes_per_layer_step": per_ls_res, "offloaded_bytes_per_layer_step": per_ls_off,
                "staged_bytes_per_layer_step": staged / n_launch,
                "roofline_tokens_per_s": roof_tps, "frac": (value / roof_tps) if roof_tps else None,
                "paper_serial_sum_ms_per_layer_step":
                    (per_ls_res / (hbm_gbs * 1e9) + (per_ls_off / (h2d * 1e9) if h2d else 0.0)) * 1e3}
    prefill_store = None
    if store["layers"] and store["ms"] > 0:
        gbs = store["bytes"] / (store["ms"] * 1e-3) / 1e9
        prefill_store = {"bytes_per_layer": store["bytes"] / store["layers"],
                         "store_ms_per_layer": store["ms"] / store["layers"],
                         "copies_per_layer": store["copies"] / store["layers"], "achieved_GBps": gbs,
                         "d2h_peak_GBps": probe_before[1], "frac": gbs / probe_before[1],
                         "what": "prompt write-back of the offloaded share (T_trans^p), device-to-host copies of isv_kv_fill"}
    breakdown = {k: v / n_launch for k, v in
                 {"append_ms": t_app, "attn_resident_ms": t_res, "h2d_ms": t_h2d, "attn_offloaded_ms": t_off,
                  "merge_ms": t_merge, "total_ms": t_tot}.items()}

    # -------- pass 3: end to end through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        B.isv_kv_reset(h)
        fill()
        hq = [torch.empty((w.layers, w.batch, w.q_heads, w.head_dim), dtype=td).pin_memory().copy_(qs[i].cpu())
              for i in range(2)]
        hk = [torch.empty((w.layers, w.batch, w.kv_heads, w.head_dim), dtype=td).pin_memory().copy_(ks[i].cpu())
              for i in range(2)]
        hv = [torch.empty((w.layers, w.batch, w.kv_heads, w.head_dim), dtype=td).pin_memory().copy_(vs[i].cpu())
              for i in range(2)]
        hout = torch.empty((w.layers, w.batch, w.q_heads, w.head_dim), dtype=td).pin_memory()
        for i in range(Wm):
            B.isv_decode_step_host(h, hq[i % 2], hk[i % 2], hv[i % 2], hout, w.batch)
        barrier()
        t0 = time.perf_counter()
        for i in range(K):
            B.isv_decode_step_host(h, hq[i % 2], hk[i % 2], hv[i % 2], hout, w.batch)
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        e2e_s = max_over_ranks(t1 - t0)
        e2e = {"value": R.aggregate_tokens_per_s(w.batch, K, e2e_s * 1e3, world), "unit": UNIT,
               "h2d_bytes_per_step": int(hq[0].numel() * 2 + hk[0].numel() * 2 + hv[0].numel() * 2),
               "d2h_bytes_per_step": int(hout.numel() * 2), "ms_per_step": e2e_s / K * 1e3,
               "api": "isv_decode_step_host (pinned host q/k/v in, out back, every step)"}
    B.isv_kv_free(h)

    # -------- CPU reference beside it (rank 0, single-GPU runs only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # C2 and the OPT-2.7B shape: the whole batch, i.e. one full layer-step; the larger shapes: 4 sequences scaled up
        n_sample = w.batch if w.name in ("c2", "tiny", "opt2.7b") else min(w.batch, 4)
        tps, t, threads, what = time_reference(w, n_sample, 3, 1)
        tps1, t1_, _, what1 = time_reference(w, min(w.batch, 2), 1, 0, n_threads=1)
        cpu = {"value": tps, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": what,
               "seconds_per_sampled_call": t,
               "one_thread": {"value": tps1, "unit": UNIT, "cores": 1, "sample": what1,
                              "seconds_per_sampled_call": t1_}}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f16" if w.dtype == "f16" else "bf16", "data": "synthetic",
            "config": workload_config(w, args, info), "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "combined_roofline": combined, "per_layer_step_ms": breakdown, "prefill_store": prefill_store,
            "cpu_baseline": cpu, "device_status": status,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--offload", type=float, default=None)
    ap.add_argument("--phys-layers", type=int, default=0)
    ap.add_argument("--layers", type=int, default=None, help="override the layer count (small profiling cases)")
    ap.add_argument("--batch", type=int, default=None, help="override the batch size (small profiling cases)")
    ap.add_argument("--zero-copy", action="store_true", help="read offloaded blocks in place instead of staging them")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    from paper_2504_11816_b200 import workloads as W
    w = W.CONFIGS[args.workload]
    if args.offload is not None:
        w = w.with_(offload_frac=args.offload)
    if args.layers is not None:
        w = w.with_(layers=args.layers)
    if args.batch is not None:
        w = w.with_(batch=args.batch)
    if args.steps is None:
        args.steps = 128 if args.impl == "ours" and w.offload_frac == 0 else (5 if args.impl == "reference" else 4)
    if args.warmup < 0 or args.steps < 1:
        raise SystemExit("steps must be >= 1 and warmup >= 0")
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
