#!/usr/bin/env python
"""Benchmark of the offloaded-KV decode path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload sweep|c2|c3|c4|c5|opt2.7b|tiny] [--offload F] [--phys-layers P]

A step is one decode step of the whole batch through all layers (KV append +
attention per layer).  One JSON line is printed by rank 0.

The default workload is the offload sweep the metric is named after: the
13B-shaped ragged batch (c5) at offload fractions 0 / 0.25 / 0.5 / 0.75 / 1, the
7B-shaped batches with nothing (c2) and half (c3) of the cache offloaded, the
8B-GQA batch with three quarters (c4) and nothing offloaded, and the paper's
own OPT-2.7B offline shape at its Table VI offload ratios (0 / 0.6 / 1).  The headline figures (`value`, `config`, `roofline`, `e2e`) are
those of c5 at offload fraction 0.5, timed for exactly --steps steps after
--warmup warm-up steps; every other point is listed under `sweep` with its own
step counts, its tokens/s, its fraction of the combined HBM / host-link
roofline, the resident kernel's HBM rate and the achieved and probed host-link
rates.  `--workload X` times that single configuration instead.

With N > 1 every rank runs an independent replica of the workload on its own
GPU (the path has no exchange step); times are the maximum over ranks.  Started
without a launcher, `--gpus N` starts its own N ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
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
HEADLINE = ("c5", 0.5)

# DRAM traffic of the resident decode kernel from one ncu capture (bytes per KV byte
# processed), valid only for the kernel source it was taken from.
NCU_TRAFFIC = {"kernels_sha1": "44aed6d32aaf25000f3eb95c035535f0ed28b65a",
               # multi-head shapes (CUDA-core arithmetic): (1094.13 MB read + 5.94 MB written) / 1078.46 MB
               # algorithmic, 2-layer case of the 7B shape (one launch per step)
               "dram_bytes_per_kv_byte": (1094.131 + 5.939) / 1078.460416,
               "source": "profiles/decode_kernel_c2_2layers.md",
               # grouped-query shapes (tensor-core arithmetic): (1080.11 MB + 5.11 MB) / 1074.92 MB, 32 sequences
               # and 2 layers of the 8B-GQA shape
               "dram_bytes_per_kv_byte_gqa": (1080.107 + 5.109) / 1074.921472,
               "source_gqa": "profiles/decode_kernel_gqa_c4shape_batch32_2layers.md"}


def kernels_sha1() -> str:
    """Hash of the decode kernels' code: comments and white space do not count, anything else does."""
    import re
    h = hashlib.sha1()
    for f in ("isv_kernels.cu", "isv_kernels.cuh"):
        src = open(os.path.join(ROOT, "paper_2504_11816_b200", "csrc", f), "r").read()
        src = re.sub(r"/\*.*?\*/", " ", src, flags=re.S)
        src = re.sub(r"//[^\n]*", " ", src)
        h.update(" ".join(src.split()).encode())
    return h.hexdigest()


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU (addressed by UUID, so that a process that
    sees only some of the machine's GPUs still reads its own) with nvidia-smi for the whole run; regions
    are cut out of the samples by host time afterwards.  Query only."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_id: str, period_ms: int = 50):
        self.gpu = gpu_id
        self.period_ms = period_ms
        self.proc = None
        self.samples = []          # (host time, sm, max sm, power, [reasons])

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", str(self.period_ms)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm, mx = float(parts[1]), float(parts[2])
            except ValueError:
                continue
            try:
                pw = float(parts[3])
            except ValueError:
                pw = None
            reasons = [n for n, v in zip(self.NAMES, parts[4:8]) if v.lower().startswith("active")]
            self.samples.append((time.time(), sm, mx, pw, reasons))

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def region(self, t0: float, t1: float):
        """Summary of the samples taken in [t0, t1] (host time)."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        rows = [r for r in self.samples if t0 <= r[0] <= t1]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["clocks not observed: no sample fell inside "
                                                                   "the region"], "samples": 0}
        reasons = sorted({x for r in rows for x in r[4]})
        pw = [r[3] for r in rows if r[3] is not None]
        return {"sm_mhz": float(np.median([r[1] for r in rows])), "sm_max_mhz": max(r[2] for r in rows),
                "sm_mhz_min": min(r[1] for r in rows), "power_w_max": max(pw) if pw else None,
                "reasons": reasons, "samples": len(rows)}


def device_uuid(index: int) -> str:
    """nvidia-smi's name for torch's device `index` (indices differ when only some GPUs are visible)."""
    import torch
    try:
        u = str(torch.cuda.get_device_properties(index).uuid)
        return u if u.startswith("GPU-") else "GPU-" + u
    except Exception:
        vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
        ids = [x for x in vis.split(",") if x.strip()]
        return ids[index] if index < len(ids) else str(index)


# ---------------------------------------------------------------- workloads and the sweep

def workload_config(w, zero_copy=False, note=None):
    """What is measured, from the workload alone (both arms print the same object)."""
    c = {"workload": f"{w.name}: {w.layers} layers, {w.q_heads} q / {w.kv_heads} kv heads x {w.head_dim}, "
                     f"{w.dtype}, batch {w.batch}, prompt {w.ctx_min}"
                     + (f"..{w.ctx_max}" if w.ctx_max != w.ctx_min else "")
                     + f" tokens, KV block {w.block_tokens}, offload {w.offload_frac:g}",
         "offload_frac": w.offload_frac, "batch": w.batch, "layers": w.layers, "accumulate": "f32",
         "l2": "KV read per layer-step exceeds L2 (inputs larger than L2)", "parallelism": "replicas",
         "offloaded_path": "zero-copy reads" if zero_copy else "staged through the ring"}
    if note:
        c["note"] = note
    return c


def sweep_points(K, Wm, layers=None, batch=None):
    """(workload, timed steps, warm-up steps, repetitions, reset between repetitions) per point.  Points where
    nothing is offloaded run in milliseconds per step: three repetitions of a region inside the
    configuration's own number of decode steps, the median reported.  Link-bound points take seconds per
    step: one region of 4 steps after 3 warm-up steps, except the headline, which takes K and Wm as given."""
    from paper_2504_11816_b200 import workloads as W
    C = W.CONFIGS
    pts = [(C["c2"], 120, max(3, min(Wm, 8)), 3, True),
           (C["opt2.7b"], 120, max(3, min(Wm, 8)), 3, True),
           (C["opt2.7b"].with_(offload_frac=0.6), 4, 3, 1, False),    # the offload ratios of the paper's Table VI
           (C["opt2.7b"].with_(offload_frac=1.0), 4, 3, 1, False),
           (C["c3"], 4, 3, 1, False),
           (C["c4"], 4, 3, 1, False),
           (C["c4"].with_(offload_frac=0.0), 9, 3, 3, False),     # the grouped-query (tensor-core) variant at the HBM rate
           (C["c5"].with_(offload_frac=0.0), 9, 3, 3, False)]
    for f in (0.25, 0.5, 0.75, 1.0):
        if ("c5", f) == HEADLINE:
            pts.append((C["c5"].with_(offload_frac=f), K, Wm, 1, False))
        else:
            pts.append((C["c5"].with_(offload_frac=f), 4, 3, 1, False))
    over = {k_: v_ for k_, v_ in (("layers", layers), ("batch", batch)) if v_ is not None}   # small test runs
    return [(w.with_(**over), k_pt, w_pt, reps, reset) for (w, k_pt, w_pt, reps, reset) in pts]


def choose_phys_layers(w, max_tokens, requested, local_ranks=1):
    """Physical KV slabs to hold: as many as fit a budget (0.7 of free HBM; 24 GiB or this rank's share of a
    third of the available host memory for the pinned pool), at most `layers`.  Every slab is far larger than L2."""
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
    host_budget = min(0.35 * avail / max(1, local_ranks), 24 << 30)
    p = w.layers
    if hbm_layer:
        p = min(p, int(hbm_budget // hbm_layer))
    if host_layer:
        p = min(p, int(host_budget // host_layer))
    return max(1, p)


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
    layers, seconds per sampled call, seconds a whole step would take at that rate,
    threads, description of the sample)."""
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
    return tps, t, w.layers * t_layer_step, (n_threads or oa.max_threads()), \
        f"{n_sample} of {w.batch} sequences x {w.q_heads} heads, one layer-step " \
        f"(contexts {int(ctx.min())}..{int(ctx.max())}), scaled by attended tokens to the batch and x{w.layers} layers"


def headline_workload(args):
    from paper_2504_11816_b200 import workloads as W
    if args.workload == "sweep":
        w = W.CONFIGS[HEADLINE[0]].with_(offload_frac=HEADLINE[1])
        note = "headline point of the offload sweep (the other points are listed under `sweep`)"
    else:
        w = W.CONFIGS[args.workload]
        note = None
        if args.offload is not None:
            w = w.with_(offload_frac=args.offload)
    if args.layers is not None:
        w = w.with_(layers=args.layers)
    if args.batch is not None:
        w = w.with_(batch=args.batch)
    return w, note


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w, note = headline_workload(args)
    n_sample = min(w.batch, 8 if w.name in ("c2", "opt2.7b") else 4)
    tps, t, t_step, threads, what = time_reference(w, n_sample, args.steps, args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, args.zero_copy, note),
        "cpu_baseline": {"value": tps, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": what,
                         "seconds_per_sampled_call": t,
                         "ms_per_step_is": "the time one whole step (all sequences, all layers) takes at the "
                                           "sampled rate; each of the timed steps ran the sample only"},
        "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------- our arm: one point

class Ctx:
    """Process-wide state of a run of the CUDA arm."""
    def __init__(self, args):
        import torch
        import torch.distributed as dist
        self.torch, self.dist = torch, dist
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (no CPU path exists)")
        if self.world != args.gpus:
            raise SystemExit(f"--gpus {args.gpus} but the launcher started {self.world} ranks")
        if torch.cuda.device_count() <= self.local_rank:
            raise SystemExit(f"rank {self.rank} needs GPU {self.local_rank} but only {torch.cuda.device_count()} "
                             "are visible")
        torch.cuda.set_device(self.local_rank)
        if self.world > 1:
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local_rank))
        self.hbm_gbs, self.peak_kind = measured_peaks()
        self.stream = torch.cuda.Stream()
        self.sampler = ClockSampler(device_uuid(self.local_rank))
        self.args = args

    def barrier(self):
        from paper_2504_11816_b200 import replicas as R
        self.torch.cuda.synchronize()
        R.barrier(self.dist)
        self.torch.cuda.synchronize()

    def max_over_ranks(self, x: float) -> float:
        from paper_2504_11816_b200 import replicas as R
        return R.max_over_ranks(x, self.dist, device="cuda")


def measure_point(cx: Ctx, w, K, Wm, reps, reset_between, want_e2e, phys_req=0):
    """Times one configuration.  Returns a dict with tokens/s (median over the repetitions), the resident
    kernel's HBM rate, the host-link rates, the combined roofline and what was run."""
    import torch
    from paper_2504_11816_b200 import binding as B
    from paper_2504_11816_b200 import replicas as R
    from paper_2504_11816_b200 import workloads as W
    args = cx.args
    offloaded = w.offload_frac > 0
    stream = cx.stream
    extra = (Wm + K) if want_e2e else 0
    total_steps = (Wm + K) if reset_between else (Wm + reps * K)
    max_tokens = w.ctx_max + total_steps + extra + 1
    lens = W.prompt_lens(w)
    phys = choose_phys_layers(w, max_tokens, phys_req, cx.world)
    t_alloc = time.perf_counter()
    h = B.isv_kv_alloc(**B.desc_from_workload(w, phys_layers=phys, max_tokens_per_seq=max_tokens,
                                              compute_stream=stream.cuda_stream))
    t_alloc = time.perf_counter() - t_alloc
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

    def step(i):
        B.isv_decode_step(h, qs[i % n_in], ks[i % n_in], vs[i % n_in], out, None, w.batch)

    t_fill = time.perf_counter()
    fill(measure_store=offloaded)
    t_fill = time.perf_counter() - t_fill
    probe_before = B.isv_link_probe(1 << 30, 10) if offloaded else None

    # per-launch events are on where they cost nothing (layer-steps of milliseconds); where a layer-step is
    # one short kernel the region's two events time it better (per-launch events add gaps)
    B.isv_set_timing(h, offloaded)
    regions = []          # per repetition: ms, bytes_res, bytes_off, bytes_staged, launches, host times
    last_step = None
    step_ms_all = []
    for rep in range(reps):
        if rep > 0 and reset_between:
            B.isv_kv_reset(h)
            fill()
            B.isv_set_timing(h, offloaded)
        t_w0 = time.time()
        if rep == 0 or reset_between:
            for i in range(Wm):
                step(i)
            B.isv_sync(h)
        launches0 = B.isv_kv_info(h).kernel_launches
        b_res = b_off = b_staged = 0
        cx.barrier()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
        t_r0 = time.time()
        evs[0].record(stream)
        for i in range(K):
            step(i)
            r, o, sg, _ = B.isv_plan_bytes(h, 0, w.batch)       # bytes of the step just enqueued (host bookkeeping)
            b_res += r * w.layers
            b_off += o * w.layers
            b_staged += sg * w.layers
            if offloaded:
                evs[i + 1].record(stream)
        if not offloaded:
            evs[K].record(stream)
        cx.barrier()
        t_r1 = time.time()
        ms = cx.max_over_ranks(evs[0].elapsed_time(evs[K]))
        if offloaded:
            step_ms_all += [evs[i].elapsed_time(evs[i + 1]) for i in range(K)]
            last_step = B.isv_step_timing(h, -1)
        status = B.isv_sync(h)
        regions.append({"ms": ms, "bytes_res": b_res, "bytes_off": b_off, "bytes_staged": b_staged,
                        "launches": B.isv_kv_info(h).kernel_launches - launches0, "t0": t_r0, "t1": t_r1,
                        "t_warm0": t_w0, "status": status})
    B.isv_set_timing(h, False)
    probe_after = B.isv_link_probe(1 << 30, 10) if offloaded else None

    order = sorted(range(reps), key=lambda i: regions[i]["ms"])
    med = regions[order[len(order) // 2]]
    ms = med["ms"]
    value = R.aggregate_tokens_per_s(w.batch, K, ms, cx.world)
    n_launch = K * w.layers
    per_ls_res = med["bytes_res"] / n_launch
    per_ls_off = med["bytes_off"] / n_launch

    # ---- the resident kernel against the HBM rate
    hbm_gbs = cx.hbm_gbs
    if offloaded:
        # the last timed step's launches, each bracketed by its own events
        avg_ms = last_step.attn_resident_ms / w.layers
        res_bytes_launch = last_step.bytes_resident / w.layers
        timed = "CUDA events around every launch of the last timed step (a launch lasts far longer than an event gap)"
    else:
        # nothing offloaded: the region holds decode_kernel launches and nothing else (bar a table update every
        # 16 steps) - one per step covering all layers, or one per layer-step where that is switched off
        whole_step = med["launches"] < n_launch
        dec_launches = K if whole_step else n_launch
        avg_ms = ms / dec_launches
        res_bytes_launch = med["bytes_res"] / dec_launches
        timed = ("CUDA events around the timed region / decode_kernel launches in it (one launch per "
                 + ("step, covering all layers" if whole_step else "layer-step")
                 + "; includes the gaps between launches)")
    achieved = res_bytes_launch / (avg_ms * 1e-3) / 1e9 if avg_ms > 0 else 0.0
    traffic = None
    if NCU_TRAFFIC["kernels_sha1"] == kernels_sha1():   # counters taken from this very kernel source
        gqa = w.q_heads // w.kv_heads >= 2               # those shapes run the tensor-core variant
        ratio = NCU_TRAFFIC["dram_bytes_per_kv_byte_gqa" if gqa else "dram_bytes_per_kv_byte"]
        traffic = ratio * res_bytes_launch if ratio else None
    roofline = {"bound": "hbm", "kernel": "decode_kernel (resident, split flash-decoding)",
                "achieved": achieved, "peak": hbm_gbs, "unit": "GB/s", "frac": achieved / hbm_gbs,
                "peak_kind": f"of {cx.peak_kind}", "traffic": traffic,
                "bytes_per_launch": res_bytes_launch, "avg_launch_ms": avg_ms, "timed": timed}

    # ---- combined roofline of the whole step: per layer-step max(resident bytes / HBM peak, offloaded bytes / link)
    # the link's rate is the better of the two probes: a probe that another tenant of the host disturbed reads low
    # and would push the fraction above what the link allows (seen once: 55.6 before, 51.4 after a point)
    h2d = max(probe_before[0], probe_after[0]) if offloaded else None
    t_star = max(per_ls_res / (hbm_gbs * 1e9), per_ls_off / (h2d * 1e9) if h2d else 0.0)
    roof_tps = w.batch / (w.layers * t_star) * cx.world if t_star > 0 else None
    combined = {"hbm_gbs": hbm_gbs, "h2d_gbs": h2d,
                "h2d_gbs_before_after": [probe_before[0], probe_after[0]] if offloaded else None,
                "h2d_gbs_achieved": (med["bytes_staged"] / (ms * 1e-3) / 1e9) if offloaded else None,
                "resident_bytes_per_layer_step": per_ls_res, "offloaded_bytes_per_layer_step": per_ls_off,
                "staged_bytes_per_layer_step": med["bytes_staged"] / n_launch,
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
    breakdown = None
    if last_step is not None:
        breakdown = {k_: getattr(last_step, k_) / w.layers for k_ in
                     ("attn_resident_ms", "h2d_ms", "attn_offloaded_ms", "merge_ms", "total_ms")}

    clocks = cx.sampler.region(med["t0"], med["t1"])
    if clocks.get("sm_mhz"):
        clocks["ms_per_step_x_sm_mhz"] = ms / K * clocks["sm_mhz"]

    # ---- end to end through the host-buffer entry point (pinned host q/k/v in, out back, every step)
    e2e = None
    if want_e2e:
        hq = [torch.empty((w.layers, w.batch, w.q_heads, w.head_dim), dtype=td).pin_memory().copy_(qs[i].cpu())
              for i in range(2)]
        hk = [torch.empty((w.layers, w.batch, w.kv_heads, w.head_dim), dtype=td).pin_memory().copy_(ks[i].cpu())
              for i in range(2)]
        hv = [torch.empty((w.layers, w.batch, w.kv_heads, w.head_dim), dtype=td).pin_memory().copy_(vs[i].cpu())
              for i in range(2)]
        hout = torch.empty((w.layers, w.batch, w.q_heads, w.head_dim), dtype=td).pin_memory()
        if reset_between:
            B.isv_kv_reset(h)
            fill()
        for i in range(Wm):
            B.isv_decode_step_host(h, hq[i % 2], hk[i % 2], hv[i % 2], hout, w.batch)
        cx.barrier()
        t0 = time.perf_counter()
        for i in range(K):
            B.isv_decode_step_host(h, hq[i % 2], hk[i % 2], hv[i % 2], hout, w.batch)
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        e2e_s = cx.max_over_ranks(t1 - t0)
        e2e = {"value": R.aggregate_tokens_per_s(w.batch, K, e2e_s * 1e3, cx.world), "unit": UNIT,
               "h2d_bytes_per_step": int(hq[0].numel() * 2 + hk[0].numel() * 2 + hv[0].numel() * 2),
               "d2h_bytes_per_step": int(hout.numel() * 2), "ms_per_step": e2e_s / K * 1e3,
               "api": "isv_decode_step_host (pinned host q/k/v in, out back, every step)"}
        del hq, hk, hv, hout
    B.isv_kv_free(h)
    del qs, ks, vs, out
    torch.cuda.empty_cache()

    return {"workload": w, "value": value, "ms": ms, "ms_per_step": ms / K, "steps": K, "warmup": Wm,
            "repetitions": {"n": reps, "ms": [r["ms"] for r in regions], "reported": "median",
                            "reset_and_reload_between": bool(reset_between),
                            "per_step_ms": ({"min": min(step_ms_all), "median": float(np.median(step_ms_all)),
                                             "max": max(step_ms_all)} if step_ms_all else None)},
            "launches": int(med["launches"]), "status": int(max(r["status"] for r in regions)),
            "roofline": roofline, "combined": combined, "prefill_store": prefill_store, "breakdown": breakdown,
            "clocks": clocks, "e2e": e2e,
            "engine": {"phys_layers": info.phys_layers, "max_ctas": info.max_ctas, "chunk_bytes": info.chunk_bytes,
                       "ring_depth": info.ring_depth, "alloc_s": t_alloc, "fill_s": t_fill}}


def point_summary(p):
    """One entry of the `sweep` array."""
    w = p["workload"]
    c = p["combined"]
    return {"workload": workload_config(w)["workload"], "name": w.name, "offload_frac": w.offload_frac,
            "tokens_per_s": p["value"], "ms_per_step": p["ms_per_step"], "steps": p["steps"], "warmup": p["warmup"],
            "repetitions": p["repetitions"], "combined_roofline_frac": c["frac"],
            "roofline_tokens_per_s": c["roofline_tokens_per_s"],
            "resident_GBps": p["roofline"]["achieved"], "resident_frac_of_hbm": p["roofline"]["frac"],
            "resident_timed": p["roofline"]["timed"],
            "h2d_GBps_achieved": c["h2d_gbs_achieved"], "h2d_GBps_probed_before_after": c["h2d_gbs_before_after"],
            "resident_bytes_per_layer_step": c["resident_bytes_per_layer_step"],
            "offloaded_bytes_per_layer_step": c["offloaded_bytes_per_layer_step"],
            "phys_layers": p["engine"]["phys_layers"], "gpu_launches": p["launches"],
            "prefill_store": p["prefill_store"], "clocks": p["clocks"], "device_status": p["status"],
            "e2e_tokens_per_s": p["e2e"]["value"] if p["e2e"] else None}


# ---------------------------------------------------------------- decode linear layers (extra key)

LINEAR_MODELS = {"llama7b": (4096, 11008, True), "opt2.7b": (2560, 10240, False)}


def linear_layers_bench(cx: Ctx, model="llama7b", batches=(1, 32, 64, 128), iters=40, eager=False):
    """Times the four projections of one transformer layer (fused QKV, output, MLP up, MLP down) through
    isv_linear_forward: the linear-layer term of T_compute^d.  Each call streams its weight matrix once;
    the figure of merit is weight bytes / time against the HBM rate.  Several weight buffers are cycled so
    that no call finds its weights in L2, and the calls are captured in a CUDA graph so that the host's
    launch rate does not enter (`eager`: plain calls instead, so that a profiler sees ordinary launches)."""
    import torch
    from paper_2504_11816_b200 import binding as B
    h1, h2, gated = LINEAR_MODELS[model]
    shapes = [("qkv", 3 * h1, h1), ("out", h1, h1), ("mlp_up", (2 if gated else 1) * h2, h1), ("mlp_down", h1, h2)]
    stream = torch.cuda.Stream()
    res = {"model": model, "hbm_peak_GBps": cx.hbm_gbs, "timed": "plain calls" if eager else "CUDA graph of the calls",
           "batches": []}
    floor_us = sum(N * K * 2 for _, N, K in shapes) / (cx.hbm_gbs * 1e9) * 1e6
    for M in batches:
        rows, total_s = [], 0.0
        for name, N, K in shapes:
            wbytes = N * K * 2
            copies = max(2, int((512 << 20) // wbytes) + 1)          # > L2 in total
            g = torch.Generator(device="cuda")
            g.manual_seed(N * 31 + K)
            ws = [(torch.randn((N, K), generator=g, device="cuda", dtype=torch.float32) / K ** 0.5).half()
                  for _ in range(copies)]
            x = torch.randn((M, K), generator=g, device="cuda", dtype=torch.float32).half()
            y = torch.zeros((M, N), device="cuda", dtype=torch.float16)
            torch.cuda.synchronize()
            hs = [B.isv_linear_create(wt, N, K, B.ISV_F16, max(M, 16), stream.cuda_stream) for wt in ws]
            try:
                for hl in hs:
                    B.isv_linear_forward(hl, x, y, None, M)
                assert B.isv_linear_status(hs[0]) == 0
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                def calls():
                    for i in range(iters):
                        B.isv_linear_forward(hs[i % copies], x, y, None, M)
                graph = None
                if not eager:
                    graph = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(graph, stream=stream):
                        calls()
                    graph.replay()
                stream.synchronize()
                torch.cuda.synchronize()
                with torch.cuda.stream(stream):
                    e0.record(stream)
                    calls() if eager else graph.replay()
                    e1.record(stream)
                stream.synchronize()
                torch.cuda.synchronize()
                t = e0.elapsed_time(e1) * 1e-3 / iters
                ref = torch.nn.functional.linear(x.float(), ws[(iters - 1) % copies].float())
                err = float((y.float() - ref).abs().max())
                del graph
            finally:
                for hl in hs:
                    B.isv_linear_free(hl)
            rows.append({"layer": name, "N": N, "K": K, "us": t * 1e6, "weight_GBps": wbytes / t / 1e9,
                         "frac": wbytes / t / 1e9 / cx.hbm_gbs, "max_abs_diff_vs_fp32_gemm": err})
            total_s += t
            del ws
            torch.cuda.empty_cache()
        res["batches"].append({"batch": M, "rows": rows, "us_per_layer": total_s * 1e6,
                               "floor_us_per_layer": floor_us, "frac": floor_us / (total_s * 1e6)})
    return res


def run_linear(args):
    """`--workload linear`: the decode linear layers alone, at one batch size (`--batch`, default 32) and
    `--steps` calls per matrix; its own JSON line, not the metric's."""
    cx = Ctx(args)
    from paper_2504_11816_b200 import binding as B
    B.lib()
    res = linear_layers_bench(cx, batches=(args.batch or 32,), iters=args.steps, eager=args.linear_eager)
    if cx.rank == 0:
        print(json.dumps({"linear_layers": res}))
    if cx.world > 1:
        cx.dist.destroy_process_group()


# ---------------------------------------------------------------- our arm: the line

def run_ours(args):
    import torch
    from paper_2504_11816_b200 import binding as B
    from paper_2504_11816_b200 import workloads as W
    cx = Ctx(args)
    B.lib()
    cx.sampler.start()
    torch.cuda.synchronize()
    K, Wm = args.steps, args.warmup
    head_w, note = headline_workload(args)

    sweep, head = [], None
    if args.workload == "sweep":
        for (w, k_pt, w_pt, reps, reset) in sweep_points(K, Wm, args.layers, args.batch):
            is_head = (w.name, w.offload_frac) == HEADLINE
            p = measure_point(cx, w, k_pt, w_pt, reps, reset, want_e2e=is_head and not args.no_e2e,
                              phys_req=args.phys_layers if is_head else 0)
            sweep.append(point_summary(p))
            if is_head:
                head = p
            if cx.rank == 0:
                print(f"[bench] {w.name} f={w.offload_frac:g}: {p['value']:.1f} tokens/s, combined roofline "
                      f"{p['combined']['frac']:.3f}, resident {p['roofline']['achieved']:.0f} GB/s", file=sys.stderr)
    else:
        reps = 3 if head_w.offload_frac == 0 else 1
        head = measure_point(cx, head_w, K, Wm, reps, reset_between=head_w.offload_frac == 0,
                             want_e2e=not args.no_e2e, phys_req=args.phys_layers)

    linear = None
    if args.workload == "sweep" and not args.no_linear:
        linear = linear_layers_bench(cx)
    cx.sampler.stop()

    # -------- CPU reference beside it (rank 0, single-GPU runs only)
    cpu = None
    w = head["workload"]
    if cx.rank == 0 and cx.world == 1 and not args.no_cpu_baseline:
        # the 7B and OPT-2.7B shapes: the whole batch, i.e. one full layer-step; the larger shapes: 4 sequences scaled up
        n_sample = w.batch if w.name in ("c2", "tiny", "opt2.7b") else min(w.batch, 4)
        tps, t, _, threads, what = time_reference(w, n_sample, 3, 1)
        tps1, t1_, _, _, what1 = time_reference(w, min(w.batch, 2), 1, 0, n_threads=1)
        cpu = {"value": tps, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": what,
               "seconds_per_sampled_call": t,
               "one_thread": {"value": tps1, "unit": UNIT, "cores": 1, "sample": what1,
                              "seconds_per_sampled_call": t1_}}

    if cx.rank == 0:
        fracs = [s["combined_roofline_frac"] for s in sweep if s["combined_roofline_frac"] is not None]
        line = {
            "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": cx.world, "steps": head["steps"],
            "warmup": head["warmup"], "ms_per_step": head["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16" if w.dtype == "f16" else "bf16",
            "data": "synthetic", "config": workload_config(w, args.zero_copy, note), "engine": head["engine"],
            "clocks": head["clocks"], "e2e": head["e2e"], "gpu_launches": head["launches"],
            "roofline": head["roofline"], "combined_roofline": head["combined"],
            "per_layer_step_ms": head["breakdown"], "prefill_store": head["prefill_store"],
            "repetitions": head["repetitions"],
            "sweep": sweep if sweep else None, "min_frac_over_sweep": min(fracs) if fracs else None,
            "linear_layers": linear, "cpu_baseline": cpu, "device_status": head["status"],
        }
        print(json.dumps(line))
    if cx.world > 1:
        cx.dist.destroy_process_group()


# ---------------------------------------------------------------- launcher

def free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def spawn_ranks(n: int) -> int:
    """Starts this script as n ranks on this node (one per GPU) and returns their exit code."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_launch_selftest(args):
    """Rank plumbing without a GPU: every rank 'times' a rank-dependent sleep, the ranks meet at a barrier and
    agree on the slowest time over gloo, rank 0 prints the line.  Exercises exactly the launcher and the
    reductions the CUDA arm uses."""
    import torch.distributed as dist
    from paper_2504_11816_b200 import replicas as R
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but the launcher started {world} ranks")
    if world > 1:
        dist.init_process_group("gloo")
    R.barrier(dist)
    t0 = time.perf_counter()
    time.sleep(0.02 * (rank + 1))
    mine = (time.perf_counter() - t0) * 1e3
    R.barrier(dist)
    worst = R.max_over_ranks(mine, dist)
    if rank == 0:
        print(json.dumps({"selftest": "launch", "n_gpus": world, "ms": worst, "slowest_rank_expected": world - 1,
                          "value": R.aggregate_tokens_per_s(1, 1, worst, world)}))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="sweep")
    ap.add_argument("--offload", type=float, default=None)
    ap.add_argument("--phys-layers", type=int, default=0)
    ap.add_argument("--layers", type=int, default=None, help="override the layer count (small profiling cases)")
    ap.add_argument("--batch", type=int, default=None, help="override the batch size (small profiling cases)")
    ap.add_argument("--zero-copy", action="store_true", help="read offloaded blocks in place instead of staging them")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-linear", action="store_true", help="skip the decode linear layers' figures")
    ap.add_argument("--linear-eager", action="store_true",
                    help="with --workload linear: plain calls instead of a CUDA graph (for a profiler)")
    ap.add_argument("--selftest-launch", action="store_true",
                    help="exercise the launcher and the rank reductions on CPU (gloo); no GPU work")
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("--gpus must be >= 1")
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started without a launcher: become one
        if not args.selftest_launch and args.impl == "ours":
            import torch
            if torch.cuda.device_count() < args.gpus:
                raise SystemExit(f"--gpus {args.gpus} but only {torch.cuda.device_count()} GPUs are visible")
        raise SystemExit(spawn_ranks(args.gpus))
    from paper_2504_11816_b200 import workloads as W
    if args.workload == "linear" and args.impl == "ours" and not args.selftest_launch:
        args.steps = args.steps or 40
        return run_linear(args)
    if args.workload != "sweep" and args.workload not in W.CONFIGS:
        raise SystemExit(f"unknown workload {args.workload!r}")
    if args.selftest_launch:
        return run_launch_selftest(args)
    if args.steps is None:
        if args.impl == "reference":
            args.steps = 5
        elif args.workload == "sweep":
            args.steps = 8
        else:
            f = args.offload if args.offload is not None else W.CONFIGS[args.workload].offload_frac
            args.steps = 120 if f == 0 else 4
    if args.warmup < 0 or args.steps < 1:
        raise SystemExit("steps must be >= 1 and warmup >= 0")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
