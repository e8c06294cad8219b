"""The paper's performance and cost model around the measured decode path.

``isv_step_timing`` reports, per layer, the host-link time (the paper's
T_trans^d), the attention time (the self-attention part of T_compute^d) and
byte counters.  This module evaluates the paper's formulas for the same
quantities (Section IV-C, Eqs. 4-7), fits the compute-time calibration
CTCF(T) = alpha * T + beta to measurements by least squares as Section IV-E
describes, and provides the selection logic around them (Section III:
Eqs. 1-3; Section IV-B: Algorithm 1; Section IV-D: final selection), so that a
measured B200 can be placed in the paper's framework.  Host arithmetic only.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Iterable, List, Sequence, Tuple


@dataclass(frozen=True)
class ModelShape:
    h1: int            # hidden size (kv_heads * head_dim for the KV terms)
    h2: int            # MLP hidden size
    n_layers: int
    prec_bytes: int = 2


@dataclass(frozen=True)
class Machine:
    flops: float       # FLOP/s used for T_compute
    bw_h2d: float      # bytes/s host -> GPU
    bw_d2h: float      # bytes/s GPU -> host


# ---- memory (Table II)

def kv_cache_bytes(m: ModelShape, BS: int, tokens: int) -> int:
    return 2 * BS * tokens * m.h1 * m.prec_bytes * m.n_layers


def offload_ratio(mem_avail: float, mem_kvcache: float) -> float:
    return 1.0 - mem_avail / mem_kvcache


# ---- time (Section IV-C), all per layer

def t_compute_d(m: ModelShape, hw: Machine, BS: int, L_in: int, L_out: int) -> Tuple[float, float]:
    """(linear-layer seconds, self-attention seconds) of one decode step of one layer."""
    lin = BS * (8.0 * m.h1 * m.h1 + 4.0 * m.h1 * m.h2) / hw.flops
    att = 4.0 * BS * (L_in + L_out / 2.0) * m.h1 / hw.flops
    return lin, att


def t_trans_d(m: ModelShape, hw: Machine, BS: int, L_in: int, L_out: int, c_off: float) -> float:
    return (c_off * 2.0 * (L_in + 1) + L_out) * m.h1 * m.prec_bytes * BS / hw.bw_h2d


def t_compute_p(m: ModelShape, hw: Machine, BS: int, L_in: int) -> Tuple[float, float]:
    lin = BS * (8.0 * L_in * m.h1 * m.h1 + 4.0 * L_in * m.h1 * m.h2) / hw.flops
    att = 4.0 * BS * float(L_in) ** 2 * m.h1 / hw.flops
    return lin, att


def t_trans_p(m: ModelShape, hw: Machine, BS: int, L_in: int, c_off: float) -> float:
    return c_off * 2.0 * (L_in + 1) * m.h1 * m.prec_bytes * BS / hw.bw_d2h


def ctcf(t: float, alpha: float = 1.0, beta: float = 0.0) -> float:
    return alpha * t + beta


def t_dec(m, hw, BS, L_in, L_out, c_off, alpha=1.0, beta=0.0) -> float:
    """Eq. 6: calibrated compute plus transfer (a sum)."""
    return ctcf(sum(t_compute_d(m, hw, BS, L_in, L_out)), alpha, beta) + t_trans_d(m, hw, BS, L_in, L_out, c_off)


def t_pre(m, hw, BS, L_in, c_off, alpha=1.0, beta=0.0) -> float:
    """Eq. 5: calibrated compute and transfer overlap (a max)."""
    return max(ctcf(sum(t_compute_p(m, hw, BS, L_in)), alpha, beta), t_trans_p(m, hw, BS, L_in, c_off))


def t_task(m, hw, BS, L_in, L_out, c_off, alpha=1.0, beta=0.0) -> float:
    """Eq. 4."""
    return (t_pre(m, hw, BS, L_in, c_off, alpha, beta) * m.n_layers
            + t_dec(m, hw, BS, L_in, L_out, c_off, alpha, beta) * m.n_layers * (L_out - 1))


def tps(BS: int, L_in: int, L_out: int, t_e2e: float) -> float:
    """Eq. 1."""
    return BS * (L_in + L_out) / t_e2e


# ---- calibration (Section IV-E, Eq. 7)

def fit_ctcf(t_model: Sequence[float], t_measured: Sequence[float]) -> Tuple[float, float, float]:
    """Least-squares line t_measured ~ alpha * t_model + beta over the given points
    (the paper's pre-profiled batch sizes).  Returns (alpha, beta, mean absolute error in percent)."""
    n = len(t_model)
    if n != len(t_measured) or n < 2:
        raise ValueError("need at least two (model, measured) pairs")
    mx = sum(t_model) / n
    my = sum(t_measured) / n
    sxx = sum((x - mx) ** 2 for x in t_model)
    if sxx == 0.0:
        raise ValueError("model times are all equal")
    sxy = sum((x - mx) * (y - my) for x, y in zip(t_model, t_measured))
    alpha = sxy / sxx
    beta = my - alpha * mx
    err = sum(abs(alpha * x + beta - y) / y for x, y in zip(t_model, t_measured)) / n * 100.0
    return alpha, beta, err


# ---- cost (Section III, Eqs. 2-3) and selection (Algorithm 1, Section IV-D)

def cost_efficiency(tps_actual: float, tps_slo: float, BS: int, L_in: int, L_out: int, vm_price: float):
    """(CE, billed hours, TPS_effective) of a task of BS * (L_in + L_out) tokens."""
    eff = min(tps_actual, tps_slo)
    hours = BS * (L_in + L_out) / (eff * 3600.0)
    billed = math.ceil(hours)
    return eff * 3600.0 / (billed * vm_price), billed, eff


def candidate_instances(instances: Iterable[Tuple[str, float, float]], mem_model: float, mem_activation: float,
                        mem_kvcache: float, mem_kv_per_layer: float, p_max: float) -> List[Tuple[str, float, float]]:
    """Algorithm 1: [(name, C_off, price)] of the instances (name, GPU memory, price) that are
    affordable and can run the task with or without KV offloading, cheapest first."""
    base = mem_model + mem_activation
    total = base + mem_kvcache
    keep = []
    for name, gpu_mem, price in instances:
        if price > p_max:
            continue
        if gpu_mem >= total:
            keep.append((name, 0.0, price))
            continue
        avail = gpu_mem - base
        if gpu_mem < mem_model or mem_kv_per_layer > avail:
            continue                       # weights do not fit, or one layer's KV does not
        keep.append((name, offload_ratio(avail, mem_kvcache), price))
    return sorted(keep, key=lambda r: r[2])


def select_instance(cands: Iterable[Tuple[str, float, float]], tps_slo: float, BS: int, L_in: int, L_out: int):
    """Final selection: candidates (name, predicted TPS, price) meeting the SLO, ranked by cost
    efficiency, ties broken by higher TPS.  Returns [(name, TPS, price, CE)] best first."""
    ok = []
    for name, t, price in cands:
        if t >= tps_slo:
            ok.append((name, t, price, cost_efficiency(t, tps_slo, BS, L_in, L_out, price)[0]))
    return sorted(ok, key=lambda r: (-r[3], -r[1]))
