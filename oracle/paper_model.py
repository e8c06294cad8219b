"""The paper's memory and time formulas, written out term by term.

TEST INFRASTRUCTURE ONLY.  These restate Table II (memory) and Section IV-C
(Eqs. 4-6 and the unnumbered T_compute / T_trans formulas) plus Eq. 7 (CTCF)
so that the library's byte counters and timing terms can be checked against
them.  Symbols follow the paper: BS batch size, L_in / L_out input / output
lengths, h1 hidden size, h2 MLP hidden size, n layers, C_off offload ratio.
"""
from __future__ import annotations


def kv_cache_bytes(BS: int, tokens: int, h1: int, prec_bytes: int, n_layers: int) -> int:
    """Table II, KV cache memory: 2 * BS * (L_in + L_out) * h1 * Precision * n.
    (The table prints the head-count symbol where the transfer formulas print
    h1; h1 is the reading used, and ``tokens`` stands for L_in + L_out.)"""
    return 2 * BS * tokens * h1 * prec_bytes * n_layers


def attn_flops_decode(BS: int, ctx: float, h1: int) -> float:
    """Self-attention part of T_compute^d's numerator: 4 * BS * ctx * h1, with
    ctx the attended context (the paper averages it as L_in + L_out / 2)."""
    return 4.0 * BS * ctx * h1


def linear_flops_decode(BS: int, h1: int, h2: int) -> float:
    """Linear-layer part of T_compute^d's numerator: BS * (8 h1^2 + 4 h1 h2)."""
    return float(BS) * (8.0 * h1 * h1 + 4.0 * h1 * h2)


def t_trans_d_bytes(C_off: float, L_in: int, L_out: int, h1: int, prec_bytes: int, BS: int) -> float:
    """Numerator of T_trans^d as printed:
    (C_off * 2 * (L_in + 1) + L_out) * h1 * Precision * BS."""
    return (C_off * 2.0 * (L_in + 1) + L_out) * h1 * prec_bytes * BS


def offloaded_kv_bytes(C_off: float, tokens: int, h1: int, prec_bytes: int, BS: int) -> float:
    """First term of that numerator for a context of ``tokens``:
    C_off * 2 * tokens * h1 * Precision * BS."""
    return C_off * 2.0 * tokens * h1 * prec_bytes * BS


def t_trans_p_bytes(C_off: float, L_in: int, h1: int, prec_bytes: int, BS: int) -> float:
    """Numerator of T_trans^p: C_off * 2 * (L_in + 1) * h1 * Precision * BS."""
    return C_off * 2.0 * (L_in + 1) * h1 * prec_bytes * BS


def ctcf(t: float, alpha: float, beta: float) -> float:
    """Eq. 7: CTCF(T) = alpha * T + beta."""
    return alpha * t + beta


def t_dec(t_compute_d: float, t_trans_d: float, alpha: float = 1.0, beta: float = 0.0) -> float:
    """Eq. 6: T_dec = CTCF(T_compute^d) + T_trans^d (a sum, not a max)."""
    return ctcf(t_compute_d, alpha, beta) + t_trans_d


def t_pre(t_compute_p: float, t_trans_p: float, alpha: float = 1.0, beta: float = 0.0) -> float:
    """Eq. 5: T_pre = max(CTCF(T_compute^p), T_trans^p)."""
    return max(ctcf(t_compute_p, alpha, beta), t_trans_p)


def t_task(t_pre_layer: float, t_dec_layer: float, n_layers: int, L_out: int) -> float:
    """Eq. 4: T_task = T_pre * n + T_dec * n * (L_out - 1)."""
    return t_pre_layer * n_layers + t_dec_layer * n_layers * (L_out - 1)


def tps(BS: int, L_in: int, L_out: int, t_e2e: float) -> float:
    """Eq. 1: TPS = BS * (L_in + L_out) / T_E2E."""
    return BS * (L_in + L_out) / t_e2e


# ---------------------------------------------------------------- cost side: Eqs. 2-3, Algorithm 1, Step 4

import math


def tps_effective(tps_actual: float, tps_slo: float) -> float:
    """Section III-A: the effective rate cannot exceed the SLO, min(TPS_actual, TPS_SLO)."""
    return min(tps_actual, tps_slo)


def t_task_hours(BS: int, L_in: int, L_out: int, tps_eff: float) -> float:
    """Eq. 2: T_task = BS * (L_in + L_out) / (TPS_effective * 3600), in hours."""
    return BS * (L_in + L_out) / (tps_eff * 3600.0)


def cost_efficiency(tps_eff: float, t_task_h: float, vm_price: float) -> float:
    """Eq. 3: CE = TPS_effective * 3600 / (ceil(T_task) * VM price)."""
    return tps_eff * 3600.0 / (math.ceil(t_task_h) * vm_price)


def offload_ratio(mem_avail: float, mem_kvcache: float) -> float:
    """Section IV-B, case 3: C_off = 1 - Mem_avail / Mem_KVcache."""
    return 1.0 - mem_avail / mem_kvcache


def candidates(instances, mem_model, mem_activation, mem_kvcache, mem_kv_per_layer, p_max):
    """Algorithm 1 (price priority).  ``instances``: iterable of (name, gpu_memory, price).
    Returns [(name, C_off, price)] sorted by ascending price.  Steps in the paper's order:
    price filter; available memory = GPU memory - (model + activation); no offloading if the
    total fits; unsuitable if the weights do not fit or one layer's KV exceeds the available
    memory; otherwise offload the fraction that does not fit."""
    out = []
    mem_total = mem_model + mem_activation + mem_kvcache
    mem_base = mem_model + mem_activation
    for name, gpu_mem, price in instances:
        if price <= p_max:
            avail = gpu_mem - mem_base
            if gpu_mem >= mem_total:
                out.append((name, 0.0, price))
            else:
                if gpu_mem < mem_model or mem_kv_per_layer > avail:
                    continue
                c_off = 1.0 - avail / mem_kvcache
                if mem_kv_per_layer <= avail:
                    out.append((name, c_off, price))
    out.sort(key=lambda r: r[2])
    return out


def select_instance(cands, tps_slo, BS, L_in, L_out):
    """Step 4: drop candidates with TPS < TPS_SLO, rank the rest by Eq. 3, ties go to the
    higher TPS.  ``cands``: iterable of (name, tps, price).  Returns the ranked list of
    (name, tps, price, CE), best first (empty if none meets the SLO)."""
    ranked = []
    for name, tps_, price in cands:
        if tps_ >= tps_slo:
            eff = tps_effective(tps_, tps_slo)
            ce = cost_efficiency(eff, t_task_hours(BS, L_in, L_out, eff), price)
            ranked.append((name, tps_, price, ce))
    ranked.sort(key=lambda r: (-r[3], -r[1]))
    return ranked
