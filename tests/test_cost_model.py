"""The package's evaluator of the paper's model against the reference restatement of the same
formulas (oracle/paper_model.py), and the reference against what the paper prints.  CPU only."""
import math
import os

import numpy as np
import pytest

from oracle import paper_model as pm
from paper_2504_11816_b200 import cost_model as cm

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
OPT27 = cm.ModelShape(h1=2560, h2=10240, n_layers=32, prec_bytes=2)
T4 = cm.Machine(flops=8.24e12, bw_h2d=6e9, bw_d2h=6e9)


# ---------------------------------------------------------------- reference vs the paper

def test_reference_cost_formulas_reproduce_the_printed_slo200_prices():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "table6_slo200_prices.txt"))
            if ln.strip() and not ln.startswith("#")]
    for name, price, tps_avg, total in rows:
        eff = pm.tps_effective(float(tps_avg), 200.0)
        hours = pm.t_task_hours(1000, 1024, 128, eff)
        assert hours == pytest.approx(1.6)
        assert math.ceil(hours) * float(price) == pytest.approx(float(total), abs=5e-4)
        assert pm.cost_efficiency(eff, hours, float(price)) == pytest.approx(200 * 3600 / float(total), rel=1e-3)


def test_reference_algorithm_1_three_cases_and_price_order():
    GB = 2 ** 30
    inst = [("big", 48 * GB, 2.7), ("mid", 24 * GB, 1.2), ("small", 16 * GB, 0.7), ("tiny", 4 * GB, 0.3),
            ("dear", 80 * GB, 9.0), ("thin", 7 * GB, 0.5)]
    model, act, kv, kv_layer = 5 * GB, 1 * GB, 30 * GB, 1.5 * GB
    got = pm.candidates(inst, model, act, kv, kv_layer, p_max=3.0)
    # dear: over budget; tiny: weights do not fit; thin: 7 - 6 = 1 GB < one layer's KV
    assert [g[0] for g in got] == ["small", "mid", "big"]
    assert got[2][1] == 0.0                                        # 48 >= 36: no offloading
    assert got[1][1] == pytest.approx(1 - 18 / 30)                 # 24 - 6 = 18 GB available
    assert got[0][1] == pytest.approx(1 - 10 / 30)
    assert pm.offload_ratio(18 * GB, 30 * GB) == pytest.approx(0.4)


def test_reference_final_selection_filters_by_slo_and_breaks_ties_by_tps():
    c = [("a", 169.0, 0.71), ("b", 415.0, 1.167), ("c", 1506.0, 2.699), ("d", 500.0, 1.167)]
    r = pm.select_instance(c, 200.0, 1000, 1024, 128)
    assert [x[0] for x in r] == ["d", "b", "c"]                   # a misses the SLO; b and d tie on CE
    assert r[0][3] == pytest.approx(200 * 3600 / (2 * 1.167))
    assert pm.select_instance(c, 5000.0, 1000, 1024, 128) == []


# ---------------------------------------------------------------- package evaluator vs reference

@pytest.mark.parametrize("BS,L_in,L_out,c_off", [(1, 128, 512, 0.0), (32, 1024, 128, 0.6), (64, 512, 128, 1.0)])
def test_time_terms_match_the_reference(BS, L_in, L_out, c_off):
    lin, att = cm.t_compute_d(OPT27, T4, BS, L_in, L_out)
    assert lin == pytest.approx(pm.linear_flops_decode(BS, 2560, 10240) / T4.flops, rel=1e-14)
    assert att == pytest.approx(pm.attn_flops_decode(BS, L_in + L_out / 2, 2560) / T4.flops, rel=1e-14)
    td = cm.t_trans_d(OPT27, T4, BS, L_in, L_out, c_off)
    assert td == pytest.approx(pm.t_trans_d_bytes(c_off, L_in, L_out, 2560, 2, BS) / T4.bw_h2d, rel=1e-14)
    tp = cm.t_trans_p(OPT27, T4, BS, L_in, c_off)
    assert tp == pytest.approx(pm.t_trans_p_bytes(c_off, L_in, 2560, 2, BS) / T4.bw_d2h, rel=1e-14)
    a, b = -0.185, 24.35e-3
    dec = cm.t_dec(OPT27, T4, BS, L_in, L_out, c_off, a, b)
    assert dec == pytest.approx(pm.t_dec(lin + att, td, a, b), rel=1e-13)
    plin, patt = cm.t_compute_p(OPT27, T4, BS, L_in)
    pre = cm.t_pre(OPT27, T4, BS, L_in, c_off, a, b)
    assert pre == pytest.approx(pm.t_pre(plin + patt, tp, a, b), rel=1e-13)
    assert cm.t_task(OPT27, T4, BS, L_in, L_out, c_off, a, b) == pytest.approx(pm.t_task(pre, dec, 32, L_out), rel=1e-13)
    assert cm.tps(BS, L_in, L_out, 3.0) == pm.tps(BS, L_in, L_out, 3.0)
    assert cm.kv_cache_bytes(OPT27, BS, L_in + L_out) == pm.kv_cache_bytes(BS, L_in + L_out, 2560, 2, 32)


def test_selection_logic_matches_the_reference_on_random_catalogues():
    rng = np.random.default_rng(3)
    GB = 2 ** 30
    for trial in range(200):
        inst = [(f"i{k}", float(rng.integers(4, 96)) * GB, float(rng.uniform(0.2, 5.0))) for k in range(8)]
        model, act = float(rng.uniform(2, 14)) * GB, float(rng.uniform(0.1, 2)) * GB
        kv = float(rng.uniform(1, 60)) * GB
        kv_layer = kv / 32
        p_max = float(rng.uniform(0.5, 5.0))
        want = pm.candidates(inst, model, act, kv, kv_layer, p_max)
        got = cm.candidate_instances(inst, model, act, kv, kv_layer, p_max)
        assert [(g[0], g[2]) for g in got] == [(w[0], w[2]) for w in want]
        assert np.allclose([g[1] for g in got], [w[1] for w in want], rtol=1e-15, atol=0)
        cands = [(n, float(rng.uniform(50, 2000)), p) for n, _, p in inst]
        slo = float(rng.uniform(50, 1500))
        assert cm.select_instance(cands, slo, 1000, 1024, 128) == pytest.approx(pm.select_instance(cands, slo, 1000, 1024, 128))
        for n, t, p in cands:
            ce, billed, eff = cm.cost_efficiency(t, slo, 1000, 1024, 128, p)
            assert eff == pm.tps_effective(t, slo)
            assert ce == pytest.approx(pm.cost_efficiency(eff, pm.t_task_hours(1000, 1024, 128, eff), p), rel=1e-15)


def test_ctcf_fit_is_the_least_squares_line():
    rng = np.random.default_rng(5)
    x = np.array([1, 2, 4, 8, 16, 32, 64], dtype=float) * 1e-3
    y = 0.8 * x + 2e-3 + rng.normal(0, 1e-5, size=x.size)
    a, b, err = cm.fit_ctcf(x.tolist(), y.tolist())
    pa, pb = np.polyfit(x, y, 1)
    assert a == pytest.approx(pa, rel=1e-9) and b == pytest.approx(pb, rel=1e-9)
    assert err == pytest.approx(float(np.mean(np.abs(pa * x + pb - y) / y)) * 100, rel=1e-6)
    # exact line: zero error; the paper's printed T4 coefficients evaluate as Eq. 7 says
    a, b, err = cm.fit_ctcf([1.0, 2.0, 3.0], [24.165, 23.98, 23.795])
    assert a == pytest.approx(-0.185) and b == pytest.approx(24.35) and err < 1e-9
    assert cm.ctcf(10.0, a, b) == pytest.approx(pm.ctcf(10.0, -0.185, 24.35))
    with pytest.raises(ValueError):
        cm.fit_ctcf([1.0], [1.0])
