"""The calibration procedure of the paper's time model (Section IV-E, Eq. 7) run on this library: what the
paper asserts about it is asserted here at a small shape.  Needs a B200."""
import numpy as np
import pytest

from paper_2504_11816_b200 import binding as B
from paper_2504_11816_b200 import calibrate as C
from paper_2504_11816_b200 import cost_model as cm
from paper_2504_11816_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_compute_time_is_linear_in_the_model_time_and_transfer_time_follows_the_link_rate():
    """(1) Over batch sizes the measured attention time per layer is a straight line in the model's
    T_compute^d attention term (4 * BS * ctx * h1 / FLOPS): the least-squares fit CTCF(T) = alpha * T + beta
    reproduces every point within a few per cent (the paper reports 2-4 % on its GPUs).  (2) With half of
    the cache offloaded, the measured host-link time per layer equals the offloaded bytes divided by the
    link rate probed in the same process, within 5 % (the paper: 1 % for decode)."""
    flops = 2.25e15
    base = W.Workload("cal", 4, 32, 32, 128, "f16", 1, 2048, 2048, 16, 16, 0.0, 0, 7)
    h1 = base.kv_heads * base.head_dim
    steps, warmup = 6, 3
    model, meas = [], []
    for bs in (1, 2, 4, 8, 16):
        m = C.measure(base.with_(batch=bs), steps, warmup)
        ctx_mean = base.ctx_max + warmup + (steps + 1) / 2.0
        model.append(4.0 * bs * ctx_mean * h1 / flops)
        meas.append(m["attn"])
        assert m["bytes_res"] == pytest.approx(bs * ctx_mean * base.kv_bytes_per_token, rel=1e-6)
    alpha, beta, err = cm.fit_ctcf(model, meas)
    assert alpha > 0 and err < 8.0, (alpha, beta, err, meas)
    worst = max(abs(cm.ctcf(t, alpha, beta) - y) / y for t, y in zip(model, meas))
    assert worst < 0.15, (worst, meas)
    assert all(b > a for a, b in zip(meas, meas[1:]))          # more sequences never take less time

    h2d, _ = B.isv_link_probe(1 << 28, 5)
    off = C.measure(base.with_(batch=32, offload_frac=0.5), 4, 3)
    assert off["bytes_off"] > 0
    t_model = off["bytes_off"] / (h2d * 1e9)                   # first term of T_trans^d at the measured rate
    assert abs(off["h2d"] / t_model - 1.0) < 0.05, (off["h2d"], t_model)
    assert off["total"] >= off["h2d"] * 0.98                   # the step cannot end before its transfer
