"""Pins for the linear-layer reference.  CPU only."""
import numpy as np
import torch

from oracle import linear as ol
from oracle import paper_model as pm


def test_matches_a_triple_loop_on_small_inputs():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((3, 5))
    w = rng.standard_normal((4, 5))
    y = ol.linear(x, w)
    for m in range(3):
        for n in range(4):
            acc = 0.0
            for k in range(5):
                acc += float(x[m, k]) * float(w[n, k])
            assert abs(y[m, n] - acc) <= 1e-14
    assert y.shape == (3, 4)


def test_identity_selection_and_linearity():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((6, 8))
    assert np.array_equal(ol.linear(x, np.eye(8)), x)                 # identity weights return the input
    w = rng.standard_normal((5, 8))
    e = np.zeros((1, 8)); e[0, 3] = 1.0
    assert np.array_equal(ol.linear(e, w)[0], w[:, 3])                # a unit token selects a weight column
    assert np.allclose(ol.linear(2 * x, w), 2 * ol.linear(x, w), rtol=1e-15)
    assert not np.allclose(ol.linear(x, w), ol.linear(x, w[::-1]))    # weight rows are not interchangeable


def test_matches_torch_float64_linear_on_half_inputs():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((7, 64)).astype(np.float16)
    w = (rng.standard_normal((32, 64)) / 8).astype(np.float16)
    ref = torch.nn.functional.linear(torch.from_numpy(x).double(), torch.from_numpy(w).double()).numpy()
    assert np.max(np.abs(ol.linear(x, w) - ref)) <= 1e-13
    xb = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16)
    wb = torch.from_numpy(w.astype(np.float32)).to(torch.bfloat16)
    refb = torch.nn.functional.linear(xb.double(), wb.double()).numpy()
    assert np.max(np.abs(ol.linear(xb, wb) - refb)) <= 1e-13


def test_flop_count_is_the_papers_linear_term():
    assert ol.linear_flops_per_layer(32, 2560, 10240) == pm.linear_flops_decode(32, 2560, 10240)
