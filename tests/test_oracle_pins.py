"""Pins for the fp64 attention oracle: each test fixes it to something other
than itself (an independently written brute force, closed forms, invariants,
library routines used as black boxes).  CPU only."""
import math

import numpy as np
import pytest

from oracle import attn as oa
from oracle import brute


def _rand(rng, *shape):
    return rng.standard_normal(shape)


# ---------------------------------------------------------------- brute force

@pytest.mark.parametrize("n,d,Hq,Hkv", [(1, 1, 1, 1), (2, 1, 1, 1), (3, 2, 2, 2), (5, 4, 4, 2),
                                        (8, 4, 6, 2), (7, 3, 4, 1)])
def test_matches_brute_force_on_tiny_inputs(n, d, Hq, Hkv):
    rng = np.random.default_rng(100 + n * 10 + d)
    n_seqs = 3
    q = _rand(rng, n_seqs, Hq, d)
    lens = [n, max(1, n - 1), n + 2]
    K = [_rand(rng, L, Hkv, d) for L in lens]
    V = [_rand(rng, L, Hkv, d) for L in lens]
    got = oa.attn_decode(q, K, V)
    want = np.array(brute.attn_batch(q.tolist(), [k.tolist() for k in K], [v.tolist() for v in V], Hq, Hkv))
    assert np.max(np.abs(got - want)) <= 1e-13


def test_hand_computed_example():
    # d = 1, q = ln 3: scores 0 and ln 3, weights 1/4 and 3/4, V = 0 and 4 -> 3
    out = oa.attn_decode(np.array([[[math.log(3.0)]]]), [np.array([[[0.0]], [[1.0]]])],
                         [np.array([[[0.0]], [[4.0]]])])
    assert abs(out[0, 0, 0] - 3.0) <= 1e-14
    # d = 4 halves the exponent: q.k = 2 ln 3 -> score ln 3 again
    q = np.array([[[2 * math.log(3.0), 0.0, 0.0, 0.0]]])
    K = [np.array([[[0.0, 5, 5, 5]], [[1.0, -7, 2, 9]]])]
    V = [np.array([[[0.0, 8, 0, -4]], [[4.0, 0, 4, 4]]])]
    out = oa.attn_decode(q, K, V)
    assert np.allclose(out[0, 0], [3.0, 2.0, 3.0, 2.0], atol=1e-13, rtol=0)


# ---------------------------------------------------------------- special cases

def test_context_length_one_returns_v_exactly():
    rng = np.random.default_rng(1)
    q = _rand(rng, 4, 6, 8)
    K = [_rand(rng, 1, 3, 8) for _ in range(4)]
    V = [_rand(rng, 1, 3, 8) for _ in range(4)]
    out = oa.attn_decode(q, K, V)
    for s in range(4):
        for h in range(6):
            assert np.array_equal(out[s, h], V[s][0, h // 2])


def test_weight_rows_sum_to_one_and_output_is_convex_combination():
    rng = np.random.default_rng(2)
    q = _rand(rng, 3, 4, 16) * 3
    lens = [17, 1, 300]
    K = [_rand(rng, L, 2, 16) for L in lens]
    V = [_rand(rng, L, 2, 16) for L in lens]
    out, w = oa.attn_decode(q, K, V, return_weights=True)
    for s, L in enumerate(lens):
        assert w[s].shape == (4, L)
        assert np.all(w[s] >= 0)
        assert np.max(np.abs(w[s].sum(axis=1) - 1.0)) <= 1e-12
        for h in range(4):
            g = h // 2
            assert np.all(out[s, h] <= V[s][:, g].max(axis=0) + 1e-12)
            assert np.all(out[s, h] >= V[s][:, g].min(axis=0) - 1e-12)
            # the weights reproduce the output
            assert np.max(np.abs(w[s][h] @ V[s][:, g] - out[s, h])) <= 1e-12


def test_zero_query_gives_mean_of_v():
    rng = np.random.default_rng(3)
    K = [_rand(rng, 37, 2, 8)]
    V = [_rand(rng, 37, 2, 8)]
    out = oa.attn_decode(np.zeros((1, 2, 8)), K, V)
    assert np.max(np.abs(out[0] - V[0].mean(axis=0))) <= 1e-13


def test_equal_keys_give_mean_of_v_and_constant_v_is_returned():
    rng = np.random.default_rng(4)
    q = _rand(rng, 1, 2, 8)
    krow = _rand(rng, 1, 2, 8)
    K = [np.repeat(krow, 21, axis=0)]
    V = [_rand(rng, 21, 2, 8)]
    out = oa.attn_decode(q, K, V)
    assert np.max(np.abs(out[0] - V[0].mean(axis=0))) <= 1e-13
    c = _rand(rng, 1, 2, 8)
    out = oa.attn_decode(q, [_rand(rng, 21, 2, 8)], [np.repeat(c, 21, axis=0)])
    assert np.max(np.abs(out[0] - c[0])) <= 1e-13


def test_dominant_key_selects_its_value_and_large_scores_do_not_overflow():
    d = 4
    K = np.zeros((10, 1, d))
    K[6, 0, 0] = 1.0
    V = np.arange(10 * d, dtype=np.float64).reshape(10, 1, d)
    # score of token 6 exceeds all others by 60; then by 2000 (exp would overflow unshifted)
    for gap in (60.0, 2000.0):
        q = np.array([[[gap * math.sqrt(d), 0, 0, 0]]])
        out = oa.attn_decode(q, [K], [V])
        assert np.max(np.abs(out[0, 0] - V[6, 0])) <= 40 * 9 * math.exp(-60.0)
        assert np.all(np.isfinite(out))
    # a negative query must select against that key: weight of token 6 vanishes
    q = np.array([[[-60.0 * math.sqrt(d), 0, 0, 0]]])
    out = oa.attn_decode(q, [K], [V])
    assert np.max(np.abs(out[0, 0] - np.delete(V[:, 0], 6, axis=0).mean(axis=0))) <= 1e-12


# ---------------------------------------------------------------- invariances

def test_shift_of_all_keys_and_joint_permutation_leave_output_unchanged():
    rng = np.random.default_rng(5)
    q = _rand(rng, 2, 4, 8)
    K = [_rand(rng, 50, 2, 8), _rand(rng, 9, 2, 8)]
    V = [_rand(rng, 50, 2, 8), _rand(rng, 9, 2, 8)]
    base = oa.attn_decode(q, K, V)
    shift = _rand(rng, 1, 2, 8)
    shifted = oa.attn_decode(q, [k + shift for k in K], V)
    assert np.max(np.abs(shifted - base)) <= 1e-12
    perms = [rng.permutation(k.shape[0]) for k in K]
    permuted = oa.attn_decode(q, [k[p] for k, p in zip(K, perms)], [v[p] for v, p in zip(V, perms)])
    assert np.max(np.abs(permuted - base)) <= 1e-13
    # permuting K alone must change the result (K and V are not interchangeable)
    wrong = oa.attn_decode(q, [k[p] for k, p in zip(K, perms)], V)
    assert np.max(np.abs(wrong - base)) > 1e-3


def test_identical_query_heads_in_a_group_match_the_single_head_result():
    rng = np.random.default_rng(6)
    Hkv, G, d = 3, 4, 8
    qg = _rand(rng, 2, Hkv, d)
    q = np.repeat(qg, G, axis=1)             # heads g*G .. g*G+G-1 are copies of qg[:, g]
    K = [_rand(rng, 33, Hkv, d), _rand(rng, 5, Hkv, d)]
    V = [_rand(rng, 33, Hkv, d), _rand(rng, 5, Hkv, d)]
    gqa = oa.attn_decode(q, K, V)
    mha = oa.attn_decode(qg, K, V)
    for h in range(Hkv * G):
        assert np.array_equal(gqa[:, h], mha[:, h // G])


# ---------------------------------------------------------------- library routines as black boxes

def test_matches_scipy_softmax_and_matmul():
    from scipy.special import softmax
    rng = np.random.default_rng(7)
    Hq, Hkv, d = 8, 2, 32
    q = _rand(rng, 2, Hq, d)
    lens = [129, 40]
    K = [_rand(rng, L, Hkv, d) for L in lens]
    V = [_rand(rng, L, Hkv, d) for L in lens]
    out = oa.attn_decode(q, K, V)
    for s in range(2):
        for h in range(Hq):
            g = h // (Hq // Hkv)
            p = softmax(K[s][:, g] @ q[s, h] / math.sqrt(d))
            assert np.max(np.abs(p @ V[s][:, g] - out[s, h])) <= 1e-13


def test_matches_torch_sdpa_float64_with_grouped_heads():
    import torch
    import torch.nn.functional as F
    rng = np.random.default_rng(8)
    Hq, Hkv, d, L = 8, 2, 16, 77
    q = _rand(rng, 3, Hq, d)
    K = [_rand(rng, L, Hkv, d) for _ in range(3)]
    V = [_rand(rng, L, Hkv, d) for _ in range(3)]
    out = oa.attn_decode(q, K, V)
    tq = torch.from_numpy(q)[:, :, None, :]                              # [B, Hq, 1, d]
    tk = torch.from_numpy(np.stack(K)).permute(0, 2, 1, 3)               # [B, Hkv, L, d]
    tv = torch.from_numpy(np.stack(V)).permute(0, 2, 1, 3)
    ref = F.scaled_dot_product_attention(tq, tk, tv, enable_gqa=True)[:, :, 0, :].numpy()
    assert np.max(np.abs(ref - out)) <= 1e-12


# ---------------------------------------------------------------- split / merge rule

def test_merging_partials_of_any_split_equals_the_unsplit_result():
    rng = np.random.default_rng(9)
    d, n = 16, 200
    q = _rand(rng, d) * 2
    K = _rand(rng, n, d)
    V = _rand(rng, n, d)
    whole = oa.attn_decode(q[None, None], [K[:, None]], [V[:, None]])[0, 0]
    for cut in (1, 16, 100, 199):
        parts = [oa.attn_partial(q, K[:cut], V[:cut]), oa.attn_partial(q, K[cut:], V[cut:])]
        assert np.max(np.abs(oa.merge_partials(parts) - whole)) <= 1e-13
    # interleaved (non-contiguous) subsets and a seven-way split
    idx = [np.arange(r, n, 7) for r in range(7)]
    parts = [oa.attn_partial(q, K[i], V[i]) for i in idx]
    assert np.max(np.abs(oa.merge_partials(parts) - whole)) <= 1e-13
    # a single partial normalises to the plain result
    assert np.max(np.abs(oa.merge_partials([oa.attn_partial(q, K, V)]) - whole)) <= 1e-13


# ---------------------------------------------------------------- input handling

def test_half_and_bfloat16_inputs_are_widened_exactly():
    import torch
    bits = np.arange(0, 65536, dtype=np.uint32).astype(np.uint16)
    h = bits.view(np.float16)
    finite = np.isfinite(h)
    w = oa.to_f64(h)
    assert np.array_equal(w[finite].astype(np.float16).view(np.uint16), bits[finite])
    # bf16: the upper half of a float32
    f32 = (bits.astype(np.uint32) << 16).view(np.float32)
    tb = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)
    wb = oa.to_f64(tb)
    fin = np.isfinite(f32)
    assert np.array_equal(wb[fin], f32[fin].astype(np.float64))


def test_bad_arguments_are_rejected():
    with pytest.raises(ValueError):
        oa.attn_decode(np.zeros((1, 3, 4)), [np.zeros((2, 2, 4))], [np.zeros((2, 2, 4))])  # 3 % 2 != 0
