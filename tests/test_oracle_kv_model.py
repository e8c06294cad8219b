"""Pins for the cache model (residency rule, byte accounting, shadow cache) and
for the paper's formulas.  CPU only."""
import os

import numpy as np
import pytest

from oracle import kv_model as km
from oracle import paper_model as pm

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- residency rule

def test_half_offload_puts_every_other_block_on_the_host():
    host = [j for j in range(16) if km.is_host_block(j, 0.5)]
    assert host == [1, 3, 5, 7, 9, 11, 13, 15]


def test_three_quarters_offload_keeps_one_block_of_four_resident():
    flags = [km.is_host_block(j, 0.75) for j in range(12)]
    assert flags == [False, True, True, True] * 3


@pytest.mark.parametrize("f", [0.0, 0.25, 0.5, 0.6, 0.75, 1.0, 1.0 / 3.0])
def test_every_prefix_holds_floor_j_f_host_blocks(f):
    import math
    cnt = 0
    for j in range(2000):
        assert cnt == math.floor(j * km.f32(f))
        cnt += km.is_host_block(j, f)
    if f == 0.0:
        assert cnt == 0
    if f == 1.0:
        assert cnt == 2000


# ---------------------------------------------------------------- byte accounting against the paper

@pytest.mark.parametrize("C_off,L_in", [(0.0, 1024), (0.25, 512), (0.5, 256), (0.75, 4096), (1.0, 64)])
def test_offloaded_bytes_reduce_to_first_term_of_t_trans_d(C_off, L_in):
    # first decode step after a prompt of L_in tokens: ctx = L_in + 1, the new token's
    # block is in GPU memory, all L_in prompt tokens sit in complete blocks
    BS, Hkv, d, prec, BT = 8, 4, 128, 2, 16
    h1 = Hkv * d
    kappa = km.kv_bytes_per_token(Hkv, d, prec)
    res, off = km.layer_step_bytes([L_in + 1] * BS, C_off, BT, kappa)
    assert off == pm.offloaded_kv_bytes(C_off, L_in, h1, prec, BS)
    # resident + offloaded = the per-layer KV size of Table II for ctx tokens
    assert res + off == pm.kv_cache_bytes(BS, L_in + 1, h1, prec, 1)
    # and the printed numerator exceeds the first term by its L_out and "+1" terms only
    L_out = 128
    extra = pm.t_trans_d_bytes(C_off, L_in, L_out, h1, prec, BS) - pm.offloaded_kv_bytes(C_off, L_in, h1, prec, BS)
    assert extra == (C_off * 2 + L_out) * h1 * prec * BS


def test_offloaded_bytes_stay_within_one_block_per_sequence_of_the_paper_form():
    rng = np.random.default_rng(0)
    Hkv, d, prec, BT = 8, 128, 2, 16
    kappa = km.kv_bytes_per_token(Hkv, d, prec)
    lens = rng.integers(1, 3000, size=50).tolist()
    for f in (0.25, 0.5, 0.6, 0.75, 1.0):
        res, off = km.layer_step_bytes(lens, f, BT, kappa)
        assert res + off == sum(lens) * kappa
        paper = sum(pm.offloaded_kv_bytes(km.f32(f), n, Hkv * d, prec, 1) for n in lens)
        assert abs(off - paper) <= len(lens) * 2 * BT * kappa
    assert km.layer_step_bytes(lens, 0.0, BT, kappa) == (sum(lens) * kappa, 0)


def test_newest_block_is_never_counted_as_offloaded():
    kappa = km.kv_bytes_per_token(1, 64, 2)
    # 32 tokens = blocks 0 and 1; block 1 is host-flagged at f = 0.5 but is the newest
    assert km.layer_step_bytes([32], 0.5, 16, kappa) == (32 * kappa, 0)
    # one more token makes block 1 complete and no longer newest
    assert km.layer_step_bytes([33], 0.5, 16, kappa) == (17 * kappa, 16 * kappa)
    # everything offloaded: all but the newest block
    assert km.layer_step_bytes([40], 1.0, 16, kappa) == (8 * kappa, 32 * kappa)


# ---------------------------------------------------------------- the paper's formulas

def test_kv_cache_size_example_from_the_paper():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "kv_cache_size_example.txt"))
            if ln.strip() and not ln.startswith("#")]
    for bs, gib in rows:
        got = pm.kv_cache_bytes(int(bs), 544, 2560, 2, 32) / 2 ** 30
        assert abs(got - float(gib)) < 1e-3, (bs, got)
    # same numbers under the other reading (1088 tokens, no factor 2)
    assert pm.kv_cache_bytes(2, 1088, 2560, 2, 32) == 2 * (2 * 1088 * 2560 * 2 * 32)


def test_time_formulas_follow_their_equations():
    # Eq. 6 is a sum, Eq. 5 a max, Eq. 7 a line, Eq. 4 weights decode by L_out - 1
    assert pm.t_dec(2.0, 3.0) == 5.0
    assert pm.t_dec(2.0, 3.0, alpha=0.5, beta=1.0) == 0.5 * 2.0 + 1.0 + 3.0
    assert pm.t_pre(2.0, 3.0) == 3.0 and pm.t_pre(4.0, 3.0) == 4.0
    assert pm.ctcf(10.0, -0.185, 24.35) == pytest.approx(22.5)
    assert pm.t_task(1.5, 0.25, 32, 128) == 1.5 * 32 + 0.25 * 32 * 127
    assert pm.tps(32, 1024, 128, 10.0) == 32 * 1152 / 10.0
    # attention flops: 2*ctx*h1 for q.K^T plus 2*ctx*h1 for p.V per sequence
    assert pm.attn_flops_decode(3, 100, 64) == 3 * (2 * 100 * 64 + 2 * 100 * 64)
    assert pm.linear_flops_decode(2, 8, 32) == 2 * (8 * 64 + 4 * 8 * 32)
    assert pm.t_trans_p_bytes(0.5, 1023, 2560, 2, 4) == 0.5 * 2 * 1024 * 2560 * 2 * 4
    assert pm.t_trans_d_bytes(0.0, 1024, 128, 2560, 2, 32) == 128 * 2560 * 2 * 32


# ---------------------------------------------------------------- shadow cache

def test_shadow_cache_keeps_rows_in_arrival_order():
    rng = np.random.default_rng(1)
    sc = km.ShadowCache(2, 2, 4)
    k = rng.integers(0, 65536, size=(3, 5, 2, 4)).astype(np.uint16)
    v = rng.integers(0, 65536, size=(3, 5, 2, 4)).astype(np.uint16)
    sc.fill(1, k, v, [5, 2, 0])
    k1 = rng.integers(0, 65536, size=(3, 2, 4)).astype(np.uint16)
    v1 = rng.integers(0, 65536, size=(3, 2, 4)).astype(np.uint16)
    sc.append(1, k1, v1)
    assert [sc.length(1, s) for s in range(3)] == [6, 3, 1]
    gk, gv = sc.gathered(1, 1)
    assert np.array_equal(gk, np.concatenate([k[1, :2], k1[1][None]]))
    assert np.array_equal(gv, np.concatenate([v[1, :2], v1[1][None]]))
    gk, gv = sc.gathered(1, 2)
    assert np.array_equal(gk, k1[2][None]) and np.array_equal(gv, v1[2][None])
    assert sc.gathered(0, 0)[0].shape == (0, 2, 4)


def test_shadow_cache_positional_store_overwrites_or_extends():
    sc = km.ShadowCache(1, 1, 2)
    a = np.array([[[1, 2]], [[3, 4]]], dtype=np.uint16)        # two sequences, one token each
    sc.store_at(0, a, a + 10, [0, 0])                          # extend empty sequences
    b = np.array([[[5, 6]], [[7, 8]]], dtype=np.uint16)
    sc.store_at(0, b, b + 10, [0, 1])                          # overwrite seq 0's token, extend seq 1
    k0, v0 = sc.gathered(0, 0)
    k1, v1 = sc.gathered(0, 1)
    assert k0.tolist() == [[[5, 6]]] and v0.tolist() == [[[15, 16]]]
    assert k1.tolist() == [[[3, 4]], [[7, 8]]] and v1.tolist() == [[[13, 14]], [[17, 18]]]
    with pytest.raises(AssertionError):
        sc.store_at(0, b, b, [3, 0])
