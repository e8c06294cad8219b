"""CPU-only checks of the C-ABI library: it loads, exports what the header
declares, and its host bookkeeping (residency rule, block tables, byte
accounting, errors) agrees with the reference cache model.  Uses plan-only
handles, which make no CUDA call; no attention is computed here."""
import os
import re

import numpy as np
import pytest

from oracle import kv_model as km
from paper_2504_11816_b200 import binding as B
from paper_2504_11816_b200 import build as isv_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    isv_build.build()


def _alloc(**kw):
    d = dict(layers=2, q_heads=8, kv_heads=4, head_dim=64, block_tokens=16, dtype=B.ISV_F16,
             offload_frac=0.5, max_seqs=6, max_tokens_per_seq=200, plan_only=1)
    d.update(kw)
    return B.isv_kv_alloc(**d)


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "isv.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(isv_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(B.EXPORTS)
    lib = B.lib()
    for name in declared:
        assert hasattr(lib, name), name


def test_bad_descriptions_are_rejected_with_a_message():
    for kw in (dict(head_dim=96), dict(q_heads=6, kv_heads=4), dict(offload_frac=1.5), dict(block_tokens=8),
               dict(max_seqs=0), dict(layers=0), dict(phys_layers=3), dict(dtype=7), dict(ring_depth=1), dict(max_ctas=-1)):
        with pytest.raises(B.IsvError) as ei:
            _alloc(**kw)
        assert ei.value.code == B.ISV_EINVAL and ei.value.message


def test_plan_only_handle_refuses_compute():
    h = _alloc()
    try:
        with pytest.raises(B.IsvError) as ei:
            B.isv_attn_decode(h, 0, 16, 16, None, None, None, 1)
        assert ei.value.code == B.ISV_ENODEVICE
        with pytest.raises(B.IsvError) as ei:
            B.isv_kv_gather(h, 0, 0, np.zeros(4, np.uint16), np.zeros(4, np.uint16))
        assert ei.value.code == B.ISV_ENODEVICE
        assert B.isv_block_table_dev(h)[0] is None
    finally:
        B.isv_kv_free(h)


@pytest.mark.parametrize("f", [0.0, 0.25, 0.5, 0.6, 0.75, 1.0])
@pytest.mark.parametrize("seed", [0, 7])
def test_block_table_follows_the_residency_rule_and_pools_stay_consistent(f, seed):
    n_seqs, max_tok = 5, 330
    h = _alloc(offload_frac=f, max_seqs=n_seqs, max_tokens_per_seq=max_tok, perm_seed=seed)
    try:
        info = B.isv_kv_info(h)
        lens = np.array([1, 16, 17, 200, 330], dtype=np.int32)
        B.isv_kv_fill(h, 0, None, None, lens, n_seqs, 330)
        B.isv_kv_fill(h, 1, None, None, lens, n_seqs, 330)
        table = B.isv_block_table_host(h, n_seqs)
        assert table.shape == (n_seqs, info.max_blocks_per_seq)
        hbm_ids, host_ids = [], []
        for s, n in enumerate(lens):
            nb = km.n_blocks(int(n), 16)
            for j in range(table.shape[1]):
                e = int(table[s, j])
                if j >= nb:
                    assert e == B.ISV_BLOCK_NONE
                    continue
                assert e != B.ISV_BLOCK_NONE
                assert bool(e & B.ISV_BLOCK_HOST_BIT) == km.is_host_block(j, f)
                (host_ids if e & B.ISV_BLOCK_HOST_BIT else hbm_ids).append(e & (B.ISV_BLOCK_HOST_BIT - 1))
        assert len(set(hbm_ids)) == len(hbm_ids) and all(0 <= i < info.hbm_blocks for i in hbm_ids)
        # host ids are unique and compact
        assert sorted(host_ids) == list(range(len(host_ids)))
        info = B.isv_kv_info(h)
        assert info.hbm_blocks_used == len(hbm_ids) and info.host_blocks_used == len(host_ids)
        if seed != 0 and len(hbm_ids) > 8:
            assert hbm_ids != sorted(hbm_ids)          # ids were handed out in permuted order
        if seed == 0:
            assert hbm_ids == list(range(len(hbm_ids)))
    finally:
        B.isv_kv_free(h)


@pytest.mark.parametrize("f", [0.0, 0.25, 0.5, 0.75, 1.0])
def test_byte_accounting_matches_the_cache_model_while_sequences_grow(f):
    n_seqs = 4
    kv_heads, d = 4, 64
    h = _alloc(offload_frac=f, max_seqs=n_seqs, max_tokens_per_seq=120, kv_heads=kv_heads, head_dim=d,
               chunk_bytes=4 * 2 * kv_heads * 16 * d * 2, perm_seed=3)
    kappa = km.kv_bytes_per_token(kv_heads, d, 2)
    info = B.isv_kv_info(h)
    assert info.kv_bytes_per_token == kappa and info.block_bytes == 16 * kappa
    try:
        lens = np.array([0, 5, 31, 64], dtype=np.int32)
        B.isv_kv_fill(h, 0, None, None, lens, n_seqs, 64)
        cur = lens.copy()
        for step in range(40):
            res, off, staged, n_chunks = B.isv_plan_bytes(h, 0, n_seqs)
            assert (res, off) == km.layer_step_bytes(cur.tolist(), f, 16, kappa), (step, cur)
            assert staged >= off and staged % info.block_bytes == 0
            assert (n_chunks == 0) == (off == 0)
            # fewer sequences: only those are counted
            res2, off2, _, _ = B.isv_plan_bytes(h, 0, 2)
            assert (res2, off2) == km.layer_step_bytes(cur[:2].tolist(), f, 16, kappa)
            B.isv_kv_append(h, 0, None, None, n_seqs)
            cur += 1
            assert np.array_equal(B.isv_seq_lens_host(h, 0, n_seqs), cur)
        # the other layer was never touched
        assert np.array_equal(B.isv_seq_lens_host(h, 1, n_seqs), np.zeros(n_seqs, np.int32))
    finally:
        B.isv_kv_free(h)


def test_capacity_errors_and_reset():
    h = _alloc(max_seqs=2, max_tokens_per_seq=20)
    try:
        with pytest.raises(B.IsvError) as ei:
            B.isv_kv_fill(h, 0, None, None, np.array([21, 1], np.int32), 2, 32)
        assert ei.value.code == B.ISV_ECAPACITY
        with pytest.raises(B.IsvError) as ei:
            B.isv_kv_fill(h, 0, None, None, np.array([5, 1], np.int32), 2, 4)     # lens > T
        assert ei.value.code == B.ISV_EINVAL
        B.isv_kv_fill(h, 0, None, None, np.array([19, 3], np.int32), 2, 32)
        B.isv_kv_append(h, 0, None, None, 2)
        with pytest.raises(B.IsvError) as ei:
            B.isv_kv_append(h, 0, None, None, 2)
        assert ei.value.code == B.ISV_ECAPACITY
        # the failed call changed nothing
        assert B.isv_seq_lens_host(h, 0, 2).tolist() == [20, 4]
        with pytest.raises(B.IsvError):
            B.isv_kv_append(h, 5, None, None, 1)                                   # bad layer
        B.isv_kv_reset(h)
        assert B.isv_seq_lens_host(h, 0, 2).tolist() == [0, 0]
        assert np.all(B.isv_block_table_host(h, 2) == B.ISV_BLOCK_NONE)
        assert B.isv_kv_info(h).hbm_blocks_used == 0
    finally:
        B.isv_kv_free(h)


def test_pool_sizes_follow_the_kv_size_formula():
    from oracle import paper_model as pm
    # all resident, capacity = BS * tokens: pool bytes equal Table II's KV size for block-aligned tokens
    h = _alloc(layers=3, offload_frac=0.0, max_seqs=8, max_tokens_per_seq=160, kv_heads=4, head_dim=64)
    try:
        info = B.isv_kv_info(h)
        assert info.host_blocks == 0
        assert info.hbm_pool_bytes == pm.kv_cache_bytes(8, 160, 4 * 64, 2, 3)
    finally:
        B.isv_kv_free(h)
    h = _alloc(layers=3, offload_frac=0.5, max_seqs=8, max_tokens_per_seq=160, kv_heads=4, head_dim=64)
    try:
        info = B.isv_kv_info(h)
        assert info.host_pool_bytes == pm.kv_cache_bytes(8, 160, 4 * 64, 2, 3) // 2
        assert info.host_blocks == info.hbm_blocks == 8 * 5
    finally:
        B.isv_kv_free(h)
    # the paper's main model, OPT-2.7B (h1 = 2560 = 32 heads x 80, 32 layers), at its offline workload:
    # batch 32, 1024 + 128 tokens, everything resident
    h = _alloc(layers=32, offload_frac=0.0, max_seqs=32, max_tokens_per_seq=1152, q_heads=32, kv_heads=32,
               head_dim=80)
    try:
        info = B.isv_kv_info(h)
        assert info.kv_bytes_per_token == 2 * 2560 * 2 and info.block_bytes == 16 * 2 * 2560 * 2
        assert info.hbm_pool_bytes == pm.kv_cache_bytes(32, 1152, 2560, 2, 32)
    finally:
        B.isv_kv_free(h)


def test_host_pool_beyond_the_pinned_limit_is_refused(monkeypatch):
    """ISV_PINNED_LIMIT_BYTES stands in for a locked-memory limit of the system: a description whose
    host pool exceeds it is refused with ISV_ENOMEM_PINNED and a message, on plan-only handles too."""
    need = B.isv_kv_info(h0 := _alloc()).host_pool_bytes
    B.isv_kv_free(h0)
    assert need > 0
    monkeypatch.setenv("ISV_PINNED_LIMIT_BYTES", str(need - 1))
    with pytest.raises(B.IsvError) as ei:
        _alloc()
    assert ei.value.code == B.ISV_ENOMEM_PINNED
    assert str(need) in ei.value.message and "ISV_PINNED_LIMIT_BYTES" in ei.value.message
    monkeypatch.setenv("ISV_PINNED_LIMIT_BYTES", str(need))
    B.isv_kv_free(_alloc())
    B.isv_kv_free(_alloc(offload_frac=0.0))          # nothing offloaded: no host pool, never refused


def test_failure_handling_knobs_validate_their_arguments():
    h = _alloc()
    try:
        B.isv_set_host_timeout(h, 2.5)
        B.isv_set_host_timeout(h, 0.0)
        with pytest.raises(B.IsvError) as ei:
            B.isv_set_host_timeout(h, -1.0)
        assert ei.value.code == B.ISV_EINVAL
        B.isv_set_wait_limit(h, 1000)
        B.isv_inject_lost_copy(h, 0)
        with pytest.raises(B.IsvError) as ei:
            B.isv_inject_lost_copy(h, -1)
        assert ei.value.code == B.ISV_EINVAL
        assert B.isv_sync(h) == 0                    # a plan-only handle has nothing to wait for
    finally:
        B.isv_kv_free(h)
