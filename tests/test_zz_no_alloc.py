"""The allocation-free entry point, ``isv_attn_decode_static``.

It serves callers that are not allowed to allocate GPU memory themselves (all
memory already belongs to a framework's allocator, or an allocation would
stall a latency-critical loop): they pass every buffer, and the split kernel's
scratch is a fixed array inside the library.  Here the caller-owned paged pool
is built with torch from the documented layout, the same logical K/V is loaded
into an ordinary handle, and the two entry points must agree within the bound
the other GPU tests use - on two calls in a row, because the shared scratch
keeps the first call's contents.  This file is named to be collected last."""
import numpy as np
import pytest
import torch

from paper_2504_11816_b200 import binding as B
from paper_2504_11816_b200 import workloads as W

from _harness import TOL, Harness, bits_to_dev

pytestmark = pytest.mark.gpu


def _paged_pool(k_bits, v_bits, lens, kv_heads, head_dim, seed):
    """Caller-side paging: pool [blocks][K|V][head][16][d] uint16, table int32 [n_seqs][stride]."""
    n_seqs = len(lens)
    nb = [(int(n) + 15) // 16 for n in lens]
    stride = max(nb) + 2
    total = sum(nb) + 3                                   # a few unused blocks
    ids = np.random.default_rng(seed).permutation(total)
    pool = np.full((total, 2, kv_heads, 16, head_dim), 0x7e00, np.uint16)   # NaN patterns in unused slots
    table = np.full((n_seqs, stride), B.ISV_BLOCK_NONE, np.int32)
    nxt = 0
    for s in range(n_seqs):
        for j in range(nb[s]):
            bid = int(ids[nxt]); nxt += 1
            table[s, j] = bid
            t0, t1 = j * 16, min(int(lens[s]), j * 16 + 16)
            pool[bid, 0, :, : t1 - t0] = k_bits[s, t0:t1].transpose(1, 0, 2)
            pool[bid, 1, :, : t1 - t0] = v_bits[s, t0:t1].transpose(1, 0, 2)
    # the documented chunk order inside a token row: 16-byte chunk c sits at position c ^ (t % 8)
    chunks = pool.reshape(total, 2, kv_heads, 16, head_dim // 8, 8)
    stored = np.empty_like(chunks)
    for t in range(16):
        for c in range(head_dim // 8):
            pos = c ^ (t % 8) if c < head_dim // 8 // 8 * 8 else c   # complete groups of eight chunks only
            stored[:, :, :, t, pos] = chunks[:, :, :, t, c]
    pool = stored.reshape(total, 2, kv_heads, 16, head_dim)
    return pool, table, total, stride, max(nb)


# the last shape (16 query heads per KV head at head_dim 128) needs 133 KB of partials per CTA: a full grid
# does not fit the fixed array, so the call runs on the 62 CTAs whose partials do
@pytest.mark.parametrize("q_heads,kv_heads,head_dim,dtype", [(8, 8, 128, "f16"), (8, 2, 64, "bf16"), (4, 4, 80, "f16"),
                                                             (32, 2, 128, "f16")])
def test_static_entry_matches_handle_entry_on_two_calls_in_a_row(q_heads, kv_heads, head_dim, dtype):
    lens = [300, 1, 16, 513, 77]
    w = W.Workload("na", 1, q_heads, kv_heads, head_dim, dtype, len(lens), 1, 513, 2, 16, 0.0, 0, 31)
    with Harness(w, lens=lens) as hz:
        # same prompt through the ordinary, allocating path
        rng = W.host_rng(w)
        T = max(lens)
        k_bits, v_bits = W.host_prompt(w, rng, T)
        kd, vd = bits_to_dev(k_bits, dtype), bits_to_dev(v_bits, dtype)
        torch.cuda.synchronize()
        B.isv_kv_fill(hz.h, 0, kd, vd, np.array(lens, np.int32), w.batch, T)

        pool, table, n_blocks, stride, max_blocks = _paged_pool(k_bits, v_bits, lens, kv_heads, head_dim, seed=5)
        pool_d = torch.from_numpy(pool.view(np.int16)).cuda()
        table_d = torch.from_numpy(table).cuda()
        lens_d = torch.tensor(lens, dtype=torch.int32, device="cuda")
        status_d = torch.zeros(1, dtype=torch.int32, device="cuda")
        stream = torch.cuda.Stream()
        dt = B.ISV_F16 if dtype == "f16" else B.ISV_BF16

        for call in range(2):                              # second call meets the first call's leftovers
            q_bits = W.normal_bits(rng, (w.batch, q_heads, head_dim), dtype)
            qd = bits_to_dev(q_bits, dtype)
            ref = torch.zeros((w.batch, q_heads, head_dim), device="cuda")
            got = torch.full((w.batch, q_heads, head_dim), float("nan"), device="cuda")
            got16 = torch.zeros((w.batch, q_heads, head_dim), device="cuda", dtype=W.torch_dtype(dtype))
            torch.cuda.synchronize()
            B.isv_attn_decode(hz.h, 0, qd, None, ref, None, None, w.batch)
            B.isv_sync(hz.h)
            B.isv_attn_decode_static(pool_d, n_blocks, table_d, stride, lens_d, w.batch, max_blocks, q_heads,
                                     kv_heads, head_dim, 16, dt, 2 if call else 0, qd, got16, got, status_d,
                                     stream.cuda_stream)
            stream.synchronize()
            torch.cuda.synchronize()
            assert int(status_d.item()) == 0
            g, r = got.cpu().numpy(), ref.cpu().numpy()
            assert np.all(np.isfinite(g))
            assert np.max(np.abs(g - r)) <= TOL, (call, float(np.max(np.abs(g - r))))
            assert np.max(np.abs(got16.float().cpu().numpy() - r)) <= TOL + 4e-3 * np.max(np.abs(r))
            # and against the fp64 reference of the handle's record
            hz.shadow.fill(0, k_bits, v_bits, lens)
            assert np.max(np.abs(g - hz.reference(0, q_bits))) <= TOL


def test_static_entry_refuses_shapes_beyond_its_fixed_scratch():
    one = torch.zeros(64, dtype=torch.int32, device="cuda")
    with pytest.raises(B.IsvError) as ei:
        # 4096 sequences x 1024 head groups: the arrival counters alone exceed the fixed array
        B.isv_attn_decode_static(one, 1, one, 64, one, 4096, 64, 1024, 1024, 128, 16, B.ISV_F16, 0, one, one, None,
                                 None, 0)
    assert ei.value.code == B.ISV_ECAPACITY
    assert "fixed array" in ei.value.message
    with pytest.raises(B.IsvError) as ei:
        B.isv_attn_decode_static(one, 1, one, 4, one, 1, 4, 8, 8, 96, 16, B.ISV_F16, 0, one, one, None, None, 0)
    assert ei.value.code == B.ISV_EINVAL
