"""Parity of the CUDA path against the fp64 reference, through the C ABI.
Needs a B200; every test here is marked gpu."""
import numpy as np
import pytest
import torch

from oracle import attn as oa
from oracle import kv_model as km
from paper_2504_11816_b200 import binding as B
from paper_2504_11816_b200 import workloads as W

from _harness import TOL, Harness, bits_to_dev, dev_to_bits, values

pytestmark = pytest.mark.gpu


def small(name="s", layers=2, q_heads=4, kv_heads=4, head_dim=128, dtype="f16", batch=5, ctx=(1, 100), steps=3,
          f=0.5, perm=0, seed=11):
    return W.Workload(name, layers, q_heads, kv_heads, head_dim, dtype, batch, ctx[0], ctx[1], steps, 16, f, perm, seed)


# ---------------------------------------------------------------- the Tiny configuration, every row

def test_tiny_config_one_append_one_decode_all_rows():
    w = W.CONFIGS["tiny"]
    with Harness(w) as hz:
        hz.fill()
        table = B.isv_block_table_host(hz.h, w.batch)
        # every other block of the 256-token prompt is host-resident
        for s in range(w.batch):
            assert [bool(e & B.ISV_BLOCK_HOST_BIT) for e in table[s, :16]] == [j % 2 == 1 for j in range(16)]
        res = hz.step()
        err = hz.check_step(res)
        assert err <= TOL
        hz.check_gather()
        # 8 of the 17 blocks of each sequence crossed the host link
        r, o, staged, n_chunks = B.isv_plan_bytes(hz.h, 0, w.batch)
        assert o == 4 * 8 * 16 * w.kv_bytes_per_token and r == 4 * (257 - 128) * w.kv_bytes_per_token


# ---------------------------------------------------------------- offload fraction, permutation, splits, chunks

@pytest.mark.parametrize("f", [0.0, 0.25, 0.5, 0.75, 1.0])
@pytest.mark.parametrize("perm", [0, 5])
@pytest.mark.parametrize("fused", [False, True])
def test_parity_over_offload_fractions_with_ragged_lengths(f, perm, fused):
    lens = [0, 1, 15, 16, 17, 31, 32, 33, 100, 257, 640]
    w = small(batch=len(lens), steps=20, f=f, perm=perm, ctx=(0, 640), q_heads=4, kv_heads=4, head_dim=128)
    with Harness(w, lens=lens) as hz:
        hz.fill()
        hz.check_gather()
        for t in range(w.steps):
            res = hz.step(fused=fused and t % 5 != 4)     # mixing the two call styles must work too
            hz.check_step(res)
            r, o, _, _ = B.isv_plan_bytes(hz.h, 0, w.batch)
            assert (r, o) == km.layer_step_bytes(hz.cur.tolist(), f, 16, w.kv_bytes_per_token)
        hz.check_gather()


@pytest.mark.parametrize("f", [0.25, 1.0])
def test_reading_host_blocks_in_place_gives_the_same_result(f):
    """isv_set_zero_copy: the offloaded blocks are read over the host link by the kernel itself."""
    lens = [0, 17, 100, 257, 640, 33]
    w = small(batch=len(lens), steps=18, f=f, perm=6, ctx=(0, 640), layers=2, q_heads=8, kv_heads=4, head_dim=128)
    with Harness(w, lens=lens) as hz:
        hz.fill()
        B.isv_set_zero_copy(hz.h, True)
        B.isv_set_timing(hz.h, True)
        for t in range(w.steps):
            hz.check_step(hz.step(fused=t % 2 == 0))
            if t == 8:
                B.isv_set_zero_copy(hz.h, False)      # switching back and forth between steps is allowed
            if t == 12:
                B.isv_set_zero_copy(hz.h, True)
        st = B.isv_step_timing(hz.h, -1)
        assert st.bytes_staged == 0 and st.bytes_offloaded > 0 and st.attn_offloaded_ms > 0
        hz.check_gather()


@pytest.mark.parametrize("ctas", [1, 2, 7, 0])
@pytest.mark.parametrize("chunk_blocks", [1, 0])
@pytest.mark.parametrize("q_heads", [8, 32])
def test_result_does_not_depend_on_split_or_chunk_size(ctas, chunk_blocks, q_heads):
    lens = [700, 33, 512, 129]
    outs = []
    w = small(batch=4, steps=2, f=0.5, perm=3, ctx=(1, 700), layers=1, q_heads=q_heads, kv_heads=8, head_dim=64)
    block_bytes = 2 * w.kv_heads * 16 * w.head_dim * 2
    with Harness(w, lens=lens, max_ctas=ctas, chunk_bytes=chunk_blocks * block_bytes) as hz:
        hz.fill()
        for t in range(w.steps):
            res = hz.step()
            hz.check_step(res)
            outs.append(res[0][1])
    # same inputs with the default configuration: results agree within the bound
    with Harness(w, lens=lens) as hz:
        hz.fill()
        for t in range(w.steps):
            res = hz.step()
            assert np.max(np.abs(res[0][1] - outs[t])) <= TOL


# ---------------------------------------------------------------- head grouping, head dim, dtype

# query heads per KV head: 1 runs on the CUDA cores (at head_dim 64 / 80 two adjacent KV heads per visit when the
# head count is even: 8 heads; one per visit otherwise: 5 heads), 2..16 as one tensor-core tile (2, 4, 8, 3, 16,
# 12, 5), 32 as two passes of 16
@pytest.mark.parametrize("q_heads,kv_heads", [(8, 8), (5, 5), (8, 4), (8, 2), (16, 2), (6, 2), (32, 2), (24, 2), (10, 2),
                                              (64, 2)])
@pytest.mark.parametrize("head_dim", [64, 80, 128])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_parity_over_head_grouping_head_dim_and_dtype(q_heads, kv_heads, head_dim, dtype):
    fused = (q_heads + head_dim) % 3 != 0
    lens = [300, 17, 64, 1]
    w = small(batch=4, steps=2, f=0.5, perm=9, ctx=(1, 300), layers=1, q_heads=q_heads, kv_heads=kv_heads,
              head_dim=head_dim, dtype=dtype, seed=21)
    with Harness(w, lens=lens) as hz:
        hz.fill()
        for t in range(w.steps):
            hz.check_step(hz.step(fused=fused))
        hz.check_gather()


@pytest.mark.parametrize("f", [0.0, 0.5])
@pytest.mark.parametrize("fused", [False, True])
def test_layers_sharing_physical_slabs(f, fused):
    """phys_layers < layers (how the benchmark fits 32-40 layers of a large batch): layers l and l + 2 write
    the same slab, the later writer's rows stay; every layer's output is checked against the slab's content
    at the time of its call, and the final slab content is read back bit for bit."""
    lens = [5, 16, 31, 100, 48]
    w = small(batch=len(lens), steps=20, f=f, perm=8, ctx=(1, 100), layers=4, q_heads=4, kv_heads=2, head_dim=64)
    with Harness(w, lens=lens, phys_layers=2) as hz:
        hz.fill()
        for t in range(w.steps):
            hz.check_step(hz.step(fused=fused))
        hz.check_gather(layers=[2, 3])


def test_identical_query_heads_of_a_group_give_identical_outputs():
    w = small(batch=2, steps=1, f=0.5, layers=1, q_heads=8, kv_heads=2, head_dim=128, ctx=(90, 90))
    with Harness(w) as hz:
        hz.fill()
        k, v, q = W.host_step(w, hz.rng)
        q[:] = np.repeat(q[:, ::4], 4, axis=1)           # heads 4g..4g+3 are copies
        kd, vd, qd = (bits_to_dev(x, w.dtype) for x in (k, v, q))
        of = torch.zeros((w.batch, w.q_heads, w.head_dim), device="cuda")
        torch.cuda.synchronize()
        B.isv_kv_append(hz.h, 0, kd, vd, w.batch)
        B.isv_attn_decode(hz.h, 0, qd, None, of, None, None, w.batch)
        B.isv_sync(hz.h)
        o = of.cpu().numpy()
        for g in range(2):
            for i in range(1, 4):
                assert np.array_equal(o[:, 4 * g], o[:, 4 * g + i])


# ---------------------------------------------------------------- special cases of the method

@pytest.mark.parametrize("f", [0.0, 1.0])
@pytest.mark.parametrize("q_heads,head_dim", [(2, 64), (4, 64), (8, 64), (2, 80), (8, 128)])
@pytest.mark.parametrize("fused", [False, True])
def test_context_of_one_token_returns_v_exactly(f, q_heads, head_dim, fused):
    # 1, 2 and 4 query heads per KV head (CUDA-core and tensor-core arithmetic); fused: the token is attended to
    # from the caller's rows, in a visit that carries no tile
    w = small(batch=3, steps=1, f=f, layers=1, q_heads=q_heads, kv_heads=2, head_dim=head_dim, ctx=(0, 0))
    with Harness(w, lens=[0, 0, 0]) as hz:
        hz.fill()
        res = hz.step(fused=fused)                        # the appended token is the whole context
        q, of, o16, _ = res[0]
        kb, vb = zip(*[hz.shadow.gathered(0, s) for s in range(w.batch)])
        for s in range(w.batch):
            for h in range(w.q_heads):
                g = h // (q_heads // 2)
                assert np.array_equal(o16[s, h], vb[s][0, g])
                assert np.array_equal(of[s, h].astype(np.float64), oa.to_f64(values(vb[s][0, g], w.dtype)))


@pytest.mark.parametrize("q_heads", [4, 16])
def test_zero_query_gives_the_mean_of_v(q_heads):
    w = small(batch=2, steps=1, f=0.5, layers=1, q_heads=q_heads, kv_heads=4, head_dim=128, ctx=(333, 333))
    with Harness(w) as hz:
        hz.fill()
        k, v, q = W.host_step(w, hz.rng)
        q[:] = 0
        kd, vd, qd = (bits_to_dev(x, w.dtype) for x in (k, v, q))
        of = torch.zeros((w.batch, w.q_heads, w.head_dim), device="cuda")
        torch.cuda.synchronize()
        B.isv_kv_append(hz.h, 0, kd, vd, w.batch)
        B.isv_attn_decode(hz.h, 0, qd, None, of, None, None, w.batch)
        B.isv_sync(hz.h)
        hz.shadow.append(0, k, v)
        for s in range(w.batch):
            vb = oa.to_f64(values(hz.shadow.gathered(0, s)[1], w.dtype))
            mean = np.repeat(vb.mean(axis=0), q_heads // 4, axis=0)   # head h reads KV head h div (Hq / Hkv)
            assert np.max(np.abs(of[s].cpu().numpy() - mean)) <= 1e-5


def test_empty_sequences_yield_zeros_and_fewer_sequences_can_be_decoded():
    w = small(batch=4, steps=1, f=0.5, layers=1, q_heads=4, kv_heads=4, head_dim=64, ctx=(0, 50))
    with Harness(w, lens=[50, 0, 20, 0]) as hz:
        hz.fill()
        _, _, q = W.host_step(w, hz.rng)
        qd = bits_to_dev(q, w.dtype)
        of = torch.full((w.batch, w.q_heads, w.head_dim), 7.0, device="cuda")
        torch.cuda.synchronize()
        B.isv_attn_decode(hz.h, 0, qd, None, of, None, None, w.batch)
        B.isv_sync(hz.h)
        o = of.cpu().numpy()
        assert np.all(o[1] == 0) and np.all(o[3] == 0)
        ref = hz.reference(0, q, seqs=[0, 2])
        assert np.max(np.abs(o[[0, 2]] - ref)) <= TOL
        # only the first sequence
        of2 = torch.full((w.batch, w.q_heads, w.head_dim), 7.0, device="cuda")
        torch.cuda.synchronize()
        B.isv_attn_decode(hz.h, 0, qd, None, of2, None, None, 1)
        B.isv_sync(hz.h)
        o2 = of2.cpu().numpy()
        assert np.max(np.abs(o2[0] - ref[0])) <= TOL and np.all(o2[1:] == 7.0)


@pytest.mark.parametrize("q_heads", [4, 16])
def test_unused_slots_may_hold_nan_patterns(q_heads):
    # fill every block with NaN bit patterns first, then reset and load short real data into the same blocks
    lens = [5, 21, 40]
    w = small(batch=3, steps=4, f=0.5, layers=1, q_heads=q_heads, kv_heads=4, head_dim=128, ctx=(1, 64))
    with Harness(w, lens=lens) as hz:
        T = 64
        nan_bits = np.full((w.batch, T, w.kv_heads, w.head_dim), 0x7e00, np.uint16)
        nd = bits_to_dev(nan_bits, w.dtype)
        torch.cuda.synchronize()
        B.isv_kv_fill(hz.h, 0, nd, nd, np.full(w.batch, T, np.int32), w.batch, T)
        B.isv_kv_reset(hz.h)
        hz.fill()
        for t in range(w.steps):
            hz.check_step(hz.step())
        hz.check_gather()


def test_explicit_table_and_lengths_pointers_are_honoured():
    w = small(batch=3, steps=1, f=0.0, layers=1, q_heads=4, kv_heads=4, head_dim=64, ctx=(70, 70))
    with Harness(w) as hz:
        hz.fill()
        _, _, q = W.host_step(w, hz.rng)
        qd = bits_to_dev(q, w.dtype)
        info = B.isv_kv_info(hz.h)
        table = torch.from_numpy(B.isv_block_table_host(hz.h, w.batch)).cuda()
        lens = torch.tensor([70, 33, 1], dtype=torch.int32, device="cuda")     # attend to prefixes
        of = torch.zeros((w.batch, w.q_heads, w.head_dim), device="cuda")
        torch.cuda.synchronize()
        B.isv_attn_decode(hz.h, 0, qd, None, of, table, lens, w.batch)
        B.isv_sync(hz.h)
        K, V = [], []
        for s, n in enumerate([70, 33, 1]):
            kb, vb = hz.shadow.gathered(0, s)
            K.append(values(kb[:n], w.dtype))
            V.append(values(vb[:n], w.dtype))
        ref = oa.attn_decode(values(q, w.dtype), K, V)
        assert np.max(np.abs(of.cpu().numpy() - ref)) <= TOL
        assert info.max_blocks_per_seq == table.shape[1]


# ---------------------------------------------------------------- whole-step entry points and timing

@pytest.mark.parametrize("f", [0.0, 0.5])
def test_decode_step_entry_points_match_per_layer_calls(f):
    w = small(batch=4, steps=3, f=f, perm=2, layers=3, q_heads=8, kv_heads=4, head_dim=128, ctx=(40, 200))
    td = W.torch_dtype(w.dtype)
    with Harness(w) as ha, Harness(w) as hb, Harness(w) as hc:
        for hz in (ha, hb, hc):
            hz.fill()
        B.isv_set_timing(hb.h, True)
        for t in range(w.steps):
            res = ha.step()
            ha.check_step(res)
            # replay the same inputs through the whole-step calls
            ks, vs, qs = [], [], []
            for layer in range(w.layers):
                k, v, q = W.host_step(w, hb.rng)
                W.host_step(w, hc.rng)
                ks.append(k); vs.append(v); qs.append(q)
                assert np.array_equal(q, res[layer][0])
            k_all, v_all, q_all = (np.stack(x) for x in (ks, vs, qs))
            kd, vd, qd = (bits_to_dev(x, w.dtype) for x in (k_all, v_all, q_all))
            od = torch.zeros((w.layers, w.batch, w.q_heads, w.head_dim), device="cuda", dtype=td)
            torch.cuda.synchronize()
            B.isv_decode_step(hb.h, qd, kd, vd, od, None, w.batch)
            B.isv_sync(hb.h)
            got = dev_to_bits(od)
            for layer in range(w.layers):      # fused append + attention against the two separate calls
                a = oa.to_f64(values(got[layer], w.dtype))
                b = oa.to_f64(values(res[layer][2], w.dtype))
                assert np.max(np.abs(a - b)) <= TOL
            # host-buffer variant
            kp, vp, qp = (torch.from_numpy(x.view(np.int16)).pin_memory() for x in (k_all, v_all, q_all))
            op = torch.zeros((w.layers, w.batch, w.q_heads, w.head_dim), dtype=torch.int16).pin_memory()
            B.isv_decode_step_host(hc.h, qp, kp, vp, op, w.batch)
            assert np.array_equal(op.numpy().view(np.uint16), got)
            # timing query: byte counters follow the cache model, times are sane
            st = B.isv_step_timing(hb.h, -1)
            res_b, off_b = km.layer_step_bytes(ha.cur.tolist(), f, 16, w.kv_bytes_per_token)
            assert st.bytes_resident == w.layers * res_b and st.bytes_offloaded == w.layers * off_b
            assert st.bytes_appended == w.layers * w.batch * w.kv_bytes_per_token
            assert st.status == 0 and st.total_ms > 0 and st.attn_resident_ms > 0 and st.append_ms == 0
            assert (st.h2d_ms > 0) == (off_b > 0) and (st.n_chunks > 0) == (off_b > 0)
            assert st.total_ms >= st.attn_resident_ms
            one = B.isv_step_timing(hb.h, 1)
            assert one.bytes_resident == res_b and one.total_ms <= st.total_ms + 1e-3


@pytest.mark.parametrize("f", [0.0, 0.5, 1.0])
def test_async_prompt_load_stores_the_offloaded_share_and_reports_it(f):
    """isv_kv_fill_async for all layers back to back (the stores of one layer overlap the packing of the
    next), then the byte counters of the timing query against the cache model and a bit-exact read-back."""
    lens = [1, 16, 33, 400, 129, 64]
    w = small(batch=len(lens), steps=2, f=f, perm=4, ctx=(1, 400), layers=3, q_heads=4, kv_heads=4, head_dim=128)
    block = 16 * w.kv_bytes_per_token
    with Harness(w, lens=lens, chunk_bytes=4 * block) as hz:       # small chunks: many copies, ring reuse
        T = max(lens)
        keep = []
        for layer in range(w.layers):
            k, v = W.host_prompt(w, hz.rng, T)
            kd, vd = bits_to_dev(k, w.dtype), bits_to_dev(v, w.dtype)
            keep.append((kd, vd))                                   # inputs stay alive until the sync
            torch.cuda.synchronize()
            B.isv_kv_fill_async(hz.h, layer, kd, vd, hz.lens, w.batch, T)
            hz.shadow.fill(layer, k, v, lens)
        ft = B.isv_fill_timing(hz.h)                                # of the last layer; synchronises
        res_b, off_b = km.layer_step_bytes(lens, f, 16, w.kv_bytes_per_token)
        assert ft.bytes_stored == off_b and ft.bytes_resident == res_b
        assert (ft.n_copies > 0) == (off_b > 0) and (ft.store_ms > 0) == (off_b > 0)
        assert ft.pack_ms > 0 and ft.total_ms >= ft.pack_ms
        if off_b:
            assert ft.n_copies >= off_b // (4 * block)
        B.isv_sync(hz.h)
        hz.check_gather()
        for t in range(w.steps):
            hz.check_step(hz.step(fused=True))
        hz.check_gather()


def test_link_probe_reports_plausible_rates():
    h2d, d2h = B.isv_link_probe(256 << 20, 3)
    assert 1.0 < h2d < 500.0 and 1.0 < d2h < 500.0


# ---------------------------------------------------------------- launch chains, bad lengths, failure paths

@pytest.mark.parametrize("layers,phys,ctas,f", [(2, 2, 4, 0.0), (3, 3, 8, 0.0), (3, 2, 6, 0.0), (2, 2, 5, 0.5)])
@pytest.mark.parametrize("per_layer", [True, False])
def test_steps_enqueued_back_to_back_on_small_grids(layers, phys, ctas, f, per_layer, monkeypatch):
    """Several whole steps are enqueued without a host wait in between, on grids far below the SM count.
    Launches then follow one another as fast as programmatic dependent launch allows, and a layer's launch of
    step t+1 must still see the lengths and the K/V rows its launch of step t wrote (with two layers the
    writer is only two launches back; with shared slabs likewise).  Every step's output is compared with
    the reference afterwards, and the cache is read back bit for bit."""
    if per_layer:      # one launch per layer even where the step's resident part could be one launch
        monkeypatch.setenv("ISV_LAYERS_PER_LAUNCH", "1")
    steps = 7
    w = small(batch=8, steps=steps, f=f, perm=13, ctx=(1900, 2040), layers=layers, q_heads=4, kv_heads=4,
              head_dim=128, seed=23)
    td = W.torch_dtype(w.dtype)
    with Harness(w, max_ctas=ctas, phys_layers=phys) as hz:
        hz.fill()
        ins = []
        for t in range(steps):
            ks, vs, qs = zip(*[W.host_step(w, hz.rng) for _ in range(layers)])
            ins.append(tuple(np.stack(x) for x in (ks, vs, qs)))
        dev = [tuple(bits_to_dev(x, w.dtype) for x in kvq) for kvq in ins]
        outs = [torch.full((layers, w.batch, w.q_heads, w.head_dim), float("nan"), device="cuda") for _ in range(steps)]
        o16 = [torch.zeros((layers, w.batch, w.q_heads, w.head_dim), device="cuda", dtype=td) for _ in range(steps)]
        torch.cuda.synchronize()
        for t in range(steps):
            kd, vd, qd = dev[t]
            B.isv_decode_step(hz.h, qd, kd, vd, o16[t], outs[t], w.batch)
        assert B.isv_sync(hz.h) == 0
        for t in range(steps):
            k, v, q = ins[t]
            res = []
            for layer in range(layers):
                if phys < layers:
                    hz.shadow.store_at(layer % phys, k[layer], v[layer], hz.cur.tolist())
                    ref = hz.reference(layer, q[layer], lens=hz.cur + 1)
                else:
                    hz.shadow.append(layer, k[layer], v[layer])
                    ref = None
                res.append((q[layer], outs[t][layer].cpu().numpy(), dev_to_bits(o16[t][layer]), ref))
            hz.cur += 1
            hz.check_step(res)
        assert np.array_equal(B.isv_seq_lens_host(hz.h, layers - 1, w.batch), hz.cur)
        hz.check_gather(layers=range(layers - phys, layers))


@pytest.mark.parametrize("q_heads,kv_heads,head_dim,dtype", [(4, 4, 128, "f16"), (8, 2, 128, "bf16"), (6, 6, 80, "f16"),
                                                             (16, 2, 64, "f16")])
@pytest.mark.parametrize("layers,phys,ctas,f", [(5, 5, 0, 0.0), (5, 2, 3, 0.0), (4, 4, 1, 0.0), (5, 5, 0, 0.5), (5, 2, 0, 0.75),
                                                 (4, 4, 2, 1.0)])
def test_whole_step_as_one_launch(q_heads, kv_heads, head_dim, dtype, layers, phys, ctas, f):
    """isv_decode_step runs the resident attention (and the appends) of all layers as one launch whose work list
    spans the layers; with host-resident blocks each layer's staged launches and merge follow it.  Ragged lengths
    (an empty sequence, one token, block boundaries), layers that share slabs, grids of 1, 2, 3 and all CTAs,
    nothing / half / three quarters / everything offloaded; every output row against the reference, lengths and
    cache read back."""
    lens = [0, 1, 15, 16, 17, 100, 257, 330]
    steps = 18                                    # crosses a block boundary for every sequence
    w = small(batch=len(lens), steps=steps + 1, f=f, perm=17, ctx=(0, 330), layers=layers, q_heads=q_heads,
              kv_heads=kv_heads, head_dim=head_dim, dtype=dtype, seed=29)
    td = W.torch_dtype(w.dtype)
    with Harness(w, lens=lens, max_ctas=ctas, phys_layers=phys) as hz:
        hz.fill()
        launches0 = B.isv_kv_info(hz.h).kernel_launches
        updates = 0
        for t in range(steps):
            ks, vs, qs = zip(*[W.host_step(w, hz.rng) for _ in range(layers)])
            k, v, q = (np.stack(x) for x in (ks, vs, qs))
            kd, vd, qd = (bits_to_dev(x, w.dtype) for x in (k, v, q))
            of = torch.full((layers, w.batch, w.q_heads, w.head_dim), float("nan"), device="cuda")
            o16 = torch.zeros((layers, w.batch, w.q_heads, w.head_dim), device="cuda", dtype=td)
            torch.cuda.synchronize()
            updates += int(np.any(hz.cur % 16 == 0))          # a step that opens new blocks also updates the table
            B.isv_decode_step(hz.h, qd, kd, vd, o16, of, w.batch)
            assert B.isv_sync(hz.h) == 0
            res = []
            for layer in range(layers):
                if phys < layers:
                    hz.shadow.store_at(layer % phys, k[layer], v[layer], hz.cur.tolist())
                    ref = hz.reference(layer, q[layer], lens=hz.cur + 1)
                else:
                    hz.shadow.append(layer, k[layer], v[layer])
                    ref = None
                res.append((q[layer], of[layer].cpu().numpy(), dev_to_bits(o16[layer]), ref))
            hz.cur += 1
            hz.check_step(res)
        if f == 0:   # one attention launch per step and group of layers on distinct slabs
            assert B.isv_kv_info(hz.h).kernel_launches - launches0 == steps * -(-layers // phys) + updates
        for layer in range(layers):
            assert np.array_equal(B.isv_seq_lens_host(hz.h, layer, w.batch), hz.cur)
        hz.check_gather(layers=range(layers - phys, layers))
        # the per-layer calls continue from the same state
        hz.check_step(hz.step(fused=True))


@pytest.mark.parametrize("f,phys", [(0.0, 6), (0.0, 2), (0.5, 6), (0.75, 3)])
def test_host_buffer_step_equals_device_buffer_step(f, phys):
    """isv_decode_step_host copies the inputs in groups of layers (1, 4, 1 of six) and runs each group as soon as
    it has arrived, the middle one as fused launches: the same result as isv_decode_step on device buffers up to
    the summation order, and both within the bound of the reference."""
    layers, steps = 6, 5
    lens = [40, 200, 17, 333, 64]
    w = small(batch=len(lens), steps=steps, f=f, perm=19, ctx=(17, 333), layers=layers, q_heads=8, kv_heads=4,
              head_dim=128, seed=37)
    td = W.torch_dtype(w.dtype)
    with Harness(w, lens=lens, phys_layers=phys) as ha, Harness(w, lens=lens, phys_layers=phys) as hb:
        ha.fill()
        hb.fill()
        for t in range(steps):
            ks, vs, qs = zip(*[W.host_step(w, ha.rng) for _ in range(layers)])
            for _ in range(layers):
                W.host_step(w, hb.rng)
            k, v, q = (np.stack(x) for x in (ks, vs, qs))
            kd, vd, qd = (bits_to_dev(x, w.dtype) for x in (k, v, q))
            od = torch.zeros((layers, w.batch, w.q_heads, w.head_dim), device="cuda", dtype=td)
            of = torch.full((layers, w.batch, w.q_heads, w.head_dim), float("nan"), device="cuda")
            torch.cuda.synchronize()
            B.isv_decode_step(ha.h, qd, kd, vd, od, of, w.batch)
            assert B.isv_sync(ha.h) == 0
            kp, vp, qp = (torch.from_numpy(x.view(np.int16)).pin_memory() for x in (k, v, q))
            op = torch.zeros((layers, w.batch, w.q_heads, w.head_dim), dtype=torch.int16).pin_memory()
            B.isv_decode_step_host(hb.h, qp, kp, vp, op, w.batch)
            got_host = op.numpy().view(np.uint16)
            # the two paths cut the work differently (other launch groups), so sums may differ in the last bits
            diff = np.abs(oa.to_f64(values(got_host, w.dtype)) - oa.to_f64(values(dev_to_bits(od), w.dtype)))
            assert float(diff.max()) <= 2.0 ** -10
            res, res_host = [], []
            for layer in range(layers):
                if phys < layers:
                    ha.shadow.store_at(layer % phys, k[layer], v[layer], ha.cur.tolist())
                    ref = ha.reference(layer, q[layer], lens=ha.cur + 1)
                else:
                    ha.shadow.append(layer, k[layer], v[layer])
                    ref = None
                res.append((q[layer], of[layer].cpu().numpy(), dev_to_bits(od[layer]), ref))
                res_host.append((q[layer], None, got_host[layer], ref if ref is not None else ha.reference(layer, q[layer])))
            ha.cur += 1
            ha.check_step(res)
            ha.check_step(res_host)
        assert B.isv_sync(hb.h) == 0
        hb.shadow, hb.cur = ha.shadow, ha.cur            # same inputs went into both caches
        hb.check_gather(layers=range(layers - phys, layers))


@pytest.mark.parametrize("f", [0.0, 0.5])
def test_step_call_over_the_first_sequences_only(f):
    """isv_decode_step with n_seqs below the cache's capacity: only those sequences advance (in every layer), the
    arrays hold n_seqs rows per layer, and the others keep their lengths and content; a later step advances all."""
    lens = [90, 16, 47, 200, 5]
    layers, n = 3, 3
    w = small(batch=len(lens), steps=6, f=f, perm=23, ctx=(5, 200), layers=layers, q_heads=8, kv_heads=8, head_dim=64,
              seed=41)
    with Harness(w, lens=lens) as hz:
        hz.fill()
        for t in range(4):
            m = n if t < 3 else w.batch                      # three partial steps, then a full one
            ks, vs, qs = zip(*[W.host_step(w, hz.rng) for _ in range(layers)])
            k, v, q = (np.stack(x)[:, :m] for x in (ks, vs, qs))
            kd, vd, qd = (bits_to_dev(np.ascontiguousarray(x), w.dtype) for x in (k, v, q))
            of = torch.full((layers, m, w.q_heads, w.head_dim), float("nan"), device="cuda")
            torch.cuda.synchronize()
            B.isv_decode_step(hz.h, qd, kd, vd, None, of, m)
            assert B.isv_sync(hz.h) == 0
            o = of.cpu().numpy()
            for layer in range(layers):
                hz.shadow.append(layer, np.ascontiguousarray(k[layer]), np.ascontiguousarray(v[layer]))
                full_q = np.zeros((w.batch, w.q_heads, w.head_dim), np.uint16)
                full_q[:m] = q[layer]
                ref = hz.reference(layer, full_q, seqs=range(m))
                assert np.max(np.abs(o[layer] - ref)) <= TOL
            hz.cur[:m] += 1
            for layer in range(layers):
                assert np.array_equal(B.isv_seq_lens_host(hz.h, layer, w.batch), hz.cur)
        hz.check_gather()


@pytest.mark.parametrize("f", [0.0, 0.5])
def test_a_full_sequence_refuses_the_step_and_changes_nothing(f):
    """When a sequence has reached max_tokens_per_seq the step is refused with ISV_ECAPACITY before anything is
    enqueued: no layer's lengths move, the cache still reads back bit for bit, and attention over it still works."""
    lens = [30, 47, 48]
    layers = 3
    w = small(batch=len(lens), steps=2, f=f, perm=29, ctx=(30, 48), layers=layers, q_heads=4, kv_heads=4, head_dim=128,
              seed=43)
    with Harness(w, lens=lens) as hz:                    # capacity 48 + 2 = 50 tokens
        hz.fill()
        for t in range(2):
            hz.check_step(hz.step(fused=True))
        assert int(hz.cur.max()) == 50
        ks, vs, qs = zip(*[W.host_step(w, hz.rng) for _ in range(layers)])
        k, v, q = (np.stack(x) for x in (ks, vs, qs))
        kd, vd, qd = (bits_to_dev(x, w.dtype) for x in (k, v, q))
        of = torch.zeros((layers, w.batch, w.q_heads, w.head_dim), device="cuda")
        torch.cuda.synchronize()
        with pytest.raises(B.IsvError) as ei:
            B.isv_decode_step(hz.h, qd, kd, vd, None, of, w.batch)
        assert ei.value.code == B.ISV_ECAPACITY and "full" in ei.value.message
        assert B.isv_sync(hz.h) == 0
        for layer in range(layers):
            assert np.array_equal(B.isv_seq_lens_host(hz.h, layer, w.batch), hz.cur)
        hz.check_gather()
        # the first two sequences still have room: a step over them alone goes through
        of2 = torch.full((layers, 2, w.q_heads, w.head_dim), float("nan"), device="cuda")
        k2, v2, q2 = (np.ascontiguousarray(x[:, :2]) for x in (k, v, q))
        B.isv_decode_step(hz.h, bits_to_dev(q2, w.dtype), bits_to_dev(k2, w.dtype), bits_to_dev(v2, w.dtype), None, of2, 2)
        assert B.isv_sync(hz.h) == 0
        for layer in range(layers):
            hz.shadow.append(layer, k2[layer], v2[layer])
            full_q = np.zeros((w.batch, w.q_heads, w.head_dim), np.uint16)
            full_q[:2] = q2[layer]
            assert np.max(np.abs(of2[layer].cpu().numpy() - hz.reference(layer, full_q, seqs=range(2)))) <= TOL
        hz.cur[:2] += 1
        hz.check_gather()


def test_device_lengths_beyond_the_table_row_are_clamped_and_flagged():
    """Caller-supplied device lengths are not trusted: one that exceeds what a table row covers (or is
    negative) is clamped, the status word says so, and the other sequences are unaffected."""
    w = small(batch=4, steps=1, f=0.0, layers=1, q_heads=4, kv_heads=4, head_dim=64, ctx=(70, 70))
    with Harness(w) as hz:
        hz.fill()
        _, _, q = W.host_step(w, hz.rng)
        qd = bits_to_dev(q, w.dtype)
        rows = B.isv_kv_info(hz.h).max_blocks_per_seq
        lens = torch.tensor([70, 16 * rows + 4000, 33, -5], dtype=torch.int32, device="cuda")
        of = torch.full((w.batch, w.q_heads, w.head_dim), 7.0, device="cuda")
        torch.cuda.synchronize()
        B.isv_attn_decode(hz.h, 0, qd, None, of, None, lens, w.batch)
        with pytest.raises(B.IsvError) as ei:
            B.isv_sync(hz.h)
        assert ei.value.code == B.ISV_EDEVICE_STATUS and "bad length" in ei.value.message
        assert B.isv_sync(hz.h) == 0                      # reported once, then cleared
        o = of.cpu().numpy()
        K, V = [], []
        for s, n in ((0, 70), (2, 33)):
            kb, vb = hz.shadow.gathered(0, s)
            K.append(values(kb[:n], w.dtype))
            V.append(values(vb[:n], w.dtype))
        ref = oa.attn_decode(values(q[[0, 2]], w.dtype), K, V)
        assert np.max(np.abs(o[[0, 2]] - ref)) <= TOL
        assert np.all(o[3] == 0)                          # a negative length counts as empty
        # the handle works normally afterwards
        hz.check_step(hz.step(fused=True))


def test_a_lost_copy_ends_in_a_status_not_a_hang():
    """A K tile whose copy never arrives: the waiting warp gives up after the configured number of polls,
    the kernel returns, the next synchronising call reports ISV_STATUS_WAIT_EXPIRED once, and the handle
    keeps working."""
    w = small(batch=4, steps=4, f=0.0, layers=1, q_heads=4, kv_heads=4, head_dim=128, ctx=(200, 300))
    with Harness(w) as hz:
        hz.fill()
        hz.check_step(hz.step(fused=True))
        B.isv_set_wait_limit(hz.h, 2000)
        B.isv_inject_lost_copy(hz.h, 1)
        k, v, q = W.host_step(w, hz.rng)
        kd, vd, qd = (bits_to_dev(x, w.dtype) for x in (k, v, q))
        of = torch.zeros((w.batch, w.q_heads, w.head_dim), device="cuda")
        torch.cuda.synchronize()
        B.isv_decode_layer(hz.h, 0, qd, kd, vd, None, of, w.batch)
        with pytest.raises(B.IsvError) as ei:
            B.isv_sync(hz.h)
        assert ei.value.code == B.ISV_EDEVICE_STATUS and "wait expired" in ei.value.message
        hz.shadow.append(0, k, v)                         # the append itself is not affected by the lost tile
        hz.cur += 1
        B.isv_set_wait_limit(hz.h, 0)
        assert B.isv_sync(hz.h) == 0
        for _ in range(2):
            hz.check_step(hz.step(fused=True))
        st = B.isv_step_timing(hz.h, -1)
        assert st.status == 0
        hz.check_gather()


def test_host_waits_honour_their_deadline():
    """With a deadline, a host-side wait that is overtaken by it returns ISV_ETIMEOUT and leaves the work
    enqueued; waiting again without the deadline completes normally with correct results."""
    w = small(batch=16, steps=2, f=1.0, perm=3, layers=4, q_heads=8, kv_heads=8, head_dim=128, ctx=(4000, 4096))
    with Harness(w) as hz:
        hz.fill()
        ks, vs, qs = zip(*[W.host_step(w, hz.rng) for _ in range(w.layers)])
        k, v, q = (np.stack(x) for x in (ks, vs, qs))
        kd, vd, qd = (bits_to_dev(x, w.dtype) for x in (k, v, q))
        of = torch.zeros((w.layers, w.batch, w.q_heads, w.head_dim), device="cuda")
        torch.cuda.synchronize()
        B.isv_set_host_timeout(hz.h, 1e-5)
        B.isv_decode_step(hz.h, qd, kd, vd, None, of, w.batch)     # ~0.5 GB over the host link: milliseconds
        with pytest.raises(B.IsvError) as ei:
            B.isv_sync(hz.h)
        assert ei.value.code == B.ISV_ETIMEOUT and "did not finish" in ei.value.message
        B.isv_set_host_timeout(hz.h, 0.0)
        assert B.isv_sync(hz.h) == 0
        res = []
        for layer in range(w.layers):
            hz.shadow.append(layer, k[layer], v[layer])
            res.append((q[layer], of[layer].cpu().numpy(), None, None))
        hz.cur += 1
        hz.check_step(res)
        B.isv_set_host_timeout(hz.h, 30.0)                # a generous deadline changes nothing
        hz.check_step(hz.step(fused=True))


def test_pinned_limit_refuses_the_host_pool_and_leaks_nothing(monkeypatch):
    w = small(batch=4, steps=1, f=0.5, layers=2, q_heads=4, kv_heads=4, head_dim=128, ctx=(500, 500))
    kw = B.desc_from_workload(w)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    monkeypatch.setenv("ISV_PINNED_LIMIT_BYTES", "4096")
    with pytest.raises(B.IsvError) as ei:
        B.isv_kv_alloc(**kw)
    assert ei.value.code == B.ISV_ENOMEM_PINNED and "ISV_PINNED_LIMIT_BYTES" in ei.value.message
    free1, _ = torch.cuda.mem_get_info()
    assert free1 >= free0 - (2 << 20)                     # the HBM pool allocated before the refusal is back
    monkeypatch.setenv("ISV_PINNED_LIMIT_BYTES", str(1 << 40))
    h = B.isv_kv_alloc(**kw)
    B.isv_kv_free(h)


# ---------------------------------------------------------------- full-size launch configurations, sampled rows

def _sample_rows(w, n_rows, seed):
    """(sequence, query head) rows to check: the corners of the batch, the longest and the shortest sequence,
    and seeded random picks; n_rows distinct pairs."""
    lens = W.prompt_lens(w)
    longest, shortest = int(np.argmax(lens)), int(np.argmin(lens))
    rows = [(0, 0), (0, w.q_heads - 1), (w.batch - 1, 0), (w.batch - 1, w.q_heads - 1),
            (longest, 1), (longest, w.q_heads - 2), (shortest, 2), (shortest, w.q_heads - 3)]
    rng = np.random.default_rng(seed)
    while len(set(rows)) < n_rows:
        rows.append((int(rng.integers(w.batch)), int(rng.integers(w.q_heads))))
    return sorted(set(rows))


def _full_size_sampled(w, n_rows, check_steps, gather_seq=None, seed=0):
    """Runs `w` at its full batch / context / head shape through isv_decode_step (the call the benchmark
    times) and compares n_rows sampled (sequence, query head) rows of every layer with the reference, which
    is computed from the generator's own tensors (never from library memory).  The fp32 output is held to
    the 2e-3 bound, the 16-bit output to the same bound plus half a unit in its last place, element by
    element.  Returns (worst fp32 error, rows compared)."""
    G = w.q_heads // w.kv_heads
    sample = _sample_rows(w, n_rows, seed)
    lens = W.prompt_lens(w)
    if gather_seq is None:
        gather_seq = int(np.argmin(lens))
    h = B.isv_kv_alloc(**B.desc_from_workload(w))
    try:
        gen = W.device_generator(w)
        T = int(lens.max())
        keep = sorted({(s, hd // G) for s, hd in sample} | {(gather_seq, g) for g in range(w.kv_heads)})
        Kh, Vh = {}, {}        # (layer, seq, kv head) -> list of [n, d] bit arrays
        for layer in range(w.layers):
            k = W.device_normal(gen, (w.batch, T, w.kv_heads, w.head_dim), w.dtype, w.outlier_prob, w.outlier_scale)
            v = W.device_normal(gen, (w.batch, T, w.kv_heads, w.head_dim), w.dtype, w.outlier_prob, w.outlier_scale)
            torch.cuda.synchronize()
            B.isv_kv_fill(h, layer, k, v, lens, w.batch, T)
            for s, g in keep:
                Kh[(layer, s, g)] = [dev_to_bits(k[s, : int(lens[s]), g])]
                Vh[(layer, s, g)] = [dev_to_bits(v[s, : int(lens[s]), g])]
            del k, v
        worst, compared = 0.0, 0
        half_ulp_rel = 2.0 ** -8 if w.dtype == "bf16" else 2.0 ** -11
        for t in range(w.steps):
            q = W.device_normal(gen, (w.layers, w.batch, w.q_heads, w.head_dim), w.dtype)
            k = W.device_normal(gen, (w.layers, w.batch, w.kv_heads, w.head_dim), w.dtype, w.outlier_prob, w.outlier_scale)
            v = W.device_normal(gen, (w.layers, w.batch, w.kv_heads, w.head_dim), w.dtype, w.outlier_prob, w.outlier_scale)
            out = torch.zeros_like(q)
            of = torch.full(q.shape, float("nan"), device="cuda", dtype=torch.float32)
            torch.cuda.synchronize()
            B.isv_decode_step(h, q, k, v, out, of, w.batch)
            assert B.isv_sync(h) == 0
            for layer in range(w.layers):
                for s, g in keep:
                    Kh[(layer, s, g)].append(dev_to_bits(k[layer, s, g])[None])
                    Vh[(layer, s, g)].append(dev_to_bits(v[layer, s, g])[None])
            if t in check_steps:
                ob, qb = dev_to_bits(out), dev_to_bits(q)
                for layer in range(w.layers):
                    for s, hd in sample:
                        g = hd // G
                        Ks = values(np.concatenate(Kh[(layer, s, g)]), w.dtype)[:, None]
                        Vs = values(np.concatenate(Vh[(layer, s, g)]), w.dtype)[:, None]
                        ref = oa.attn_decode(values(qb[layer, s:s + 1, hd:hd + 1], w.dtype), [Ks], [Vs])[0, 0]
                        got32 = of[layer, s, hd].cpu().numpy().astype(np.float64)
                        err = float(np.max(np.abs(got32 - ref)))
                        assert err <= TOL, (layer, s, hd, err)
                        got16 = oa.to_f64(values(ob[layer, s, hd], w.dtype))
                        excess = float(np.max(np.abs(got16 - ref) - half_ulp_rel * np.abs(ref)))
                        assert excess <= TOL, (layer, s, hd, excess)
                        worst = max(worst, err)
                        compared += 1
        # gather of one sequence is bit-exact (resident, tail and host-resident blocks alike)
        n = int(lens[gather_seq]) + w.steps
        kh = np.zeros((n, w.kv_heads, w.head_dim), np.uint16)
        vh = np.zeros_like(kh)
        last = w.layers - 1
        assert B.isv_kv_gather(h, last, gather_seq, kh, vh) == n
        for g in range(w.kv_heads):
            assert np.array_equal(kh[:, g], np.concatenate(Kh[(last, gather_seq, g)]))
            assert np.array_equal(vh[:, g], np.concatenate(Vh[(last, gather_seq, g)]))
        return worst, compared
    finally:
        B.isv_kv_free(h)


def test_full_size_c2_shape_sampled_rows():
    """Llama-2-7B-shaped decode batch (32 sequences x 32 heads x 128, context 1024, everything resident) in
    the launch configuration the benchmark times; two layers; steps at 1025, 1040 (block just filled) and
    1041 tokens are checked: 3 x 64 (layer, sequence, head) triples."""
    w = W.CONFIGS["c2"].with_(layers=2, steps=17)
    worst, n = _full_size_sampled(w, 32, check_steps=(0, 15, 16), gather_seq=13)
    assert n == 3 * 64 and worst <= TOL


def test_full_size_c3_shape_half_offloaded_permuted_sampled_rows():
    """Llama-2-7B-shaped offline batch: 128 sequences x 32 heads x 128, fp16, context 2048, every other block
    host-resident, both pools permuted; two layers, 64 triples per checked step."""
    w = W.CONFIGS["c3"].with_(layers=2, steps=2)
    worst, n = _full_size_sampled(w, 32, check_steps=(0, 1), gather_seq=77)
    assert n == 2 * 64 and worst <= TOL


def test_full_size_gqa_bf16_three_quarters_offloaded_sampled_rows():
    """Llama-3-8B-shaped batch: 256 sequences, 32 query / 8 KV heads x 128, bf16, context 4096, three quarters
    of the blocks host-resident, permuted block ids; two layers, 64 triples per checked step."""
    w = W.CONFIGS["c4"].with_(layers=2, steps=2)
    worst, n = _full_size_sampled(w, 32, check_steps=(0, 1), gather_seq=100)
    assert n == 2 * 64 and worst <= TOL


@pytest.mark.parametrize("f", [0.0, 0.5, 1.0])
def test_full_size_ragged_outliers_sampled_rows(f):
    """13B-shaped batch: 64 sequences of 512..8192 tokens, 40 heads x 128, K/V with x8 outliers, permuted block
    ids, nothing / half / everything host-resident; two layers, 64 triples per checked step, the longest and
    the shortest sequence among them."""
    w = W.CONFIGS["c5"].with_(layers=2, steps=2, offload_frac=f)
    worst, n = _full_size_sampled(w, 32, check_steps=(0, 1))
    assert n == 2 * 64 and worst <= TOL
