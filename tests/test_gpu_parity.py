"""CUDA path vs the CPU oracle, element by element, through the C ABI (run on a B200)."""
import math

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import pool as op
from oracle.attention import attend_request, attend_rows
from oracle.layer import attention_layer_step
from oracle.lora import lora_project
from paper_2505_03756_b200 import synth

from _util import REDUCED, assert_close, oracle_adapters, oracle_context, replay_trace


@pytest.fixture(scope="module")
def H():
    assert torch.cuda.is_available(), "these tests need a GPU"
    from paper_2505_03756_b200 import binding, harness
    return harness


def _session(H, wl, **kw):
    s = H.Session(wl, **kw)
    s.load_adapters()
    s.build_batch()
    return s


# ------------------------------------------------------------------ a1: allocator, tables, adapter bytes
@pytest.mark.parametrize("name", ["tiny", "decode13b", "swapstress"])
def test_allocator_tables_and_adapter_bytes_bit_exact(H, name):
    wl = synth.make_workload(name, **REDUCED[name])
    s = _session(H, wl)
    try:
        model = replay_trace(s)                                   # every id handed out matches the model
        from paper_2505_03756_b200 import binding as fl
        assert np.array_equal(fl.fl_pool_snapshot(s.pool), np.array(model.free_list(), dtype=np.uint32))
        assert np.array_equal(fl.fl_pool_snapshot(s.pool, host=True), np.array(model.free_list(host=True), dtype=np.uint32))
        st = s.status()
        assert st["device_flags"] == 0 and st["blocks_used"] + st["blocks_free"] == wl.pool_blocks
        assert st["lora_blocks"] == sum(s.n_table.values())
        mats = s.mats
        hslab = fl.host_slab(s.pool, s.block_bytes, max(1, s.n_host_blocks))
        for a in s.adapter_ids:
            A = [synth.bf16_bits(wl.adapter(a, n)[0]) for n, _, _ in wl.shape.mats]
            B = [synth.bf16_bits(wl.adapter(a, n)[1]) for n, _, _ in wl.shape.mats]
            rank = int(wl.ranks[a])
            n_tab, where = op.lora_layout(s.block_bytes, rank, mats)
            assert n_tab == s.n_table[a]
            model.pack_lora([int(b) for b in s.lora_host_tables[a]], rank, mats, A, B, host=True)
            model.swap_in([int(b) for b in s.lora_tables[a]], [int(b) for b in s.lora_host_tables[a]])
            got = fl.device_block_bytes(s.pool, s.block_bytes, s.lora_tables[a])
            used = np.zeros((n_tab, s.block_bytes), dtype=bool)      # bytes the layout defines
            for (m, side), (base, first, rpb, width) in where.items():
                for r in range(rank):
                    g = first + r
                    used[base + g // rpb, (g % rpb) * 2 * width:(g % rpb + 1) * 2 * width] = True
            for k, (db, hb) in enumerate(zip(s.lora_tables[a], s.lora_host_tables[a])):
                want = model.block(int(db))
                assert np.array_equal(got[k][used[k]], want[used[k]]), (a, k)
                assert np.array_equal(hslab[int(hb)][used[k]], want[used[k]]), (a, k)
    finally:
        s.close()


def test_allocator_error_paths(H):
    from paper_2505_03756_b200 import binding as fl
    pool = fl.fl_pool_create(4096, 6, 2, 0)
    try:
        assert fl.fl_block_alloc(pool, 3).tolist() == [0, 1, 2]
        fl.fl_block_free(pool, [0, 2])
        assert fl.fl_block_alloc(pool, 3).tolist() == [2, 0, 3]
        with pytest.raises(fl.FlError) as e:
            fl.fl_block_alloc(pool, 3)
        assert e.value.code == fl.FL_ENOMEM
        assert fl.fl_pool_snapshot(pool).tolist() == [5, 4]
        for bad in ([1, 1], [9], [4]):
            with pytest.raises(fl.FlError) as e:
                fl.fl_block_free(pool, bad)
            assert e.value.code == fl.FL_EBADID
        assert fl.fl_pool_snapshot(pool).tolist() == [5, 4]
        with pytest.raises(fl.FlError) as e:
            fl.fl_swap_out(pool, [4], [0], torch.cuda.current_stream())   # neither block is allocated
        assert e.value.code == fl.FL_EBADID
        with pytest.raises(fl.FlError):
            fl.fl_pool_create(1000, 4, 0, 0)                              # block size not a multiple of 512
        with pytest.raises(fl.FlError):
            fl.fl_lora_register(pool, 0, 8, [(64, 64)], [5])             # block 5 is not allocated
        with pytest.raises(fl.FlError):
            fl.fl_lora_register(pool, 0, 8, [(64, 60)], [1])             # width not a multiple of 8
    finally:
        fl.fl_pool_destroy(pool)


# ------------------------------------------------------------------ a2/a3: LoRA projection
@pytest.mark.parametrize("name,shrink", [(n, 0) for n in REDUCED] + [("gqa34b", 1), ("swapstress", 1)])
def test_sgmv_parity(H, name, shrink):
    """shrink = 1: the mma.sync shrink also where long segments above rank 16 would take the tcgen05 one."""
    from paper_2505_03756_b200 import binding as fl
    wl = synth.make_workload(name, **REDUCED[name])
    s = _session(H, wl)
    try:
        fl.fl_pool_set_option(s.pool, fl.FL_OPT_SGMV_SHRINK, shrink)
        seg, ids = wl.segments()
        groups = [["q", "k", "v"], ["o"]] + ([["up"], ["down"]] if wl.shape.inter else [])
        for grp in groups:
            x = wl.x(grp[0])
            tx = H.f32_to_dev(x, s.dev)
            for zero_base in (False, True):
                yb = {m: (np.zeros_like(wl.y_base(m)) if zero_base else wl.y_base(m)) for m in grp}
                ty = [H.f32_to_dev(yb[m], s.dev) for m in grp]
                s.sgmv(ty, tx, grp)
                torch.cuda.synchronize()
                for m, t in zip(grp, ty):
                    want = lora_project(yb[m], x, seg, ids, oracle_adapters(wl, m), wl.scale)
                    assert_close(H.dev_to_f32(t), want, f"{name}/{m}/zero_base={zero_base}")
        assert s.status()["device_flags"] == 0
    finally:
        s.close()


def test_sgmv_identities_and_edges(H):
    wl = synth.make_workload("prefill7b", n_req=5, len_range=(20, 150), n_adapters=4)
    s = _session(H, wl)
    try:
        from paper_2505_03756_b200 import binding as fl
        seg, ids = wl.segments()
        x, yb = wl.x("q"), wl.y_base("q")
        tx = H.f32_to_dev(x, s.dev)
        base_bits = synth.bf16_bits(yb)
        # scale 0 and "no adapter" segments leave y bit for bit
        ty = H.f32_to_dev(yb, s.dev)
        s.sgmv([ty], tx, ["q"], scale=0.0)
        assert np.array_equal(ty.view(torch.int16).cpu().numpy().view(np.uint16), base_bits)
        none = torch.full_like(s.t_seg_lora, -1)
        ws = s.workspace("sgmv", fl.fl_lora_sgmv_workspace(wl.n_tokens, 1))
        fl.fl_lora_sgmv(s.pool, ty, tx, 0, s.t_seg_indptr, none, s.n_seg, wl.n_tokens, 2.0, ws)
        assert np.array_equal(ty.view(torch.int16).cpu().numpy().view(np.uint16), base_bits)
        # only some segments carry an adapter
        mixed = ids.copy()
        mixed[::2] = -1
        fl.fl_lora_sgmv(s.pool, ty, tx, 0, s.t_seg_indptr, torch.from_numpy(mixed).to(s.dev), s.n_seg, wl.n_tokens,
                        2.0, ws)
        want = lora_project(yb, x, seg, mixed, oracle_adapters(wl, "q"), 2.0)
        got = H.dev_to_f32(ty)
        assert_close(got, want, "mixed")
        for k, lid in enumerate(mixed):
            if lid < 0:
                assert np.array_equal(got[seg[k]:seg[k + 1]], yb[seg[k]:seg[k + 1]])
        # empty batch, and an unknown adapter id only raises the sticky flag
        fl.fl_lora_sgmv(s.pool, ty, tx, 0, s.t_seg_indptr, s.t_seg_lora, 0, 0, 2.0, ws)
        assert s.status()["device_flags"] == 0
        bad = torch.full_like(s.t_seg_lora, 3000)
        fl.fl_lora_sgmv(s.pool, ty, tx, 0, s.t_seg_indptr, bad, s.n_seg, wl.n_tokens, 2.0, ws)
        assert s.status(clear=True)["device_flags"] & 4
        assert s.status()["device_flags"] == 0
    finally:
        s.close()


def test_sgmv_zero_B_is_base_and_odd_rank(H):
    shape = synth.LayerShape(512, 4, 4)
    for rank in (5, 24):
        wl = synth.make_workload("tiny", n_req=5, len_range=(16, 9), n_adapters=3, shape=shape, rank=rank)
        s = H.Session(wl)
        try:
            from paper_2505_03756_b200 import binding as fl
            # adapter 2 gets B = 0: packed by hand through the C ABI
            for a in s.adapter_ids:
                A = [synth.bf16_bits(wl.adapter(a, n)[0]) for n, _, _ in wl.shape.mats]
                B = [synth.bf16_bits(wl.adapter(a, n)[1] * (0.0 if a == 2 else 1.0)) for n, _, _ in wl.shape.mats]
                ht = s.alloc(s.n_table[a], host=True)
                fl.fl_lora_pack_host(s.pool, rank, s.mats, A, B, ht)
                dt = s.alloc(s.n_table[a])
                fl.fl_swap_in(s.pool, dt, ht, torch.cuda.current_stream())
                fl.fl_lora_register(s.pool, a, rank, s.mats, dt)
            s.build_batch()
            seg, ids = wl.segments()
            x, yb = wl.x("o"), wl.y_base("o")
            ty = H.f32_to_dev(yb, s.dev)
            s.sgmv([ty], H.f32_to_dev(x, s.dev), ["o"])
            ad = oracle_adapters(wl, "o")
            ad[2] = (ad[2][0], 0 * ad[2][1])
            got = H.dev_to_f32(ty)
            assert_close(got, lora_project(yb, x, seg, ids, ad, wl.scale), f"rank {rank}")
            rows = np.concatenate([np.arange(seg[k], seg[k + 1]) for k, l in enumerate(ids) if l == 2])
            assert np.array_equal(got[rows], yb[rows])
        finally:
            s.close()


# ------------------------------------------------------------------ a4: KV store
@pytest.mark.parametrize("name", ["tiny", "prefill7b", "decode13b", "gqa34b"])
def test_kv_append_bit_exact(H, name):
    wl = synth.make_workload(name, **REDUCED[name])
    s = H.Session(wl, adapters=[])
    try:
        from paper_2505_03756_b200 import binding as fl
        s.build_batch()
        s.fill_prefix_kv()
        k_new, v_new = wl.kv_new()
        s.kv_append(H.f32_to_dev(k_new, s.dev), H.f32_to_dev(v_new, s.dev))
        model = replay_trace(s)
        sh = wl.shape
        tables = [[int(b) for b in t] for t in s.kv_tables]
        for i in range(wl.n_req):
            kp, vp = wl.kv_prefix(i)
            model.kv_append(synth.bf16_bits(kp), synth.bf16_bits(vp), [0, len(kp)], [tables[i]], [0], sh.n_kv_heads, 128)
        model.kv_append(synth.bf16_bits(k_new), synth.bf16_bits(v_new), wl.req_indptr, tables, wl.prefix_lens,
                        sh.n_kv_heads, 128)
        bt = sh.block_tokens
        for i in range(wl.n_req):
            ctx = int(wl.prefix_lens[i] + wl.new_lens[i])
            got = fl.device_block_bytes(s.pool, s.block_bytes, tables[i]).view(np.uint16)
            got = got.reshape(len(tables[i]), 2, sh.n_kv_heads, bt, 128)
            for e, b in enumerate(tables[i]):
                valid = min(bt, ctx - e * bt)
                want = model.block(b).view(np.uint16).reshape(2, sh.n_kv_heads, bt, 128)
                assert np.array_equal(got[e][:, :, :valid], want[:, :, :valid]), (i, e)
        assert s.status()["device_flags"] == 0
    finally:
        s.close()


# ------------------------------------------------------------------ a5/a6: attention
def _attention_case(H, wl, sm_scale=None, prefill_kernel=0):
    from paper_2505_03756_b200 import binding as fl
    s = H.Session(wl, adapters=[])
    try:
        fl.fl_pool_set_option(s.pool, fl.FL_OPT_PREFILL_KERNEL, prefill_kernel)
        s.build_batch()
        s.fill_prefix_kv()
        k_new, v_new = wl.kv_new()
        q = wl.q()
        s.kv_append(H.f32_to_dev(k_new, s.dev), H.f32_to_dev(v_new, s.dev))
        out = torch.zeros(q.shape, dtype=torch.bfloat16, device=s.dev)
        s.attention(out, H.f32_to_dev(q, s.dev), sm_scale=sm_scale)
        torch.cuda.synchronize()
        got = H.dev_to_f32(out)
        scale = 1.0 / math.sqrt(128) if sm_scale is None else sm_scale
        for i in range(wl.n_req):
            lo, hi = int(wl.req_indptr[i]), int(wl.req_indptr[i + 1])
            k, v = oracle_context(wl, i, k_new, v_new)
            want = attend_request(q[lo:hi], k, v, int(wl.prefix_lens[i]), scale)
            assert_close(got[lo:hi], want, f"{wl.name} request {i}")
        assert s.status()["device_flags"] == 0
        return got
    finally:
        s.close()


@pytest.mark.parametrize("kernel", [0, 1])
@pytest.mark.parametrize("name", list(REDUCED))
def test_attention_parity(H, name, kernel):
    _attention_case(H, synth.make_workload(name, **REDUCED[name]), prefill_kernel=kernel)


def test_attention_sharp_softmax_rescales_accumulator(H):
    # large logits that keep growing along the keys force the running maximum up tile after tile
    wl = synth.make_workload("prefill7b", n_req=2, len_range=(300, 700))
    for kernel in (0, 1):
        _attention_case(H, wl, sm_scale=1.5, prefill_kernel=kernel)


@pytest.mark.parametrize("kernel", [0, 1])
def test_attention_edges(H, kernel):
    sh = synth.LayerShape(512, 4, 4)
    # no prefix, one token, ragged tails, a request with no new token, long decode context (several chunks)
    wl = synth.make_workload("tiny", n_req=6, len_range=(0, 0), n_adapters=1, shape=sh)
    wl.prefix_lens[:] = [0, 0, 17, 63, 1500, 40]
    wl.new_lens[:] = [1, 70, 1, 65, 1, 0]
    wl.pool_blocks = 256
    _attention_case(H, wl, prefill_kernel=kernel)
    # grouped heads: decode rows = 2 tokens x 8 heads, and a sharp softmax
    sh = synth.LayerShape(1024, 16, 2)
    wl = synth.make_workload("tiny", n_req=3, len_range=(0, 0), n_adapters=1, shape=sh)
    wl.prefix_lens[:] = [300, 5, 0]
    wl.new_lens[:] = [2, 1, 130]
    _attention_case(H, wl, sm_scale=0.5, prefill_kernel=kernel)


def test_attention_prefix_reuse_equals_recompute_and_block_choice(H):
    wl = synth.make_workload("prefill7b", n_req=3, len_range=(100, 260))
    a = _attention_case(H, wl)
    wl2 = synth.make_workload("prefill7b", n_req=3, len_range=(100, 260))
    wl2.seed = wl.seed
    s = H.Session(wl2, adapters=[], scramble=False)          # same data in other physical blocks
    try:
        s.build_batch()
        s.fill_prefix_kv()
        k_new, v_new = wl2.kv_new()
        s.kv_append(H.f32_to_dev(k_new, s.dev), H.f32_to_dev(v_new, s.dev))
        out = torch.zeros(wl2.q().shape, dtype=torch.bfloat16, device=s.dev)
        s.attention(out, H.f32_to_dev(wl2.q(), s.dev))
        assert np.array_equal(H.dev_to_f32(out), a)           # block ids do not change a single bit
    finally:
        s.close()


# ------------------------------------------------------------------ a7: swap
def test_swap_roundtrip_bit_exact(H):
    from paper_2505_03756_b200 import binding as fl
    wl = synth.make_workload("swapstress", **REDUCED["swapstress"])
    s = H.Session(wl, adapters=[], extra_host_blocks=40)
    try:
        dev = s.alloc(48)
        host = s.alloc(40, host=True)
        n = s.block_bytes
        rs = synth.Stream(9, "blocks")
        data = (rs.bits(48 * n // 8)).view(np.uint8).reshape(48, n)
        for k, b in enumerate(dev):
            fl.fl_block_write(s.pool, b, data[k])
        side = torch.cuda.Stream()
        out_d, out_h = dev[:20], host[20:][::-1]
        fl.fl_swap_out(s.pool, out_d, out_h, side)
        ev = torch.cuda.Event()
        fl.fl_swap_record(s.pool, ev, side)
        assert fl.fl_swap_wait(s.pool, ev, 20000) == fl.FL_OK
        hs = fl.host_slab(s.pool, n, s.n_host_blocks)
        for d, h in zip(range(20), out_h):
            assert np.array_equal(hs[int(h)], data[d])
        fl.fl_swap_in(s.pool, dev[28:48], out_h, side)             # back into different device blocks
        fl.fl_swap_record(s.pool, ev, side)
        assert fl.fl_swap_wait(s.pool, ev, 20000) == fl.FL_OK
        got = fl.device_block_bytes(s.pool, n, dev)
        assert np.array_equal(got[28:48], data[:20])
        assert np.array_equal(got[:28], data[:28])                 # every other block untouched
        st = s.status()
        assert st["bytes_swapped_out"] == 20 * n and st["bytes_swapped_in"] == 20 * n
        model = replay_trace(s)
        for k, b in enumerate(dev):
            model.block(int(b))[:] = data[k]
        model.swap_out([int(b) for b in out_d], [int(b) for b in out_h])
        model.swap_in([int(b) for b in dev[28:48]], [int(b) for b in out_h])
        for k, b in enumerate(dev):
            assert np.array_equal(got[k], model.block(int(b)))
    finally:
        s.close()


# ------------------------------------------------------------------ the whole layer step on the tiny configuration
def test_layer_step_tiny(H):
    wl = synth.make_workload("tiny")
    s = _session(H, wl)
    try:
        s.fill_prefix_kv()
        sh = wl.shape
        T = wl.n_tokens
        x = wl.x("q")
        yb = {m: wl.y_base(m) for m in "qkvo"}
        tx = H.f32_to_dev(x, s.dev)
        ty = {m: H.f32_to_dev(yb[m], s.dev) for m in "qkvo"}
        s.sgmv([ty["q"], ty["k"], ty["v"]], tx, ["q", "k", "v"])
        s.kv_append(ty["k"], ty["v"])
        attn = torch.empty(T, sh.n_q_heads, 128, dtype=torch.bfloat16, device=s.dev)
        s.attention(attn, ty["q"])
        s.sgmv([ty["o"]], attn.view(T, -1), ["o"])
        torch.cuda.synchronize()
        model = replay_trace(s)
        tables = [[int(b) for b in t] for t in s.kv_tables]
        for i in range(wl.n_req):
            kp, vp = wl.kv_prefix(i)
            model.kv_append(synth.bf16_bits(kp), synth.bf16_bits(vp), [0, len(kp)], [tables[i]], [0], sh.n_kv_heads, 128)
        seg, ids = wl.segments()
        ref = attention_layer_step(model, x, yb, {m: oracle_adapters(wl, m) for m in "qkvo"}, seg, ids, wl.req_indptr,
                                   tables, wl.prefix_lens, wl.new_lens, sh.n_q_heads, sh.n_kv_heads, 128, wl.scale,
                                   1.0 / math.sqrt(128))
        for m in "qkv":
            assert_close(H.dev_to_f32(ty[m]), ref[m], m)
        assert_close(H.dev_to_f32(attn), ref["attn"], "attn")
        assert_close(H.dev_to_f32(ty["o"]), ref["o"], "o")
    finally:
        s.close()


# ------------------------------------------------------------------ the same step replayed from a CUDA graph
def test_layer_step_replayed_from_cuda_graph_is_bit_identical(H):
    wl = synth.make_workload("prefill7b", n_req=5, len_range=(60, 300), n_adapters=4)
    s = _session(H, wl)
    try:
        s.fill_prefix_kv()
        sh, T = wl.shape, wl.n_tokens
        tx = H.f32_to_dev(wl.x("q"), s.dev)
        y0 = {m: H.f32_to_dev(wl.y_base(m), s.dev) for m in "qkvo"}
        ty = {m: y0[m].clone() for m in "qkvo"}
        attn = torch.zeros(T, sh.n_q_heads, 128, dtype=torch.bfloat16, device=s.dev)
        main = torch.cuda.Stream()

        def compute():
            s.sgmv([ty["q"], ty["k"], ty["v"]], tx, ["q", "k", "v"], stream=main)
            s.kv_append(ty["k"], ty["v"], stream=main)
            s.attention(attn, ty["q"], stream=main)
            s.sgmv([ty["o"]], attn.view(T, -1), ["o"], stream=main)

        with torch.cuda.stream(main):
            compute()                                   # eager (also the first-use set-up of every kernel)
            main.synchronize()
            want = {m: ty[m].clone() for m in "qkvo"}
            want_attn = attn.clone()
            g = torch.cuda.CUDAGraph()
            for m in "qkvo":
                ty[m].copy_(y0[m])
            main.synchronize()
            with torch.cuda.graph(g, stream=main):
                compute()
            for _ in range(2):                          # replay twice from the same inputs
                for m in "qkvo":
                    ty[m].copy_(y0[m])
                attn.zero_()
                g.replay()
                main.synchronize()
                for m in "qkvo":
                    assert torch.equal(ty[m], want[m]), m
                assert torch.equal(attn, want_attn)
        assert s.status()["device_flags"] == 0
    finally:
        s.close()


# ------------------------------------------------------------------ q/k/v projection with the KV store folded in
@pytest.mark.parametrize("name", ["tiny", "prefill7b", "decode13b", "gqa34b", "swapstress"])
def test_sgmv_qkv_append_equals_projection_then_append(H, name):
    from paper_2505_03756_b200 import binding as fl
    wl = synth.make_workload(name, **REDUCED[name])
    s = _session(H, wl)
    try:
        s.fill_prefix_kv()
        sh, T = wl.shape, wl.n_tokens
        tx = H.f32_to_dev(wl.x("q"), s.dev)
        seg, ids = wl.segments()
        for drop_some in (False, True):           # second pass: every other segment has no adapter (base K/V only)
            lora = s.t_seg_lora
            if drop_some:
                mixed = ids.copy()
                mixed[::2] = -1
                lora = torch.from_numpy(mixed).to(s.dev)
            tables = [[int(b) for b in t] for t in s.kv_tables]
            blocks = sorted({b for t in tables for b in t})
            # reference: the two calls
            ty = {m: H.f32_to_dev(wl.y_base(m), s.dev) for m in "qkv"}
            ws = s.workspace("sgmv", fl.fl_lora_sgmv_workspace(T, 3))
            fl.fl_lora_sgmv_multi(s.pool, [ty["q"], ty["k"], ty["v"]], tx, [s.mat_index[m] for m in "qkv"], s.t_seg_indptr,
                                  lora, s.n_seg, T, wl.scale, ws)
            s.kv_append(ty["k"], ty["v"])
            torch.cuda.synchronize()
            want_q = ty["q"].clone()
            want_blocks = fl.device_block_bytes(s.pool, s.block_bytes, blocks)
            # scribble over the new tokens' slots so that a missing write shows
            junk = torch.full_like(ty["k"], 7.0)
            s.kv_append(junk, junk)
            # the fused call
            tz = {m: H.f32_to_dev(wl.y_base(m), s.dev) for m in "qkv"}
            fl.fl_lora_sgmv_qkv_append(s.pool, tz["q"], tz["k"], tz["v"], tx, s.mat_index["q"], s.mat_index["k"],
                                       s.mat_index["v"], s.t_seg_indptr, lora, s.n_seg, T, wl.scale, s.t_req_indptr,
                                       s.t_tbl_indptr, s.t_tbl, s.t_prefix, wl.n_req, sh.n_kv_heads, ws)
            torch.cuda.synchronize()
            assert s.status()["device_flags"] == 0
            assert torch.equal(tz["q"], want_q)
            got_blocks = fl.device_block_bytes(s.pool, s.block_bytes, blocks)
            assert np.array_equal(got_blocks, want_blocks), (name, drop_some)
            # and against the oracle itself: q, and the K, V rows read back out of the pool blocks
            lid = mixed if drop_some else ids
            x = wl.x("q")
            want = {m: lora_project(wl.y_base(m), x, seg, lid, oracle_adapters(wl, m), wl.scale) for m in "qkv"}
            assert_close(H.dev_to_f32(tz["q"]), want["q"], f"{name}/fused q")
            pos_of = {b: k for k, b in enumerate(blocks)}
            gb = got_blocks.view(np.uint16).reshape(len(blocks), 2, sh.n_kv_heads, sh.block_tokens, 128)
            for i in range(wl.n_req):
                lo, hi = int(wl.req_indptr[i]), int(wl.req_indptr[i + 1])
                pos = int(wl.prefix_lens[i]) + np.arange(hi - lo)
                blk = np.array([pos_of[tables[i][e]] for e in pos // sh.block_tokens])
                rows = op.bf16_bits_to_f64(gb[blk, :, :, pos % sh.block_tokens, :])       # [n, 2, n_kv, 128]
                assert_close(rows[:, 0].reshape(hi - lo, -1), want["k"][lo:hi], f"{name}/fused K in pool")
                assert_close(rows[:, 1].reshape(hi - lo, -1), want["v"][lo:hi], f"{name}/fused V in pool")
            # k, v inputs are left as they were
            assert np.array_equal(H.dev_to_f32(tz["k"]), wl.y_base("k")) and np.array_equal(H.dev_to_f32(tz["v"]), wl.y_base("v"))
    finally:
        s.close()


@pytest.mark.parametrize("heads", [(6, 2), (64, 2), (5, 5)])
def test_attention_unusual_head_groupings(H, heads):
    # odd group sizes take the one-head-per-unit path of the tensor-core kernel; a group wider than the decode
    # kernel's 16 rows sends even one-token requests through the prefill kernel
    n_q, n_kv = heads
    sh = synth.LayerShape(n_q * 128, n_q, n_kv)
    wl = synth.make_workload("tiny", n_req=4, len_range=(0, 0), n_adapters=1, shape=sh)
    wl.prefix_lens[:] = [200, 0, 33, 500]
    wl.new_lens[:] = [1, 140, 300, 2]
    wl.pool_blocks = 160
    for kernel in (0, 1):
        _attention_case(H, wl, prefill_kernel=kernel)


def test_attention_odd_tile_counts_without_grouped_heads(H):
    # one head per KV head: a unit pairs two consecutive 128-row tiles of a request; with 1, 3, 5 and 7 tiles the first
    # tile goes alone and the pairs start at token 128, with 2 and 4 tiles they start at token 0; ragged last tiles
    sh = synth.LayerShape(512, 4, 4)
    wl = synth.make_workload("tiny", n_req=6, len_range=(0, 0), n_adapters=1, shape=sh)
    wl.prefix_lens[:] = [0, 130, 16, 300, 0, 77]
    wl.new_lens[:] = [100, 300, 256, 640, 512, 800]
    wl.pool_blocks = 320
    _attention_case(H, wl)


def test_attention_output_on_a_16_byte_boundary(H):
    """The output pointer must be 16-byte aligned; on a 32-byte boundary the tensor-core kernel stores 32 bytes per
    instruction, otherwise 16: the two paths give the same bits."""
    wl = synth.make_workload("prefill7b", n_req=2, len_range=(150, 400))
    want = _attention_case(H, wl)
    s = H.Session(wl, adapters=[])
    try:
        s.build_batch()
        s.fill_prefix_kv()
        k_new, v_new = wl.kv_new()
        q = wl.q()
        s.kv_append(H.f32_to_dev(k_new, s.dev), H.f32_to_dev(v_new, s.dev))
        n = int(np.prod(q.shape))
        buf = torch.zeros(n + 8, dtype=torch.bfloat16, device=s.dev)
        out = buf[8:].view(wl.n_tokens, -1)
        assert out.data_ptr() % 32 == 16
        s.attention(out, H.f32_to_dev(q, s.dev))
        torch.cuda.synchronize()
        assert np.array_equal(H.dev_to_f32(out).reshape(want.shape), want)
        assert float(buf[:8].float().abs().sum()) == 0.0
        assert s.status()["device_flags"] == 0
    finally:
        s.close()
