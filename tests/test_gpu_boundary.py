"""Boundary checks on the GPU: read-back of the device-side adapter directory and block tables (Section 4.3),
the host-side deadline of a swap wait (Section 4.3: a query whose blocks are in flight waits), the staging
memory the pool reports, the freed-block poison switch, and the fused q/k/v + KV-store call against the oracle
for blocks of 32 tokens."""
import math

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import pool as op
from oracle.attention import attend_request
from oracle.lora import lora_project
from paper_2505_03756_b200 import synth

from _util import assert_close, oracle_adapters, oracle_context, replay_trace


@pytest.fixture(scope="module")
def H():
    assert torch.cuda.is_available(), "these tests need a GPU"
    from paper_2505_03756_b200 import binding, harness
    return harness


@pytest.mark.parametrize("name,kw", [("gqa34b", dict(n_req=3, len_range=(48, 40), n_adapters=3)),
                                     ("decode13b", dict(n_req=6, len_range=(30, 90), n_adapters=4)),
                                     ("swapstress", dict(n_req=8, len_range=(100, 300), n_adapters=12))])
def test_device_directory_and_tables_match_the_layout_model(H, name, kw):
    from paper_2505_03756_b200 import binding as fl
    wl = synth.make_workload(name, **kw)
    s = H.Session(wl)
    try:
        s.load_adapters()
        arena = []
        for a in s.adapter_ids:
            rank = int(wl.ranks[a])
            n_tab, where = op.lora_layout(s.block_bytes, rank, s.mats)
            entry, table = fl.fl_lora_snapshot(s.pool, a)
            assert (entry["rank"], entry["n_mats"], entry["n_table"]) == (rank, len(s.mats), n_tab)
            assert np.array_equal(table, np.asarray(s.lora_tables[a], dtype=np.uint32)), a
            for m, (d_in, d_out) in enumerate(s.mats):
                e = entry["mats"][m]
                assert (e["a_tab"], e["a_row0"], e["a_rpb"], e["d_in"]) == where[(m, "A")], (a, m)
                assert (e["b_tab"], e["b_row0"], e["b_rpb"], e["d_out"]) == where[(m, "B")], (a, m)
            arena.append((entry["table_off"], entry["n_table"]))
        arena.sort()
        for (o0, n0), (o1, _) in zip(arena, arena[1:]):
            assert o0 + n0 <= o1, "two adapters share table entries"
        with pytest.raises(fl.FlError) as e:
            fl.fl_lora_snapshot(s.pool, 3999)
        assert e.value.code == fl.FL_EBADID
        # an adapter that was unregistered is gone from the device's directory too
        gone = s.adapter_ids[0]
        fl.fl_lora_unregister(s.pool, gone)
        with pytest.raises(fl.FlError):
            fl.fl_lora_snapshot(s.pool, gone)
    finally:
        s.close()


def test_swap_wait_runs_out_then_succeeds(H):
    from paper_2505_03756_b200 import binding as fl
    wl = synth.make_workload("tiny")
    s = H.Session(wl, adapters=[], extra_host_blocks=8)
    try:
        dev, host = s.alloc(4), s.alloc(4, host=True)
        st = s.status()
        assert st["staging_bytes"] == 2 * min(256, wl.pool_blocks, s.n_host_blocks) * s.block_bytes
        side = torch.cuda.Stream()
        khz = getattr(torch.cuda.get_device_properties(0), "clock_rate", 1_900_000)
        with torch.cuda.stream(side):
            torch.cuda._sleep(int(0.5 * khz * 1000))          # a bounded delay of about half a second, then the copies
        fl.fl_swap_in(s.pool, dev, host, side)
        ev = torch.cuda.Event()
        fl.fl_swap_record(s.pool, ev, side)
        assert fl.fl_swap_wait(s.pool, ev, 1) == fl.FL_ETIMEOUT      # the deadline passes on the host, nothing waits on the device
        assert fl.fl_swap_wait(s.pool, ev, 20000) == fl.FL_OK
        assert fl.fl_swap_wait(s.pool, ev, 0) == fl.FL_OK            # a finished event needs no time at all
        assert s.status()["device_flags"] == 0
    finally:
        s.close()


def test_poisoned_freed_block_shows_up_as_nan(H):
    from paper_2505_03756_b200 import binding as fl
    wl = synth.make_workload("tiny")
    s = H.Session(wl, adapters=[])
    try:
        s.build_batch()
        s.fill_prefix_kv()
        k_new, v_new = wl.kv_new()
        s.kv_append(H.f32_to_dev(k_new, s.dev), H.f32_to_dev(v_new, s.dev))
        tq = H.f32_to_dev(wl.q(), s.dev)
        out = torch.zeros(wl.q().shape, dtype=torch.bfloat16, device=s.dev)
        s.attention(out, tq)
        torch.cuda.synchronize()
        clean = H.dev_to_f32(out)
        assert np.isfinite(clean).all()
        fl.fl_pool_set_option(s.pool, fl.FL_OPT_POISON_FREED, 1)
        victim = 1
        fl.fl_block_free(s.pool, s.kv_tables[victim][:1])          # freed while request 1's table still names it
        s.attention(out, tq)
        torch.cuda.synchronize()
        got = H.dev_to_f32(out)
        lo, hi = int(wl.req_indptr[victim]), int(wl.req_indptr[victim + 1])
        assert np.isnan(got[lo:hi]).any(), "a read of a freed block went unnoticed"
        keep = np.ones(len(got), dtype=bool)
        keep[lo:hi] = False
        assert np.array_equal(got[keep], clean[keep])
        # switched off again, a free leaves the bytes alone
        fl.fl_pool_set_option(s.pool, fl.FL_OPT_POISON_FREED, 0)
        other = s.kv_tables[2][:1]
        before = fl.device_block_bytes(s.pool, s.block_bytes, other)
        fl.fl_block_free(s.pool, other)
        assert np.array_equal(fl.device_block_bytes(s.pool, s.block_bytes, other), before)
    finally:
        s.close()


@pytest.mark.parametrize("bt", [32, 8])
def test_fused_qkv_append_with_other_block_sizes_matches_the_oracle(H, bt):
    """Blocks of 32 (and 8) tokens: positions, slots and the cleared V tail against the oracle's byte model."""
    from paper_2505_03756_b200 import binding as fl
    shape = synth.LayerShape(512, 4, 2, block_tokens=bt)
    wl = synth.make_workload("prefill7b", n_req=6, len_range=(30, 200), n_adapters=3, shape=shape, rank=16)
    wl.prefix_lens[:] = [0, 5, 33, 64, 17, 90][:wl.n_req]           # prefixes that end inside a block
    s = H.Session(wl)
    try:
        s.load_adapters()
        s.build_batch()
        sh, T = wl.shape, wl.n_tokens
        x = wl.x("q")
        tx = H.f32_to_dev(x, s.dev)
        seg, ids = wl.segments()
        ty = {m: H.f32_to_dev(wl.y_base(m), s.dev) for m in "qkv"}
        ws = s.workspace("sgmv", fl.fl_lora_sgmv_workspace(T, 3))
        fl.fl_lora_sgmv_qkv_append(s.pool, ty["q"], ty["k"], ty["v"], tx, s.mat_index["q"], s.mat_index["k"],
                                   s.mat_index["v"], s.t_seg_indptr, s.t_seg_lora, s.n_seg, T, wl.scale, s.t_req_indptr,
                                   s.t_tbl_indptr, s.t_tbl, s.t_prefix, wl.n_req, sh.n_kv_heads, ws)
        torch.cuda.synchronize()
        assert s.status()["device_flags"] == 0
        want = {m: lora_project(wl.y_base(m), x, seg, ids, oracle_adapters(wl, m), wl.scale) for m in "qkv"}
        assert_close(H.dev_to_f32(ty["q"]), want["q"], f"q bt={bt}")
        model = replay_trace(s)
        tables = [[int(b) for b in t] for t in s.kv_tables]
        # the oracle's K, V (rounded to bf16 once) stored by the oracle's own byte model
        model.kv_append(op.f64_to_bf16_bits(want["k"]).reshape(T, sh.n_kv_heads, 128),
                        op.f64_to_bf16_bits(want["v"]).reshape(T, sh.n_kv_heads, 128), wl.req_indptr, tables,
                        wl.prefix_lens, sh.n_kv_heads, 128)
        for i in range(wl.n_req):
            p, n = int(wl.prefix_lens[i]), int(wl.new_lens[i])
            lo = int(wl.req_indptr[i])
            gk = np.empty((n, sh.n_kv_heads, 128)), np.empty((n, sh.n_kv_heads, 128))
            got = fl.device_block_bytes(s.pool, s.block_bytes, tables[i]).view(np.uint16)
            got = got.reshape(len(tables[i]), 2, sh.n_kv_heads, bt, 128)
            ref = np.stack([model.block(b).view(np.uint16).reshape(2, sh.n_kv_heads, bt, 128) for b in tables[i]])
            pos = p + np.arange(n)
            g = op.bf16_bits_to_f64(got[pos // bt, :, :, pos % bt, :])       # [n, 2, n_kv, 128]
            r = op.bf16_bits_to_f64(ref[pos // bt, :, :, pos % bt, :])
            assert_close(g[:, 0], r[:, 0], f"K in pool bt={bt}")
            assert_close(g[:, 1], r[:, 1], f"V in pool bt={bt}")
            # slots behind the last token of the last block: V cleared
            last = (p + n - 1) // bt
            tail = (p + n) % bt
            if tail:
                assert not got[last, 1, :, tail:, :].any(), (i, "V tail not cleared")
    finally:
        s.close()


def test_fused_qkv_append_refuses_blocks_it_cannot_address(H):
    from paper_2505_03756_b200 import binding as fl
    shape = synth.LayerShape(256, 2, 1, block_tokens=256)           # 256 tokens per block: beyond the 128 it packs
    wl = synth.make_workload("prefill7b", n_req=2, len_range=(30, 60), n_adapters=2, shape=shape, rank=16)
    s = H.Session(wl)
    try:
        s.load_adapters()
        s.build_batch()
        T = wl.n_tokens
        ty = {m: H.f32_to_dev(wl.y_base(m), s.dev) for m in "qkv"}
        ws = s.workspace("sgmv", fl.fl_lora_sgmv_workspace(T, 3))
        with pytest.raises(fl.FlError) as e:
            fl.fl_lora_sgmv_qkv_append(s.pool, ty["q"], ty["k"], ty["v"], H.f32_to_dev(wl.x("q"), s.dev),
                                       s.mat_index["q"], s.mat_index["k"], s.mat_index["v"], s.t_seg_indptr,
                                       s.t_seg_lora, s.n_seg, T, wl.scale, s.t_req_indptr, s.t_tbl_indptr, s.t_tbl,
                                       s.t_prefix, wl.n_req, shape.n_kv_heads, ws)
        assert e.value.code == fl.FL_EINVAL
    finally:
        s.close()
