"""fl_lora_linear: base projection with the LoRA branch folded into the GEMM (Eq. 1, Eq. 2), against the oracle's
y = x W + s (x A_i) B_i, through the C ABI (run on a B200)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import pool as op
from oracle.lora import lora_linear
from paper_2505_03756_b200 import synth

from _util import REDUCED, assert_close, oracle_adapters, replay_trace


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


def _groups(wl):
    return [["q", "k", "v"], ["o"]] + ([["up"], ["down"]] if wl.shape.inter else [])


@pytest.mark.parametrize("name", list(REDUCED))
def test_lora_linear_parity(H, name):
    wl = synth.make_workload(name, **REDUCED[name])
    s = _session(H, wl)
    try:
        seg, ids = wl.segments()
        for grp in _groups(wl):
            x = wl.x(grp[0])
            tx = H.f32_to_dev(x, s.dev)
            tw = [H.f32_to_dev(wl.weight(m), s.dev) for m in grp]
            d_out = dict((n, o) for n, _, o in wl.shape.mats)
            ty = [torch.full((wl.n_tokens, d_out[m]), 7.0, dtype=torch.bfloat16, device=s.dev) for m in grp]
            s.lora_linear(ty, tx, tw, grp)
            torch.cuda.synchronize()
            assert s.status()["device_flags"] == 0
            for m, t in zip(grp, ty):
                want = lora_linear(x, wl.weight(m), seg, ids, oracle_adapters(wl, m), wl.scale)
                assert_close(H.dev_to_f32(t), want, f"{name}/linear {m}")
    finally:
        s.close()


def test_lora_linear_lora_term_alone_and_identities(H):
    """W = 0 leaves the LoRA term as the whole output (so its own error is measured against itself); scale = 0,
    no segments and segments without an adapter give the plain product; an unknown adapter only raises the flag."""
    from paper_2505_03756_b200 import binding as fl
    wl = synth.make_workload("prefill7b", n_req=6, len_range=(20, 260), n_adapters=4)
    s = _session(H, wl)
    try:
        seg, ids = wl.segments()
        x = wl.x("q")
        tx = H.f32_to_dev(x, s.dev)
        W = wl.weight("q")
        T = wl.n_tokens
        ws = s.workspace("linear", fl.fl_lora_linear_workspace(T, 1))
        y = torch.empty(T, 4096, dtype=torch.bfloat16, device=s.dev)
        zero_w = torch.zeros(4096, 4096, dtype=torch.bfloat16, device=s.dev)
        fl.fl_lora_linear(s.pool, y, tx, zero_w, 0, s.t_seg_indptr, s.t_seg_lora, s.n_seg, T, wl.scale, ws)
        want = lora_linear(x, np.zeros_like(W), seg, ids, oracle_adapters(wl, "q"), wl.scale)
        assert_close(H.dev_to_f32(y), want, "linear/W=0")
        tw = H.f32_to_dev(W, s.dev)
        plain = x.astype(np.float64) @ W.astype(np.float64)
        fl.fl_lora_linear(s.pool, y, tx, tw, 0, s.t_seg_indptr, s.t_seg_lora, s.n_seg, T, 0.0, ws)
        got0 = H.dev_to_f32(y)
        assert_close(got0, plain, "linear/scale=0")
        fl.fl_lora_linear(s.pool, y, tx, tw, 0, s.t_seg_indptr, s.t_seg_lora, 0, T, wl.scale, ws)
        assert np.array_equal(H.dev_to_f32(y), got0), "no segments: the plain product, bit for bit the same"
        none = torch.full_like(s.t_seg_lora, -1)
        fl.fl_lora_linear(s.pool, y, tx, tw, 0, s.t_seg_indptr, none, s.n_seg, T, wl.scale, ws)
        assert np.array_equal(H.dev_to_f32(y), got0)
        mixed = ids.copy()
        mixed[::2] = -1
        fl.fl_lora_linear(s.pool, y, tx, tw, 0, s.t_seg_indptr, torch.from_numpy(mixed).to(s.dev), s.n_seg, T,
                          wl.scale, ws)
        got = H.dev_to_f32(y)
        assert_close(got, lora_linear(x, W, seg, mixed, oracle_adapters(wl, "q"), wl.scale), "linear/mixed")
        for k, lid in enumerate(mixed):
            if lid < 0:
                assert np.array_equal(got[seg[k]:seg[k + 1]], got0[seg[k]:seg[k + 1]])
        assert s.status()["device_flags"] == 0
        bad = torch.full_like(s.t_seg_lora, 3000)
        fl.fl_lora_linear(s.pool, y, tx, tw, 0, s.t_seg_indptr, bad, s.n_seg, T, wl.scale, ws)
        assert s.status(clear=True)["device_flags"] & 4
        assert np.array_equal(H.dev_to_f32(y), got0)
        # argument checks
        with pytest.raises(fl.FlError) as e:
            fl.fl_lora_linear(s.pool, y, tx, tw, 0, s.t_seg_indptr, s.t_seg_lora, s.n_seg, T, 1.0, ws[:256])
        assert e.value.code == fl.FL_ENOMEM
        with pytest.raises(fl.FlError):
            fl.fl_lora_linear(s.pool, y, tx, tw, 9, s.t_seg_indptr, s.t_seg_lora, s.n_seg, T, 1.0, ws)
    finally:
        s.close()


@pytest.mark.parametrize("hidden,heads,rank", [(320, (4, 4), 5), (200, (2, 1), 24), (1024, (8, 8), 64)])
def test_lora_linear_odd_shapes_and_ranks(H, hidden, heads, rank):
    """Output widths that end inside a column tile, an input width that ends inside a k-stage, ranks that are no
    multiple of 16, one-token segments next to long ones."""
    shape = synth.LayerShape(hidden, heads[0], heads[1])
    wl = synth.make_workload("swapstress", n_req=12, len_range=(40, 600), n_adapters=5, shape=shape)
    wl.ranks[:] = rank
    s = _session(H, wl)
    try:
        seg, ids = wl.segments()
        for grp in _groups(wl):
            x = wl.x(grp[0])
            tx = H.f32_to_dev(x, s.dev)
            tw = [H.f32_to_dev(wl.weight(m), s.dev) for m in grp]
            d_out = dict((n, o) for n, _, o in wl.shape.mats)
            ty = [torch.full((wl.n_tokens, d_out[m]), -3.0, dtype=torch.bfloat16, device=s.dev) for m in grp]
            s.lora_linear(ty, tx, tw, grp)
            torch.cuda.synchronize()
            for m, t in zip(grp, ty):
                want = lora_linear(x, wl.weight(m), seg, ids, oracle_adapters(wl, m), wl.scale)
                assert_close(H.dev_to_f32(t), want, f"linear {hidden}/{rank}/{m}")
        assert s.status()["device_flags"] == 0
    finally:
        s.close()


@pytest.mark.parametrize("name", list(REDUCED))
def test_lora_linear_qkv_append_stores_kv_in_the_pool(H, name):
    """The fused q/k/v projection with the KV store folded in: q against the oracle, the pool bytes against the oracle's
    byte model fed with the oracle's K, V, and bit for bit against projection followed by fl_kv_append."""
    from paper_2505_03756_b200 import binding as fl
    wl = synth.make_workload(name, **REDUCED[name])
    s = _session(H, wl)
    try:
        s.fill_prefix_kv()
        sh, T = wl.shape, wl.n_tokens
        x = wl.x("q")
        tx = H.f32_to_dev(x, s.dev)
        tw = {m: H.f32_to_dev(wl.weight(m), s.dev) for m in "qkv"}
        dims = dict((n, o) for n, _, o in sh.mats)
        seg, ids = wl.segments()
        tables = [[int(b) for b in t] for t in s.kv_tables]
        blocks = sorted({b for t in tables for b in t})
        # reference: projection into y, then the KV store
        ty = [torch.empty(T, dims[m], dtype=torch.bfloat16, device=s.dev) for m in "qkv"]
        s.lora_linear(ty, tx, [tw[m] for m in "qkv"], ["q", "k", "v"])
        s.kv_append(ty[1], ty[2])
        torch.cuda.synchronize()
        want_blocks = fl.device_block_bytes(s.pool, s.block_bytes, blocks)
        junk = torch.full_like(ty[1], 7.0)
        s.kv_append(junk, junk)                      # a missing write would show
        y_q = torch.full_like(ty[0], -5.0)
        s.lora_linear_qkv_append(y_q, tx, tw["q"], tw["k"], tw["v"])
        torch.cuda.synchronize()
        assert s.status()["device_flags"] == 0
        assert torch.equal(y_q, ty[0])
        got_blocks = fl.device_block_bytes(s.pool, s.block_bytes, blocks)
        assert np.array_equal(got_blocks, want_blocks), name
        # against the oracle
        want = {m: lora_linear(x, wl.weight(m), seg, ids, oracle_adapters(wl, m), wl.scale) for m in "qkv"}
        assert_close(H.dev_to_f32(y_q), want["q"], f"{name}/linear+append q")
        pos_of = {b: k for k, b in enumerate(blocks)}
        gb = got_blocks.view(np.uint16).reshape(len(blocks), 2, sh.n_kv_heads, sh.block_tokens, 128)
        for i in range(wl.n_req):
            lo, hi = int(wl.req_indptr[i]), int(wl.req_indptr[i + 1])
            pos = int(wl.prefix_lens[i]) + np.arange(hi - lo)
            blk = np.array([pos_of[tables[i][e]] for e in pos // sh.block_tokens], dtype=np.int64)
            rows = op.bf16_bits_to_f64(gb[blk, :, :, pos % sh.block_tokens, :])
            assert_close(rows[:, 0].reshape(hi - lo, -1), want["k"][lo:hi], f"{name}/linear+append K in pool")
            assert_close(rows[:, 1].reshape(hi - lo, -1), want["v"][lo:hi], f"{name}/linear+append V in pool")
    finally:
        s.close()


def test_fused_layer_replayed_from_cuda_graph_is_bit_identical(H):
    """The layer with its base projections, recorded once into a CUDA graph after one ordinary pass, replays bit for bit."""
    wl = synth.make_workload("prefill7b", n_req=5, len_range=(60, 300), n_adapters=4)
    s = _session(H, wl)
    try:
        s.fill_prefix_kv()
        sh, T = wl.shape, wl.n_tokens
        tx = H.f32_to_dev(wl.x("q"), s.dev)
        tw = {m: H.f32_to_dev(wl.weight(m), s.dev) for m in "qkvo"}
        y_q = torch.zeros(T, sh.n_q_heads * 128, dtype=torch.bfloat16, device=s.dev)
        y_o = torch.zeros(T, sh.hidden, dtype=torch.bfloat16, device=s.dev)
        attn = torch.zeros(T, sh.n_q_heads, 128, dtype=torch.bfloat16, device=s.dev)
        main = torch.cuda.Stream()

        def compute():
            s.lora_linear_qkv_append(y_q, tx, tw["q"], tw["k"], tw["v"], stream=main)
            s.attention(attn, y_q.view(T, sh.n_q_heads, 128), stream=main)
            s.lora_linear([y_o], attn.view(T, -1), [tw["o"]], ["o"], stream=main)

        with torch.cuda.stream(main):
            compute()
            main.synchronize()
            want = (y_q.clone(), attn.clone(), y_o.clone())
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=main):
                compute()
            for _ in range(2):
                for t in (y_q, attn, y_o):
                    t.zero_()
                g.replay()
                main.synchronize()
                assert torch.equal(y_q, want[0]) and torch.equal(attn, want[1]) and torch.equal(y_o, want[2])
        assert s.status()["device_flags"] == 0
    finally:
        s.close()


@pytest.mark.parametrize("name,kw", [("decode13b", dict(n_req=200, len_range=(30, 90), n_adapters=20)),
                                     ("prefill7b", dict(n_req=2, len_range=(400, 600), n_adapters=2))])
def test_lora_linear_mid_sized_batches(H, name, kw):
    """Batches between the decode and the prefill regime: a few token tiles, so the call picks 128-column tiles (with
    LoRA stages for the long segments, without them for the batch of one-token segments)."""
    wl = synth.make_workload(name, **kw)
    s = _session(H, wl)
    try:
        seg, ids = wl.segments()
        d_out = dict((n, o) for n, _, o in wl.shape.mats)
        for grp in _groups(wl):
            x = wl.x(grp[0])
            tx = H.f32_to_dev(x, s.dev)
            tw = [H.f32_to_dev(wl.weight(m), s.dev) for m in grp]
            ty = [torch.full((wl.n_tokens, d_out[m]), 3.0, dtype=torch.bfloat16, device=s.dev) for m in grp]
            s.lora_linear(ty, tx, tw, grp)
            torch.cuda.synchronize()
            for m, t in zip(grp, ty):
                want = lora_linear(x, wl.weight(m), seg, ids, oracle_adapters(wl, m), wl.scale)
                assert_close(H.dev_to_f32(t), want, f"{name}/mid-sized linear {m}")
        assert s.status()["device_flags"] == 0
    finally:
        s.close()
