"""The four large workloads at their full sizes, run as bench.py runs them (one layer step through the
C ABI: the q/k/v projection with the KV store folded in, attention, the o projection), checked against the CPU
oracle on sampled outputs: token rows of every LoRA projection (K and V rows read back out of their pool blocks),
attention rows (first and last new token of sampled requests plus random rows), and the allocator trace.  Every
sampled output is computed by the oracle from the stage's own inputs.  A second test does the same for the layer
with its base projections on the path (fl_lora_linear)."""
import math

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle.attention import attend_rows
from oracle.lora import lora_linear, lora_project
from paper_2505_03756_b200 import synth

from _util import assert_close, replay_trace

N_ROWS = 48        # sampled token rows per projection
N_REQ = 12         # sampled requests for attention and KV


def _rows_sample(wl, rs):
    """First and last token of sampled segments plus random rows."""
    seg, _ = wl.segments()
    rows = set()
    for k in rs.integers(0, len(seg) - 2, 8):
        if seg[k + 1] > seg[k]:
            rows.add(int(seg[k]))
            rows.add(int(seg[k + 1] - 1))
    rows.update(int(t) for t in rs.integers(0, wl.n_tokens - 1, N_ROWS))
    return np.array(sorted(rows))


def _seg_of_rows(wl, rows):
    seg, ids = wl.segments()
    return ids[np.searchsorted(seg, rows, side="right") - 1]


def _check_projection(H, wl, rows, x_rows, yb_rows, got_rows, mat, what):
    lids = _seg_of_rows(wl, rows)
    want = np.empty_like(yb_rows, dtype=np.float64)
    for r in range(len(rows)):
        ad = {int(lids[r]): wl.adapter(int(lids[r]), mat)}
        want[r] = lora_project(yb_rows[r:r + 1], x_rows[r:r + 1], [0, 1], [int(lids[r])], ad, wl.scale)[0]
    assert_close(got_rows, want, what)
    # the LoRA term is a tenth of the base output or less, so the bound above could hide an error in it:
    # output minus base must match the oracle's term to within the noise of the output's one bf16
    # rounding (spacing 2^-8 .. 2^-7 of |y|, rms error about 2^-9 |y|)
    delta_got, delta_want = got_rows - yb_rows, want - yb_rows
    rms = lambda a: float(np.sqrt(np.mean(a * a)))
    assert rms(delta_want) > 0, what
    assert rms(delta_got - delta_want) <= 2.0 ** -8 * rms(want), (what, "LoRA term", rms(delta_got - delta_want), rms(delta_want))


@pytest.mark.parametrize("name", ["prefill7b", "decode13b", "gqa34b", "swapstress"])
def test_full_size_layer_step_sampled(name):
    assert torch.cuda.is_available(), "these tests need a GPU"
    from paper_2505_03756_b200 import binding as fl, harness as H
    wl = synth.make_workload(name)
    sh, T = wl.shape, wl.n_tokens
    s = H.Session(wl, register_all=(name == "swapstress"))
    try:
        s.load_adapters()
        s.build_batch()
        s.fill_prefix_kv()
        rs = synth.Stream(wl.seed, "fullsize-sample")
        rows = _rows_sample(wl, rs)
        groups = [["q", "k", "v"], ["o"]] + ([["up"], ["down"]] if sh.inter else [])
        x = wl.x("q")
        tx = H.f32_to_dev(x, s.dev)
        ty = {}
        yb_rows = {}
        for m in "qkv":
            yb = wl.y_base(m)
            yb_rows[m] = yb[rows].astype(np.float64)
            ty[m] = H.f32_to_dev(yb, s.dev)
            del yb
        s.sgmv_qkv_append(ty["q"], ty["k"], ty["v"], tx)          # k, v results go to the pool blocks only
        attn = torch.empty(T, sh.n_q_heads, 128, dtype=torch.bfloat16, device=s.dev)
        s.attention(attn, ty["q"])
        yb = wl.y_base("o")
        yb_rows["o"] = yb[rows].astype(np.float64)
        ty["o"] = H.f32_to_dev(yb, s.dev)
        del yb
        s.sgmv([ty["o"]], attn.view(T, -1), ["o"])
        torch.cuda.synchronize()
        assert s.status()["device_flags"] == 0
        trows = torch.from_numpy(rows).to(s.dev)

        def take(t):
            return H.dev_to_f32(t.view(T, -1)[trows]).astype(np.float64)

        bt = sh.block_tokens
        blocks = {}

        def block(b):
            if b not in blocks:
                blocks[b] = fl.fl_block_read(s.pool, int(b), s.block_bytes).view(np.uint16).reshape(2, sh.n_kv_heads, bt, 128)
            return blocks[b]

        def kv_rows_from_pool(tokens):
            """K and V rows of the given token rows, read through the requests' block tables: [n, 2, n_kv * 128]."""
            out = np.empty((len(tokens), 2, sh.n_kv_heads * 128), dtype=np.float64)
            for k, t in enumerate(tokens):
                i = int(np.searchsorted(wl.req_indptr, t, side="right") - 1)
                pos = int(wl.prefix_lens[i]) + int(t) - int(wl.req_indptr[i])
                blk = block(s.kv_tables[i][pos // bt])
                out[k] = synth.bf16_to_f32(blk[:, :, pos % bt, :]).reshape(2, -1)
            return out

        # a2/a3 (+ a4): sampled rows of every projection; k and v come out of the pool blocks
        x_rows = x[rows].astype(np.float64)
        kv_got = kv_rows_from_pool(rows)
        _check_projection(H, wl, rows, x_rows, yb_rows["q"], take(ty["q"]), "q", f"{name}/q")
        _check_projection(H, wl, rows, x_rows, yb_rows["k"], kv_got[:, 0], "k", f"{name}/k in pool")
        _check_projection(H, wl, rows, x_rows, yb_rows["v"], kv_got[:, 1], "v", f"{name}/v in pool")
        for m in "kv":      # the inputs of the fused call are left as they were
            assert np.array_equal(take(ty[m]), yb_rows[m]), m
        _check_projection(H, wl, rows, take(attn), yb_rows["o"], take(ty["o"]), "o", f"{name}/o")
        if sh.inter:
            for m, src in (("up", "o"), ("down", "up")):
                yb = wl.y_base(m)
                yb_rows[m] = yb[rows].astype(np.float64)
                ty[m] = H.f32_to_dev(yb, s.dev)
                del yb
                x_in = take(ty[src])
                s.sgmv([ty[m]], ty[src], [m])
                torch.cuda.synchronize()
                _check_projection(H, wl, rows, x_in, yb_rows[m], take(ty[m]), m, f"{name}/{m}")
        # a1: allocator trace replayed on the model, free lists bit for bit
        model = replay_trace(s)
        assert np.array_equal(fl.fl_pool_snapshot(s.pool), np.array(model.free_list(), dtype=np.uint32))
        # a5/a6 on sampled requests: the context is the cached prefix plus the new K, V as the pool holds them
        reqs = sorted(set(int(r) for r in rs.integers(0, wl.n_req - 1, N_REQ)) | {0, wl.n_req - 1})
        q_all = ty["q"].view(T, sh.n_q_heads, 128)
        for i in reqs:
            lo, hi = int(wl.req_indptr[i]), int(wl.req_indptr[i + 1])
            n, p = hi - lo, int(wl.prefix_lens[i])
            if n == 0:
                continue
            kv_new = kv_rows_from_pool(np.arange(lo, hi)).reshape(n, 2, sh.n_kv_heads, 128)
            k_new, v_new = kv_new[:, 0], kv_new[:, 1]
            # V slots behind the request's last token are cleared
            last = p + n - 1
            if (last + 1) % bt:
                assert not block(s.kv_tables[i][last // bt])[1, :, last % bt + 1:, :].any(), (name, i)
            kp, vp = wl.kv_prefix(i)
            k_ctx = np.concatenate([kp, k_new]).astype(np.float64)
            v_ctx = np.concatenate([vp, v_new]).astype(np.float64)
            js = sorted({0, n - 1} | set(int(j) for j in rs.integers(0, n - 1, 2)))
            q_rows = H.dev_to_f32(q_all[lo:hi][js])
            want = attend_rows(q_rows, [p + j for j in js], k_ctx, v_ctx, 1.0 / math.sqrt(128))
            got = H.dev_to_f32(attn[lo:hi][js])
            assert_close(got, want, f"{name}/attention request {i}")
    finally:
        s.close()


@pytest.mark.parametrize("name", ["prefill7b", "decode13b", "gqa34b", "swapstress"])
def test_full_size_fused_projections_sampled(name):
    """y = x W + s (x A) B in one GEMM (fl_lora_linear) at the full batch sizes, sampled token rows against the oracle."""
    assert torch.cuda.is_available(), "these tests need a GPU"
    from paper_2505_03756_b200 import harness as H
    wl = synth.make_workload(name)
    if name == "gqa34b":                    # the same batch in a pool that just fits (the 60 GB slab adds nothing here)
        wl.pool_blocks = int(sum(-(-(int(p) + int(n)) // wl.shape.block_tokens) for p, n in zip(wl.prefix_lens, wl.new_lens))) + 2000
    sh, T = wl.shape, wl.n_tokens
    s = H.Session(wl, scramble=False, register_all=(name == "swapstress"))
    try:
        s.load_adapters()
        s.build_batch()
        rs = synth.Stream(wl.seed, "fullsize-linear")
        rows = _rows_sample(wl, rs)
        lids = _seg_of_rows(wl, rows)
        trows = torch.from_numpy(rows).to(s.dev)
        dims = {n: (i, o) for n, i, o in sh.mats}
        groups = [["q", "k", "v"], ["o"]] + ([["up"], ["down"]] if sh.inter else [])
        for grp in groups:
            x = wl.x(grp[0])
            tx = H.f32_to_dev(x, s.dev)
            tw = [H.f32_to_dev(wl.weight(m), s.dev) for m in grp]
            ty = [torch.empty(T, dims[m][1], dtype=torch.bfloat16, device=s.dev) for m in grp]
            s.lora_linear(ty, tx, tw, grp)
            torch.cuda.synchronize()
            assert s.status()["device_flags"] == 0
            x_rows = x[rows].astype(np.float64)
            for m, t in zip(grp, ty):
                W = wl.weight(m)
                want = np.empty((len(rows), dims[m][1]), dtype=np.float64)
                for r in range(len(rows)):
                    ad = {int(lids[r]): wl.adapter(int(lids[r]), m)}
                    want[r] = lora_linear(x_rows[r:r + 1], W, [0, 1], [int(lids[r])], ad, wl.scale)[0]
                got = H.dev_to_f32(t[trows]).astype(np.float64)
                assert_close(got, want, f"{name}/linear {m}")
                base = x_rows @ W.astype(np.float64)
                rms = lambda a: float(np.sqrt(np.mean(a * a)))
                assert rms((got - base) - (want - base)) <= 2.0 ** -8 * rms(want), (name, m, "LoRA term")
            del tx, tw, ty
    finally:
        s.close()
