"""The four large workloads at their full sizes, run as bench.py runs them (one layer step through the
C ABI), checked against the CPU oracle on sampled outputs: token rows of every LoRA projection, appended
KV rows bit for bit, attention rows (first and last new token of sampled requests plus random rows), and
the allocator trace.  Every sampled output is computed by the oracle from the stage's own inputs."""
import math

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle.attention import attend_rows
from oracle.lora import lora_project
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
        s.sgmv([ty["q"], ty["k"], ty["v"]], tx, ["q", "k", "v"])
        s.kv_append(ty["k"], ty["v"])
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

        # a2/a3: sampled rows of every projection
        x_rows = x[rows].astype(np.float64)
        for m in "qkv":
            _check_projection(H, wl, rows, x_rows, yb_rows[m], take(ty[m]), m, f"{name}/{m}")
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
        # a4 + a5/a6 on sampled requests
        bt = sh.block_tokens
        reqs = sorted(set(int(r) for r in rs.integers(0, wl.n_req - 1, N_REQ)) | {0, wl.n_req - 1})
        k_all, v_all, q_all = ty["k"].view(T, sh.n_kv_heads, 128), ty["v"].view(T, sh.n_kv_heads, 128), ty["q"].view(T, sh.n_q_heads, 128)
        for i in reqs:
            lo, hi = int(wl.req_indptr[i]), int(wl.req_indptr[i + 1])
            n, p = hi - lo, int(wl.prefix_lens[i])
            if n == 0:
                continue
            k_new, v_new = H.dev_to_f32(k_all[lo:hi]), H.dev_to_f32(v_all[lo:hi])
            # KV rows of the first and last new token, bit for bit, read back from their pool blocks
            for j in {0, n - 1}:
                pos = p + j
                blk = fl.fl_block_read(s.pool, int(s.kv_tables[i][pos // bt]), s.block_bytes).view(np.uint16)
                blk = blk.reshape(2, sh.n_kv_heads, bt, 128)
                assert np.array_equal(blk[0, :, pos % bt], synth.bf16_bits(k_new[j])), (name, i, j)
                assert np.array_equal(blk[1, :, pos % bt], synth.bf16_bits(v_new[j])), (name, i, j)
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
