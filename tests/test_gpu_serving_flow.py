"""The cache manager's tree and the swapper driving the hot path on a GPU: a multi-turn conversation whose
second and third turns reuse the KV blocks the tree matched (Section 4.2), an eviction chosen by the cost model
(Section 5.3) carried out with fl_swap_out, a root-first swap-in before the next turn, and a second adapter whose
branch shares nothing (Eq. 2).  Every turn's attention output is compared with the oracle's full recomputation of
the whole conversation: reused prefix KV, also after a round trip through host memory, must equal recomputation."""
import math

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle.attention import attend_request
from oracle.lora import lora_project
from paper_2505_03756_b200 import synth

from _util import assert_close

VOCAB = 384


def test_multi_turn_conversation_through_tree_swapper_and_kernels():
    assert torch.cuda.is_available(), "this test needs a GPU"
    from paper_2505_03756_b200 import binding as fl, harness as H
    sh = synth.LayerShape(1024, 8, 8)
    bt, nq, nkv, d = sh.block_tokens, sh.n_q_heads, sh.n_kv_heads, 128
    wl = synth.make_workload("tiny", n_req=2, len_range=(0, 1), n_adapters=2, shape=sh)
    wl.pool_blocks = 96
    s = H.Session(wl, adapters=[0, 1], extra_host_blocks=32)
    tree = fl.fl_tree_create(bt)
    try:
        dev = s.dev
        s.load_adapters()
        for a in (0, 1):
            fl.fl_tree_add_lora(tree, a, s.lora_tables[a], 1, 0.0)
        rs = synth.Stream(77, "serving-flow")
        # a token's layer input and base projections depend on the token only, so cached KV equals recomputed KV
        emb = synth.round_bf16(rs.normal((VOCAB, sh.hidden), 1.0))
        base = {m: synth.round_bf16(rs.normal((VOCAB, sh.hidden), 1.0)) for m in "qkv"}
        t_emb = H.f32_to_dev(emb, dev)
        t_base = {m: H.f32_to_dev(base[m], dev) for m in "qkv"}
        mats = {m: s.mat_index[m] for m in "qkv"}
        now = [1.0]

        def oracle_turn(lora, tokens, n_prefix):
            tok = np.asarray(tokens)
            proj = {}
            for m in "qkv":
                y = lora_project(base[m][tok], emb[tok], [0, len(tok)], [lora], {lora: wl.adapter(lora, m)}, wl.scale)
                proj[m] = synth.round_bf16(y.astype(np.float32)).astype(np.float64)      # q, K, V are stored in bf16
            out = attend_request(proj["q"].reshape(-1, nq, d)[n_prefix:], proj["k"].reshape(-1, nkv, d),
                                 proj["v"].reshape(-1, nkv, d), n_prefix, 1.0 / math.sqrt(d))
            return out

        def run_turn(lora, tokens):
            """Match, swap in what lives in host memory, run the layer step on the unmatched tokens, insert."""
            now[0] += 1.0
            ln, path, matched = fl.fl_tree_match(tree, lora, tokens, now[0])
            stats, _, _ = fl.fl_tree_stats(tree)
            for n in [ln] + path:                                    # root first
                if not stats[n]["in_hbm"]:
                    host_blocks = fl.fl_tree_node_blocks(tree, n)
                    new_dev = s.alloc(len(host_blocks))
                    fl.fl_swap_in(s.pool, new_dev, host_blocks, torch.cuda.current_stream())
                    torch.cuda.synchronize()
                    s.free(np.array(host_blocks, dtype=np.uint32), host=True)
                    fl.fl_tree_set_location(tree, n, 1, new_dev)
            if matched == len(tokens):                               # keep at least one token to compute
                matched -= bt
                path = path[:-1]
            prefix_blocks = [fl.fl_tree_node_blocks(tree, n)[0] for n in path]
            n_new = len(tokens) - matched
            new_blocks = s.alloc(-(-n_new // bt))
            tok = torch.tensor(tokens[matched:], dtype=torch.long, device=dev)
            x = t_emb[tok].contiguous()
            y = {m: t_base[m][tok].contiguous() for m in "qkv"}
            i32 = lambda v: torch.tensor(v, dtype=torch.int32, device=dev)
            seg, ids = i32([0, n_new]), i32([lora])
            ws = s.workspace("sgmv", fl.fl_lora_sgmv_workspace(n_new, 3))
            fl.fl_lora_sgmv_multi(s.pool, [y["q"], y["k"], y["v"]], x, [mats[m] for m in "qkv"], seg, ids, 1, n_new,
                                  wl.scale, ws)
            table = prefix_blocks + [int(b) for b in new_blocks]
            tbl, tbl_ind = i32(table), i32([0, len(table)])
            req, pre, new = i32([0, n_new]), i32([matched]), i32([n_new])
            fl.fl_kv_append(s.pool, y["k"], y["v"], req, tbl_ind, tbl, pre, 1, n_new, nkv)
            out = torch.empty(n_new, nq, d, dtype=torch.bfloat16, device=dev)
            wsa = s.workspace("attn", fl.fl_paged_attention_workspace(1, n_new, len(table), nq, nkv))
            fl.fl_paged_attention(s.pool, out, y["q"], req, tbl_ind, tbl, pre, new, 1, n_new, len(table), nq, nkv,
                                  1.0 / math.sqrt(d), wsa)
            torch.cuda.synchronize()
            assert s.status()["device_flags"] == 0
            # whole new blocks become nodes below the last matched node; a partly filled block is not cached
            n_full = (len(tokens) // bt) - len(path)
            parent = path[-1] if path else ln
            fl.fl_tree_insert(tree, parent, tokens[matched:matched + n_full * bt], new_blocks[:n_full], now[0])
            if n_full < len(new_blocks):
                s.free(new_blocks[n_full:])
            assert_close(H.dev_to_f32(out), oracle_turn(lora, tokens, matched), f"turn of {len(tokens)} tokens")
            return matched

        conv = [int(v) for v in rs.integers(0, VOCAB - 1, 3 * bt)]
        assert run_turn(0, conv) == 0                                  # nothing cached yet
        conv = conv + [int(v) for v in rs.integers(0, VOCAB - 1, 2 * bt + 8)]
        assert run_turn(0, conv) == 3 * bt                             # turn 2 reuses the three blocks of turn 1
        assert run_turn(1, conv[:3 * bt]) == 0                         # another adapter's branch shares nothing
        # the pool is "busy": the cost model picks victims among the HBM leaves; their blocks go to host memory
        arr, n, total, now_lora = fl.fl_tree_stats(tree, raw=True)
        used = sum(arr[i].n_blocks for i in range(n) if arr[i].in_hbm)
        prm = dict(now_s=now[0] + 1, total_visits=total, low_lora=2.0, now_lora=now_lora, block_bytes=s.block_bytes,
                   link_bytes_per_s=50e9, upper=0.5, lower=0.2)
        direction, victims = fl.fl_swapper_decide(arr, prm, used, used + 2)
        assert direction == -1 and victims
        evicted = 0
        while direction == -1 and evicted < 6:                         # leaves first, tick after tick
            for n_id in victims:
                dev_blocks = fl.fl_tree_node_blocks(tree, n_id)
                host_blocks = s.alloc(len(dev_blocks), host=True)
                fl.fl_swap_out(s.pool, dev_blocks, host_blocks, torch.cuda.current_stream())
                torch.cuda.synchronize()
                s.free(np.array(dev_blocks, dtype=np.uint32))
                fl.fl_tree_set_location(tree, n_id, 0, host_blocks)
                evicted += 1
            assert fl.fl_tree_check(tree) == (fl.FL_OK, -1)
            arr, n, total, now_lora = fl.fl_tree_stats(tree, raw=True)
            used = sum(arr[i].n_blocks for i in range(n) if arr[i].in_hbm)
            direction, victims = fl.fl_swapper_decide(arr, prm, used, 2 * used - 1 if evicted < 4 else 100 * used)
        assert evicted >= 4
        # turn 3 of the conversation: part of its prefix now lives in host memory and comes back root first
        conv = conv + [int(v) for v in rs.integers(0, VOCAB - 1, bt + 5)]
        assert run_turn(0, conv) == 5 * bt
        assert fl.fl_tree_check(tree) == (fl.FL_OK, -1)
    finally:
        fl.fl_tree_destroy(tree)
        s.close()
