"""Usage dependency tree (Section 4): pins of the oracle, then the library's host code against the oracle on a
synthetic multi-turn trace with cache-swapper ticks in between.  No GPU needed."""
import time

import numpy as np
import pytest

from oracle import swapper as osw
from oracle import tree as otree
from paper_2505_03756_b200 import synth

BT = 4


def _ids(words, vocab):
    return [vocab.setdefault(w, len(vocab) + 1) for w in words]


# ------------------------------------------------------------------ the oracle against the paper's own example
def test_section_4_1_example_shared_prefix_and_independent_branches():
    # "To be or not to be" and "To be the best" share the prefix "To be" below one LoRA (Section 4.1); with two
    # tokens per block the tree is  LoRA-1 -> [To be] -> {[or not] -> [to be], [the best]}
    vocab = {}
    t = otree.Tree(2)
    l1 = t.add_lora(1, [100, 101], True, 0.0)
    l2 = t.add_lora(2, [102], True, 0.0)
    s1 = _ids("To be or not to be".split(), vocab)
    s2 = _ids("To be the best".split(), vocab)
    assert t.match(1, s1, 1.0) == (l1, [], 0)
    a = t.insert(l1, s1, [10, 11, 12], 1.0)
    ln, path, m = t.match(1, s2, 2.0)
    assert (ln, path, m) == (l1, [a[0]], 2)                       # only "To be" is reused
    b = t.insert(path[-1], s2[m:], [13], 2.0)
    assert t.nodes[a[0]]["children"].keys() == {tuple(s1[2:4]), tuple(s2[2:4])}
    assert t.match(1, s1, 3.0)[1] == a and t.match(1, s2, 3.0)[1] == [a[0], b[0]]
    assert t.match(2, s1, 3.0) == (l2, [], 0)                     # another LoRA's branch shares nothing (Eq. 2)
    assert t.nodes[a[0]]["visits"] == 1 + 3 and t.nodes[a[0]]["last_use_s"] == 3.0   # generated once, matched three times
    assert t.match(1, s1[:5], 4.0)[2] == 4                        # whole blocks only


def test_swap_rules_keep_every_hbm_node_valid():
    t = otree.Tree(1)
    ln = t.add_lora(0, [5], True, 0.0)
    a, b, c = t.insert(ln, [1, 2, 3], [10, 11, 12], 0.0)
    st, _, now_lora = t.stats()
    assert [s["candidate"] for s in st] == [0, 0, 0, 1] and now_lora == 1     # only the deepest node may leave
    with pytest.raises(otree.TreeError):
        t.set_location(a, False, [0])                                          # a node with a child in HBM stays
    t.set_location(c, False, [0])
    t.set_location(b, False, [1])
    st, _, _ = t.stats()
    assert [s["candidate"] for s in st] == [0, 1, 1, 0]                        # a: HBM leaf; b: root of the host part
    with pytest.raises(otree.TreeError):
        t.set_location(c, True, [12])                                          # its parent is still in host memory
    assert t.valid()
    t.nodes[c]["in_hbm"] = True                                                # what the rule prevents
    assert not t.valid()


# ------------------------------------------------------------------ the library against the oracle
def _trace(seed, n_lora, n_conv, n_turns):
    """Multi-turn conversations: every turn repeats the conversation so far and adds new tokens."""
    rs = synth.Stream(seed, "tree-trace")
    convs = [dict(lora=int(rs.integers(0, n_lora - 1, 1)[0]), tokens=[]) for _ in range(n_conv)]
    system = [int(v) for v in rs.integers(1, 50, 3 * BT)]          # a prompt prefix shared by all conversations
    events = []
    for turn in range(n_turns):
        for ci in rs.permutation(n_conv):
            c = convs[int(ci)]
            if not c["tokens"]:
                c["tokens"] = list(system)
            c["tokens"] = c["tokens"] + [int(v) for v in rs.integers(1, 30000, int(rs.integers(3, 40, 1)[0]))]
            events.append((c["lora"], list(c["tokens"])))
    return events


def test_library_tree_matches_oracle_on_multi_turn_trace():
    from paper_2505_03756_b200 import binding as fl
    n_lora = 6
    events = _trace(3, n_lora, 40, 5)
    ot, lt = otree.Tree(BT), fl.fl_tree_create(BT)
    try:
        next_block, host_block = 0, 0
        for a in range(n_lora):
            blocks = list(range(next_block, next_block + 2))
            next_block += 2
            assert fl.fl_tree_add_lora(lt, a, blocks, 1, 0.0) == ot.add_lora(a, blocks, True, 0.0)
        n_moves = 0
        for step, (lora, tokens) in enumerate(events):
            now = 1.0 + 0.05 * step
            got, want = fl.fl_tree_match(lt, lora, tokens, now), ot.match(lora, tokens, now)
            assert got == want, step
            ln, path, matched = want
            # a query's adapter and prefix must be in HBM before it runs: swap in, root first (Section 4.2)
            for n in [ln] + path:
                if not ot.nodes[n]["in_hbm"]:
                    nb = list(range(next_block, next_block + len(ot.nodes[n]["blocks"])))
                    next_block += len(nb)
                    ot.set_location(n, True, nb)
                    fl.fl_tree_set_location(lt, n, 1, nb)
            n_new = len(tokens) // BT - len(path)
            blocks = list(range(next_block, next_block + n_new))
            next_block += n_new
            parent = path[-1] if path else ln
            new_tok = tokens[matched:matched + n_new * BT]
            assert fl.fl_tree_insert(lt, parent, new_tok, blocks, now) == ot.insert(parent, new_tok, blocks, now)
            if step % 7 == 6:      # a monitor tick: pretend the pool is busy and let the swapper pick victims
                st_o, tot_o, nl_o = ot.stats()
                st_l, tot_l, nl_l = fl.fl_tree_stats(lt)
                assert st_l == st_o and tot_l == tot_o and nl_l == nl_o
                used = sum(s["n_blocks"] for s in st_o if s["in_hbm"])
                prm = dict(now_s=now, total_visits=tot_o, low_lora=3.0, now_lora=nl_o, block_bytes=65536,
                           link_bytes_per_s=50e9, upper=0.95, lower=0.70)
                d_o, order_o = osw.decide(st_o, prm, used, int(used / 0.99))
                arr, n, _, _ = fl.fl_tree_stats(lt, raw=True)
                d_l, order_l = fl.fl_swapper_decide(arr, prm, used, int(used / 0.99))
                assert (d_l, order_l) == (d_o, order_o) and d_o == -1 and order_o
                for n in order_o:
                    hb = list(range(host_block, host_block + len(ot.nodes[n]["blocks"])))
                    host_block += len(hb)
                    ot.set_location(n, False, hb)
                    fl.fl_tree_set_location(lt, n, 0, hb)
                    n_moves += 1
                assert ot.valid() and fl.fl_tree_check(lt) == (fl.FL_OK, -1)
        assert n_moves > 10 and fl.fl_tree_size(lt) == len(ot.nodes) > 500
        for n in range(len(ot.nodes)):
            assert fl.fl_tree_node_blocks(lt, n) == ot.nodes[n]["blocks"]
        # the rule is enforced: an inner node cannot leave HBM, a node below host memory cannot enter
        inner = next(i for i, nd in enumerate(ot.nodes) if nd["in_hbm"] and ot._hbm_children(i) > 0)
        with pytest.raises(fl.FlError) as e:
            fl.fl_tree_set_location(lt, inner, 0, ot.nodes[inner]["blocks"])
        assert e.value.code == fl.FL_EBUSY
        deep = next((i for i, nd in enumerate(ot.nodes) if not nd["in_hbm"] and nd["parent"] >= 0
                     and not ot.nodes[nd["parent"]]["in_hbm"]), None)
        if deep is not None:
            with pytest.raises(fl.FlError) as e:
                fl.fl_tree_set_location(lt, deep, 1, ot.nodes[deep]["blocks"])
            assert e.value.code == fl.FL_EBUSY
    finally:
        fl.fl_tree_destroy(lt)


def test_library_match_is_fast_on_a_large_tree():
    from paper_2505_03756_b200 import binding as fl
    t = fl.fl_tree_create(16)
    try:
        rs = synth.Stream(5, "big-tree")
        ln = fl.fl_tree_add_lora(t, 0, [0], 1, 0.0)
        convs = []
        for c in range(300):                                  # 300 conversations x 128 blocks = 38 400 KV nodes
            tok = rs.integers(1, 30000, 2048).astype(np.int32)
            fl.fl_tree_insert(t, ln, tok, np.arange(128, dtype=np.uint32), 0.0)
            convs.append(tok)
        t0 = time.perf_counter()
        for c in range(300):
            _, path, m = fl.fl_tree_match(t, 0, convs[c], 1.0)
            assert m == 2048
        per_match = (time.perf_counter() - t0) / 300
        assert per_match < 5e-3, per_match     # the paper reports under 0.5 ms on average; this bound only catches a gross regression
    finally:
        fl.fl_tree_destroy(t)
