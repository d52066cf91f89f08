"""The paper's ablations (Section 6: without the cache manager's dependencies "WOM", without the cost model "WOS",
without the LoRA reward "WOL") on synthetic conversation traces: pins of the oracle's policy switches, parity of the
library's switches with them, and parity of the two trace replays.  Host code on both sides: no GPU needed."""
import numpy as np
import pytest

from oracle import cache_sim as osim, swapper as osw, tree as otree
from paper_2505_03756_b200 import synth

PRM = dict(now_s=10.0, total_visits=10.0, low_lora=4.0, now_lora=2, block_bytes=10**6, link_bytes_per_s=1e9,
           upper=0.5, lower=0.2)


def _node(kind, visits, last_use, in_hbm=1, n_blocks=1):
    return dict(kind=kind, in_hbm=in_hbm, candidate=1, n_blocks=n_blocks, visits=visits, last_use_s=last_use)


# ------------------------------------------------------------------ pins of the oracle's switches (worked by hand)
def test_lru_orders_by_last_use_alone():
    # four resident one-block nodes of nearly the same age, pool of 4 blocks, upper = 0.5: two must leave.  LRU sends
    # out the two used longest ago: node 1 (last use 4.9), then node 0 (5.0).  The cost model keeps node 1, whose nine
    # visits outweigh a tenth of a second of age, and sends out nodes 0 and 2 (one visit each, the older first).
    nodes = [_node(osw.KV, 1.0, 5.0), _node(osw.KV, 9.0, 4.9), _node(osw.KV, 1.0, 5.2), _node(osw.KV, 1.0, 5.5)]
    assert osw.decide(nodes, PRM, 4, 4, lru=True) == (-1, [1, 0])
    assert osw.decide(nodes, PRM, 4, 4) == (-1, [0, 2])
    # swap-in takes the most recently used first
    host = [dict(n, in_hbm=0) for n in nodes]
    assert osw.decide(host, dict(PRM, lower=0.5, upper=1.0), 0, 4, lru=True) == (1, [3, 2])


def test_lora_reward_flips_an_order_and_its_ablation_restores_it():
    # same age, same size: Eq. 5 is proportional to the visits.  KV node: 3 visits; LoRA node: 2 visits, times
    # Low_lora / Now_LoRA = 4 / 2 under Eq. 4 -> 4 > 3, so the KV node leaves first; without the reward 2 < 3 and
    # the LoRA node leaves first.
    nodes = [_node(osw.LORA, 2.0, 9.0), _node(osw.KV, 3.0, 9.0)]
    assert osw.decide(nodes, PRM, 2, 2)[1][0] == 1
    assert osw.decide(nodes, PRM, 2, 2, lora_reward=False)[1][0] == 0
    # at or above the expected demand the coefficient is 1 and the switch changes nothing
    enough = dict(PRM, now_lora=4)
    assert osw.decide(nodes, enough, 2, 2) == osw.decide(nodes, enough, 2, 2, lora_reward=False)


def test_request_for_room_counts_blocks_not_yet_allocated():
    # 2 of 4 blocks used (exactly at upper = 0.5): nothing moves; asking for 2 more pushes usage to 1.0
    nodes = [_node(osw.KV, 1.0, 5.0), _node(osw.KV, 2.0, 5.0)]
    assert osw.decide(nodes, PRM, 2, 4) == (0, [])
    assert osw.decide(nodes, PRM, 2 + 2, 4) == (-1, [0, 1])
    assert osw.decide(nodes, PRM, 2 + 3, 4) == (-1, [0, 1])      # more than the pool holds: everything offered goes


def test_invalid_kv_counts_nodes_below_a_departed_ancestor():
    t = otree.Tree(2, dependency=False)
    ln = t.add_lora(0, [0], True, 0.0)
    k = t.insert(ln, [1, 2, 3, 4, 5, 6], [10, 11, 12], 1.0)
    assert t.invalid() == (0, 3)
    t.set_location(k[1], False, [0])            # the middle block leaves: the block behind it can no longer be matched
    assert t.invalid() == (1, 2)
    t.set_location(ln, False, [1])              # the adapter leaves: nothing below it is usable
    assert t.invalid() == (2, 2)
    strict = otree.Tree(2)
    ln = strict.add_lora(0, [0], True, 0.0)
    k = strict.insert(ln, [1, 2, 3, 4], [10, 11], 1.0)
    with pytest.raises(otree.TreeError):
        strict.set_location(k[0], False, [0])   # with dependencies kept the same move is refused
    assert strict.invalid() == (0, 2) and all(s["candidate"] == 1 for s in t.stats()[0])


# ------------------------------------------------------------------ whole replays worked by hand
TRACES = {
    "A": dict(events=[(0, [1, 2, 3, 4]), (1, [5, 6, 7, 8]), (0, [1, 2, 3, 4, 9, 10]), (1, [5, 6, 11, 12]), (0, [1, 2, 3, 4])],
              kw=dict(n_lora=2, capacity=6, bt=2, lora_blocks=1, tick_every=2)),
    "B": dict(events=[(0, [1, 2, 3, 4]), (0, [1, 2, 3, 4]), (0, [1, 2, 5, 6]), (1, [7, 8, 9, 10]),
                      (1, [7, 8, 11, 12, 13, 14]), (0, [1, 2, 3, 4])],
              kw=dict(n_lora=2, capacity=8, bt=2, lora_blocks=1, tick_every=100)),
    "C": dict(events=[(0, list(range(1, 9))), (0, list(range(11, 19))), (0, list(range(1, 9)))],
              kw=dict(n_lora=2, capacity=10, bt=2, lora_blocks=1, tick_every=1, lora_share=0.4)),
}


def _by_hand():
    import os
    rows = []
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "replay_by_hand.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        rows.append((f[0], f[1], dict(asked_blocks=int(f[2]), hit_blocks=int(f[3]), lora_cold=int(f[4]),
                                      swapped_in=int(f[5]), swapped_out=int(f[6]), used_blocks=int(f[7]), n_nodes=int(f[8]),
                                      invalid_samples=[] if f[9] == "-" else [float(v) for v in f[9].split(",")])))
    return rows


@pytest.mark.parametrize("trace,variant,want", _by_hand())
def test_oracle_replay_matches_the_hand_worked_traces(trace, variant, want):
    c = TRACES[trace]
    kw = dict(c["kw"])
    n_lora = kw.pop("n_lora")
    capacity = kw.pop("capacity")
    got = osim.replay(c["events"], n_lora, variant, capacity, **kw)
    assert got == want, (trace, variant)


@pytest.mark.parametrize("trace,variant,want", _by_hand())
def test_library_replay_matches_the_hand_worked_traces(trace, variant, want):
    from paper_2505_03756_b200 import cache_sim
    c = TRACES[trace]
    kw = dict(c["kw"])
    n_lora = kw.pop("n_lora")
    capacity = kw.pop("capacity")
    assert cache_sim.replay(c["events"], n_lora, variant, capacity, **kw) == want, (trace, variant)


def test_static_partition_switches_by_hand():
    # adapters and KV apart: an adapter may leave above resident KV (which turns unusable), KV keeps its own leaf rule
    t = otree.Tree(2, dependency="kv")
    ln = t.add_lora(0, [0], True, 0.0)
    k = t.insert(ln, [1, 2, 3, 4], [10, 11], 1.0)
    st = t.stats()[0]
    assert [s["candidate"] for s in st] == [1, 0, 1]          # the adapter is offered although n1 lies below it
    with pytest.raises(otree.TreeError):
        t.set_location(k[0], False, [0])                      # not a KV leaf
    t.set_location(ln, False, [1])
    assert t.invalid() == (2, 2)
    t.set_location(k[1], False, [2])
    t.set_location(k[0], False, [3])
    assert [s["candidate"] for s in t.stats()[0]] == [1, 1, 0]   # n1 may come back below its (absent) adapter, n2 not yet
    t.set_location(k[0], True, [12])
    # a partition of one kind: only nodes of that kind are offered, least recently used first
    nodes = [_node(osw.LORA, 5.0, 1.0), _node(osw.KV, 1.0, 3.0), _node(osw.KV, 1.0, 2.0), _node(osw.LORA, 1.0, 0.5)]
    prm = dict(PRM, upper=1.0, lower=0.0)
    assert osw.decide(nodes, prm, 3, 2, lru=True, only_kind=osw.KV) == (-1, [2])
    assert osw.decide(nodes, prm, 3, 1, lru=True, only_kind=osw.LORA) == (-1, [3, 0])


# ------------------------------------------------------------------ the library's switches against the oracle's
def _random_nodes(seed, n):
    rs = synth.Stream(seed, "ablation-nodes")
    u = rs.uniform(4 * n).reshape(4, n)
    nodes = [dict(kind=int(u[0, i] < 0.15), in_hbm=int(u[1, i] < 0.6), candidate=int(u[2, i] < 0.7),
                  n_blocks=1 + int(u[3, i] * 6), visits=float(1 + int(rs.uniform(1)[0] * 50)),
                  last_use_s=float(np.floor(rs.uniform(1)[0] * 5000) / 100)) for i in range(n)]
    for nd in nodes:
        nd["kind"] = osw.LORA if nd["kind"] else osw.KV
    prm = dict(now_s=60.0, total_visits=sum(nd["visits"] for nd in nodes), low_lora=9.0,
               now_lora=sum(1 for nd in nodes if nd["kind"] == osw.LORA and nd["in_hbm"]) or 1,
               block_bytes=65536, link_bytes_per_s=50e9, upper=0.95, lower=0.70)
    return nodes, prm


def test_library_policy_flags_match_oracle():
    from paper_2505_03756_b200 import binding as fl
    for seed in range(8):
        nodes, prm = _random_nodes(seed, 300)
        used = sum(nd["n_blocks"] for nd in nodes if nd["in_hbm"])
        for total in (int(used / 0.99), int(used / 0.4), max(1, used - 7)):     # busy, idle, over-asked
            for flag, kw in ((fl.FL_POLICY_LRU, dict(lru=True)), (fl.FL_POLICY_NO_LORA_REWARD, dict(lora_reward=False)),
                             (0, {})):
                assert fl.fl_swapper_decide_policy(nodes, prm, used, total, flag) == osw.decide(nodes, prm, used, total, **kw)
            for flag, kind in ((fl.FL_POLICY_ONLY_LORA, osw.LORA), (fl.FL_POLICY_ONLY_KV, osw.KV)):
                assert fl.fl_swapper_decide_policy(nodes, prm, used, total, flag | fl.FL_POLICY_LRU) == \
                    osw.decide(nodes, prm, used, total, lru=True, only_kind=kind)
    with pytest.raises(fl.FlError):
        fl.fl_swapper_decide_policy(nodes, prm, used, used, 16)                # unknown flag
    with pytest.raises(fl.FlError):
        fl.fl_swapper_decide_policy(nodes, prm, used, used, 12)                # both kinds at once
    with pytest.raises(fl.FlError):
        fl.fl_swapper_decide(nodes, prm, used + 1, used)                       # the plain tick keeps its range check
    # the tree option
    lt = fl.fl_tree_create(2)
    try:
        fl.fl_tree_set_option(lt, fl.FL_TREE_OPT_DEPENDENCY, 0)
        ln = fl.fl_tree_add_lora(lt, 0, [0], 1, 0.0)
        k = fl.fl_tree_insert(lt, ln, [1, 2, 3, 4, 5, 6], [10, 11, 12], 1.0)
        assert fl.fl_tree_invalid(lt) == (0, 3)
        fl.fl_tree_set_location(lt, k[1], 0, [0])
        assert fl.fl_tree_invalid(lt) == (1, 2)
        fl.fl_tree_set_location(lt, ln, 0, [1])
        assert fl.fl_tree_invalid(lt) == (2, 2)
        assert all(s["candidate"] == 1 for s in fl.fl_tree_stats(lt)[0])
    finally:
        fl.fl_tree_destroy(lt)
    # adapters and KV managed apart: the same moves as in the oracle's pin
    lt = fl.fl_tree_create(2)
    try:
        fl.fl_tree_set_option(lt, fl.FL_TREE_OPT_DEPENDENCY, 2)
        ln = fl.fl_tree_add_lora(lt, 0, [0], 1, 0.0)
        k = fl.fl_tree_insert(lt, ln, [1, 2, 3, 4], [10, 11], 1.0)
        assert [s["candidate"] for s in fl.fl_tree_stats(lt)[0]] == [1, 0, 1]
        with pytest.raises(fl.FlError):
            fl.fl_tree_set_location(lt, k[0], 0, [0])
        fl.fl_tree_set_location(lt, ln, 0, [1])
        assert fl.fl_tree_invalid(lt) == (2, 2)
        fl.fl_tree_set_location(lt, k[1], 0, [2])
        fl.fl_tree_set_location(lt, k[0], 0, [3])
        assert [s["candidate"] for s in fl.fl_tree_stats(lt)[0]] == [1, 1, 0]
        fl.fl_tree_set_location(lt, k[0], 1, [12])
    finally:
        fl.fl_tree_destroy(lt)


# ------------------------------------------------------------------ the two replays, and what the ablations show
CASES = {
    "large adapters": dict(trace=dict(n_lora=24, n_conv=36, n_turns=4), sim=dict(capacity=260, lora_blocks=8, batch_size=16)),
    "small adapters": dict(trace=dict(n_lora=40, n_conv=60, n_turns=3, system_blocks=1, turn_tokens=(8, 40)),
                           sim=dict(capacity=130, lora_blocks=1, batch_size=128)),
}


@pytest.mark.parametrize("case", sorted(CASES))
@pytest.mark.parametrize("popularity", ["uniform", "distinct", "skewed-3"])
def test_library_replay_equals_oracle_replay(case, popularity):
    from paper_2505_03756_b200 import cache_sim
    c = CASES[case]
    events = synth.conversation_trace(21, popularity=popularity, **c["trace"])
    res = {}
    for variant in cache_sim.VARIANTS:
        got = cache_sim.replay(events, c["trace"]["n_lora"], variant, **c["sim"])
        want = osim.replay(events, c["trace"]["n_lora"], variant, **c["sim"])
        assert got == want, (case, popularity, variant)
        res[variant] = want
    # the fixed split serves fewer cached blocks than the unified pool on every trace of this suite
    assert res["static"]["hit_blocks"] <= res["full"]["hit_blocks"]
    # with the dependencies kept no KV cache in HBM is ever invalid; without them some are
    for variant in ("full", "wos", "wol"):
        assert max(res[variant]["invalid_samples"]) == 0.0
    assert res["full"]["asked_blocks"] == res["wom"]["asked_blocks"] > 0
    # the cost model keeps adapters resident better than LRU does, on every trace of this suite
    assert res["full"]["lora_cold"] <= res["wos"]["lora_cold"]


def test_ignoring_dependencies_leaves_invalid_kv_in_hbm():
    c = CASES["large adapters"]
    events = synth.conversation_trace(21, popularity="distinct", **c["trace"])
    m = osim.replay(events, c["trace"]["n_lora"], "wom", **c["sim"])
    assert max(m["invalid_samples"]) > 0.0
