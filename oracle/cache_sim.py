"""Replay of a conversation trace through the cache manager and the cache swapper (test infrastructure).

What the paper's Sections 4 and 5 do per arriving query, on the oracle's tree and cost model, with the HBM pool
reduced to a block budget: match the query (Section 4.2), count what it can reuse, swap in what it needs root
first, make room with the swapper when the pool would get busy (Section 5.3; nodes of the running query are not
offered), insert the new KV below the matched prefix, and run the monitor tick every few queries.  Variants are the
paper's ablations (Section 6): "full", "wos" (LRU instead of the cost model), "wol" (no LoRA reward, Eq. 4 = 1),
"wom" (usage dependencies ignored), and "static": the setting the paper argues against (Section 2.2, Section 3), HBM
cut once into a LoRA partition (a fixed share of the blocks, the paper quotes 0.2) and a KV partition, each run by
LRU on its own and on demand only (no monitor tick moves anything).  Numbers that come out: fraction of asked-for blocks found usable in HBM,
queries whose adapter was not resident, blocks moved each way, and the share of KV nodes in HBM that are invalid
(an ancestor is not in HBM), sampled at every monitor tick.

Readings (the paper gives no replay procedure): whole blocks only; an adapter is a node of `lora_blocks` blocks
that starts in host memory; a request for room is a swapper tick with the needed blocks added to the usage; the
popularity of an adapter in Eq. 3 is its node's share of the visits of all adapter nodes.  Static partition: the LoRA
partition holds floor(share * capacity) blocks, the KV partition the rest; an adapter that is needed evicts the
least recently used other adapters until it fits, whatever KV lies below them (that KV stays in HBM, unusable); KV
that is needed evicts the least recently used KV leaves until it fits; evicted nodes go to host memory as in the
other variants.

Pins (tests/test_policy_ablation.py, tests/golden/replay_by_hand.txt): three small traces replayed by hand, every
counter written out, for every variant.
"""
from oracle import demand, swapper, tree as otree


class CapacityError(Exception):
    pass


def replay(events, n_lora, variant, capacity, bt=16, lora_blocks=2, tick_every=8, batch_size=8,
           block_bytes=65536, link_bytes_per_s=50e9, upper=0.95, lower=0.70, t0=1.0, dt=0.05, lora_share=0.2):
    static = variant == "static"
    t = otree.Tree(bt, dependency=("kv" if static else variant != "wom"))
    cap = {otree.LORA: int(lora_share * capacity), otree.KV: capacity - int(lora_share * capacity)}
    part = {otree.LORA: 0, otree.KV: 0}        # blocks in use per partition (static variant)
    fresh = {"dev": 0, "host": 0}

    def ids(kind, n):
        out = list(range(fresh[kind], fresh[kind] + n))
        fresh[kind] += n
        return out

    for a in range(n_lora):
        t.add_lora(a, ids("host", lora_blocks), False, 0.0)
    m = dict(asked_blocks=0, hit_blocks=0, lora_cold=0, swapped_in=0, swapped_out=0, invalid_samples=[])
    state = {"used": 0}

    def params(now):
        lora_visits = [t.nodes[t.lora_node[a]]["visits"] for a in range(n_lora)]
        s = sum(lora_visits)
        prob = [v / s for v in lora_visits] if s > 0 else [0.0] * n_lora
        return dict(now_s=now, total_visits=t.total_visits, low_lora=demand.expected_distinct(prob, batch_size),
                    now_lora=sum(1 for a in range(n_lora) if t.nodes[t.lora_node[a]]["in_hbm"]),
                    block_bytes=block_bytes, link_bytes_per_s=link_bytes_per_s, upper=upper, lower=lower)

    def decide(stats, now, used):
        return swapper.decide(stats, params(now), used, capacity, lru=(variant == "wos"),
                              lora_reward=(variant != "wol"))

    def move(n, to_hbm):
        nb = len(t.nodes[n]["blocks"])
        t.set_location(n, to_hbm, ids("dev" if to_hbm else "host", nb))
        state["used"] += nb if to_hbm else -nb
        part[t.nodes[n]["kind"]] += nb if to_hbm else -nb
        m["swapped_in" if to_hbm else "swapped_out"] += nb

    def make_room_static(need, kind, pinned, now):
        # least recently used nodes of that partition leave until the request fits; the set of leaves changes as
        # nodes leave, so the candidates are taken afresh each round
        while part[kind] + need > cap[kind]:
            stats, _, _ = t.stats()
            for n in pinned:
                stats[n]["candidate"] = 0
            prm = dict(params(now), upper=1.0, lower=0.0)
            direction, order = swapper.decide(stats, prm, part[kind] + need, cap[kind], lru=True, only_kind=kind)
            if direction != -1 or not order:
                raise CapacityError("the running query does not fit its partition")
            for n in order:
                move(n, False)

    def make_room(need, pinned, now, kind=otree.KV):
        if static:
            return make_room_static(need, kind, pinned, now)
        stats, _, _ = t.stats()
        for n in pinned:
            stats[n]["candidate"] = 0
        direction, order = decide(stats, now, state["used"] + need)
        if direction == -1:
            for n in order:
                move(n, False)
        if state["used"] + need > capacity:
            raise CapacityError("the running query does not fit")

    for step, (lora, tokens) in enumerate(events):
        now = t0 + dt * step
        ln, path, matched = t.match(lora, tokens, now)
        usable = 0
        if t.nodes[ln]["in_hbm"]:
            for n in path:
                if not t.nodes[n]["in_hbm"]:
                    break
                usable += 1
        else:
            m["lora_cold"] += 1
        m["hit_blocks"] += usable
        m["asked_blocks"] += len(tokens) // bt
        pinned = [ln] + path
        for n in pinned:                                   # root first
            if not t.nodes[n]["in_hbm"]:
                make_room(len(t.nodes[n]["blocks"]), pinned, now, t.nodes[n]["kind"])
                move(n, True)
        n_new = len(tokens) // bt - len(path)
        if n_new > 0:
            make_room(n_new, pinned, now)
            t.insert(path[-1] if path else ln, tokens[matched:matched + n_new * bt], ids("dev", n_new), now)
            state["used"] += n_new
            part[otree.KV] += n_new
        if step % tick_every == tick_every - 1:
            if not static:
                stats, _, _ = t.stats()
                direction, order = decide(stats, now, state["used"])
                for n in order:
                    move(n, direction == 1)
            bad, total = t.invalid()
            m["invalid_samples"].append(bad / total if total else 0.0)
    m["used_blocks"] = state["used"]
    m["n_nodes"] = len(t.nodes)
    return m
