"""Cache swapper of the paper's Section 5, restated step by step in float64 (test infrastructure).

Section 5.1, Eq. 3:  Low_lora = sum_i (1 - (1 - prob_i)^BS)        (oracle/demand.py)
Section 5.2, Eq. 4:  LoRA_Eval_i = max(1, Low_lora / Now_LoRA)
             Eq. 5:  Retain_Eval_i = cost_i * prob_i * (1 - sigmoid(t_i)),  t_i = now - last use,
                     cost_i = node size / host-link bandwidth
             Eq. 6:  Eval_i = LoRA_Eval_i * Retain_Eval_i
Section 5.3: every tick, usage above the upper threshold -> candidates in HBM sorted by increasing Eval are
swapped out one by one; usage below the lower threshold -> candidates in host memory sorted by decreasing
Eval are swapped in one by one; "until the HBM is at a balanced status".

Readings where the paper is silent: the Eq. 4 coefficient applies to LoRA nodes (KV nodes take 1: as a factor
common to all nodes it would change no order); t_i is in seconds; "balanced" = usage back inside
[lower, upper]; a swap-in that would push usage above the upper threshold is skipped; equal Eval keeps the
lower node index first.

Pins (tests/test_oracle_swapper.py): Eq. 4 equals 1 at or above the demand and the ratio below it; Eq. 5 at
t = 0 is cost * prob / 2, decays monotonically and is linear in cost and prob; a hand-worked five-node tick
in each direction (tests/golden/swapper_tick.txt); nothing moves between the thresholds.
"""
import math

LORA, KV = 0, 1


def lora_eval(low_lora, now_lora):
    if now_lora <= 0:
        return math.inf if low_lora > 0 else 1.0
    return max(1.0, low_lora / now_lora)


def retain_eval(n_blocks, block_bytes, link_bytes_per_s, visits, total_visits, t):
    cost = n_blocks * block_bytes / link_bytes_per_s
    prob = visits / total_visits
    sigmoid = 1.0 / (1.0 + math.exp(-t))
    return cost * prob * (1.0 - sigmoid)


def evaluate(nodes, prm):
    """nodes: list of dicts (kind, in_hbm, candidate, n_blocks, visits, last_use_s); prm: dict.  Returns Eval_i."""
    le = lora_eval(prm["low_lora"], prm["now_lora"])
    out = []
    for nd in nodes:
        r = retain_eval(nd["n_blocks"], prm["block_bytes"], prm["link_bytes_per_s"], nd["visits"],
                        prm["total_visits"], prm["now_s"] - nd["last_use_s"])
        out.append((le if nd["kind"] == LORA else 1.0) * r)
    return out


def decide(nodes, prm, blocks_used, blocks_total, lru=False, lora_reward=True, only_kind=None):
    """One monitor tick.  Returns (direction, ordered node indices): -1 swap-out, +1 swap-in, 0 nothing.

    The paper's ablations (Section 6): lru=True replaces the cost model by last use alone (the variant "WOS":
    least recently used leaves first, most recently used enters first); lora_reward=False drops the coefficient of
    Eq. 4 (the variant "WOL").  blocks_used may include blocks the caller is about to allocate.  only_kind = LORA or KV
    offers nodes of that kind alone (a partition that holds one kind, Section 2.2)."""
    usage = blocks_used / blocks_total
    if prm["lower"] <= usage <= prm["upper"]:
        return 0, []
    if lru:
        ev = [nd["last_use_s"] for nd in nodes]
    else:
        ev = evaluate(nodes, prm if lora_reward else dict(prm, low_lora=0.0))
    out = usage > prm["upper"]
    cand = [i for i, nd in enumerate(nodes) if nd["candidate"] and bool(nd["in_hbm"]) == out and
            (only_kind is None or nd["kind"] == only_kind)]
    cand.sort(key=lambda i: (ev[i] if out else -ev[i], i))
    used, order = float(blocks_used), []
    for i in cand:
        if out:
            if used <= prm["upper"] * blocks_total:
                break
            used -= nodes[i]["n_blocks"]
            order.append(i)
        else:
            if used >= prm["lower"] * blocks_total:
                break
            if used + nodes[i]["n_blocks"] > prm["upper"] * blocks_total:
                continue
            used += nodes[i]["n_blocks"]
            order.append(i)
    return (-1 if out else 1), order
