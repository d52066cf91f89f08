"""Trace replay through the library's dependency tree and cache swapper: the harness behind the policy ablations.

Drives fl_tree_* and fl_swapper_decide_policy query by query with the HBM pool reduced to a block budget, and
reports reuse, adapter cold starts, swap volume and the share of invalid KV nodes for the full policy and the
three ablations of the paper's Section 6 (no cost model, no LoRA reward, no usage dependencies)."""
import numpy as np

from . import binding as fl

VARIANTS = ("full", "wos", "wol", "wom")


class CapacityError(Exception):
    pass


class Replay:
    def __init__(self, n_lora, variant, capacity, bt=16, lora_blocks=2, tick_every=8, batch_size=8,
                 block_bytes=65536, link_bytes_per_s=50e9, upper=0.95, lower=0.70):
        assert variant in VARIANTS
        self.n_lora, self.capacity, self.bt = n_lora, capacity, bt
        self.tick_every, self.batch_size = tick_every, batch_size
        self.fixed = dict(block_bytes=block_bytes, link_bytes_per_s=link_bytes_per_s, upper=upper, lower=lower)
        self.policy = {"wos": fl.FL_POLICY_LRU, "wol": fl.FL_POLICY_NO_LORA_REWARD}.get(variant, 0)
        self.tree = fl.fl_tree_create(bt)
        if variant == "wom":
            fl.fl_tree_set_option(self.tree, fl.FL_TREE_OPT_DEPENDENCY, 0)
        self.next_id = [0, 0]                  # host, device
        self.used = 0
        self.lora_nodes = [fl.fl_tree_add_lora(self.tree, a, self._ids(0, lora_blocks), 0, 0.0) for a in range(n_lora)]
        self.metrics = dict(asked_blocks=0, hit_blocks=0, lora_cold=0, swapped_in=0, swapped_out=0, invalid_samples=[])

    def close(self):
        fl.fl_tree_destroy(self.tree)

    def _ids(self, dev, n):
        first = self.next_id[dev]
        self.next_id[dev] += n
        return np.arange(first, first + n, dtype=np.uint32)

    def _decide(self, arr, now, used):
        n, tot, now_lora = self._last
        visits = np.array([arr[k].visits for k in self.lora_nodes], dtype=np.float64)
        prob = visits / visits.sum() if visits.sum() > 0 else np.zeros(self.n_lora)
        prm = dict(self.fixed, now_s=now, total_visits=tot, now_lora=now_lora,
                   low_lora=fl.fl_expected_lora_demand(prob, self.batch_size))
        return fl.fl_swapper_decide_policy(arr, prm, used, self.capacity, self.policy)

    def _stats(self):
        arr, n, tot, now_lora = fl.fl_tree_stats(self.tree, raw=True)
        self._last = (n, tot, now_lora)
        return arr

    def _move(self, arr, node, to_hbm):
        nb = int(arr[node].n_blocks)
        fl.fl_tree_set_location(self.tree, node, to_hbm, self._ids(1 if to_hbm else 0, nb))
        self.used += nb if to_hbm else -nb
        self.metrics["swapped_in" if to_hbm else "swapped_out"] += nb

    def _make_room(self, need, pinned, now):
        arr = self._stats()
        for n in pinned:
            arr[n].candidate = 0               # the running query's own nodes stay
        direction, order = self._decide(arr, now, self.used + need)
        if direction == -1:
            for n in order:
                self._move(arr, n, 0)
        if self.used + need > self.capacity:
            raise CapacityError("the running query does not fit")

    def query(self, step, lora, tokens, now):
        m, bt = self.metrics, self.bt
        ln, path, matched = fl.fl_tree_match(self.tree, lora, tokens, now)
        chain = [ln] + path
        arr = self._stats()
        resident = [bool(arr[n].in_hbm) for n in chain]
        if resident[0]:
            usable = 0
            while usable < len(path) and resident[1 + usable]:
                usable += 1
            m["hit_blocks"] += usable
        else:
            m["lora_cold"] += 1
        m["asked_blocks"] += len(tokens) // bt
        for k, n in enumerate(chain):          # swap in what the query needs, root first
            if not resident[k]:
                self._make_room(int(arr[n].n_blocks), chain, now)
                self._move(arr, n, 1)
        n_new = len(tokens) // bt - len(path)
        if n_new > 0:
            self._make_room(n_new, chain, now)
            fl.fl_tree_insert(self.tree, chain[-1], tokens[matched:matched + n_new * bt], self._ids(1, n_new), now)
            self.used += n_new
        if step % self.tick_every == self.tick_every - 1:
            arr = self._stats()
            direction, order = self._decide(arr, now, self.used)
            for n in order:
                self._move(arr, n, 1 if direction == 1 else 0)
            bad, total = fl.fl_tree_invalid(self.tree)
            m["invalid_samples"].append(bad / total if total else 0.0)


def replay(events, n_lora, variant, capacity, t0=1.0, dt=0.05, **kw):
    r = Replay(n_lora, variant, capacity, **kw)
    try:
        for step, (lora, tokens) in enumerate(events):
            r.query(step, lora, tokens, t0 + dt * step)
        out = dict(r.metrics)
        out["used_blocks"] = r.used
        out["n_nodes"] = fl.fl_tree_size(r.tree)
        return out
    finally:
        r.close()


def summary(m):
    inv = m["invalid_samples"]
    return dict(hit_rate=m["hit_blocks"] / max(1, m["asked_blocks"]), lora_cold=m["lora_cold"],
                swapped_in=m["swapped_in"], swapped_out=m["swapped_out"],
                invalid_kv=sum(inv) / len(inv) if inv else 0.0)
