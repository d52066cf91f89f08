"""Usage dependency tree of the paper's Section 4, as plain Python dictionaries (test infrastructure).

Section 4.1: a virtual root connects one subtree per LoRA; LoRA nodes sit on the second layer; below a LoRA node
every path is a conversation prefix and conversations with a common prefix share its nodes.
Section 4.2: a query matches its LoRA node, then KV nodes depth first until a leaf is reached or no node carries
the next tokens; new KV is inserted below the last matched node.  Swap-out starts from the leaves in HBM,
swap-in from the roots of the parts that live in host memory, so every KV cache in HBM is a valid one.
Section 4.3: each node keeps its visit frequency, last use and size, updated when it is generated, matched or
swapped.

Readings where the paper is silent: one KV node per pool block of `bt` tokens (the node label is the block's
token sequence); a generated node starts with one visit; a matched node gets one visit per match.

Pins (tests/test_oracle_tree.py): the paper's own example of Section 4.1 ("To be or not to be" / "To be the
best" share the prefix "To be" below one LoRA and nothing across LoRAs); matching stops at the first missing
block; leaf-only swap-out and root-first swap-in keep the invariant, and breaking either rule is refused.
"""
LORA, KV = 0, 1


class TreeError(Exception):
    pass


class Tree:
    def __init__(self, bt, dependency=True):
        """dependency=False is the paper's ablation "WOM" (Section 6): usage dependencies are ignored, every node is
        a swap candidate and no move is refused, so KV nodes may stay in HBM below a node that has left.
        dependency="kv" models a cache whose adapters and KV caches are managed apart from each other (the static
        partition of Section 2.2): adapters come and go freely whatever lies below them, KV nodes keep the leaf /
        root rules among themselves (a KV node right below its adapter's node counts as a root)."""
        self.bt = bt
        self.dependency = dependency
        self.nodes = []          # dicts: parent, kind, lora_id, in_hbm, visits, last_use_s, blocks, children {label: id}
        self.lora_node = {}
        self.total_visits = 0.0

    def _new(self, **kw):
        kw.setdefault("children", {})
        self.nodes.append(kw)
        return len(self.nodes) - 1

    def add_lora(self, lora_id, blocks, in_hbm, now):
        if lora_id in self.lora_node:
            raise TreeError("adapter already has a node")
        n = self._new(parent=-1, kind=LORA, lora_id=lora_id, in_hbm=bool(in_hbm), visits=0.0, last_use_s=now,
                      blocks=list(blocks))
        self.lora_node[lora_id] = n
        return n

    def _touch(self, n, now):
        self.nodes[n]["visits"] += 1.0
        self.nodes[n]["last_use_s"] = now
        self.total_visits += 1.0

    def match(self, lora_id, tokens, now):
        """Returns (LoRA node, [matched KV nodes in path order], matched token count)."""
        cur = self.lora_node[lora_id]
        self._touch(cur, now)
        path = []
        for k in range(len(tokens) // self.bt):
            label = tuple(int(t) for t in tokens[k * self.bt:(k + 1) * self.bt])
            child = self.nodes[cur]["children"].get(label)
            if child is None:
                break
            self._touch(child, now)
            path.append(child)
            cur = child
        return self.lora_node[lora_id], path, len(path) * self.bt

    def insert(self, parent, tokens, block_ids, now):
        if block_ids and not self.nodes[parent]["in_hbm"]:
            raise TreeError("new KV is generated below a prefix that is in HBM")
        new = []
        for k, b in enumerate(block_ids):
            label = tuple(int(t) for t in tokens[k * self.bt:(k + 1) * self.bt])
            if label in self.nodes[parent]["children"]:
                raise TreeError("block already cached")
            n = self._new(parent=parent, kind=KV, lora_id=self.nodes[parent]["lora_id"], in_hbm=True, visits=1.0,
                          last_use_s=now, blocks=[int(b)])
            self.total_visits += 1.0
            self.nodes[parent]["children"][label] = n
            new.append(n)
            parent = n
        return new

    def _hbm_children(self, n):
        return sum(1 for c in self.nodes[n]["children"].values() if self.nodes[c]["in_hbm"])

    def stats(self):
        """Per node: dict for the swapper (candidate flags per Section 4.2), plus total visits and adapters in HBM."""
        out = []
        for i, nd in enumerate(self.nodes):
            if not self.dependency or (self.dependency == "kv" and nd["kind"] == LORA):
                cand = True
            elif self.dependency == "kv" and not nd["in_hbm"]:
                par = self.nodes[nd["parent"]]
                cand = par["kind"] == LORA or par["in_hbm"]
            elif nd["in_hbm"]:
                cand = self._hbm_children(i) == 0
            else:
                cand = nd["parent"] < 0 or self.nodes[nd["parent"]]["in_hbm"]
            out.append(dict(kind=nd["kind"], in_hbm=int(nd["in_hbm"]), candidate=int(cand), n_blocks=len(nd["blocks"]),
                            visits=nd["visits"], last_use_s=nd["last_use_s"]))
        now_lora = sum(1 for nd in self.nodes if nd["kind"] == LORA and nd["in_hbm"])
        return out, self.total_visits, now_lora

    def set_location(self, n, in_hbm, blocks):
        nd = self.nodes[n]
        in_hbm = bool(in_hbm)
        if len(blocks) != len(nd["blocks"]) or in_hbm == nd["in_hbm"]:
            raise TreeError("bad move")
        free = not self.dependency or (self.dependency == "kv" and nd["kind"] == LORA)
        if not free and not in_hbm and self._hbm_children(n) != 0:
            raise TreeError("only a leaf of the HBM part may leave")
        if not free and in_hbm and nd["parent"] >= 0 and not self.nodes[nd["parent"]]["in_hbm"] and \
                not (self.dependency == "kv" and self.nodes[nd["parent"]]["kind"] == LORA):
            raise TreeError("only a root of the host part may enter")
        nd["in_hbm"] = in_hbm
        nd["blocks"] = [int(b) for b in blocks]

    def valid(self):
        return all(not nd["in_hbm"] or nd["parent"] < 0 or self.nodes[nd["parent"]]["in_hbm"] for nd in self.nodes)

    def invalid(self):
        """(KV nodes in HBM that some ancestor outside HBM makes unusable, KV nodes in HBM): Section 3's
        "invalid KV caches"."""
        bad = total = 0
        for i, nd in enumerate(self.nodes):
            if nd["kind"] != KV or not nd["in_hbm"]:
                continue
            total += 1
            p = nd["parent"]
            while p >= 0 and self.nodes[p]["in_hbm"]:
                p = self.nodes[p]["parent"]
            bad += 1 if p >= 0 else 0
        return bad, total
