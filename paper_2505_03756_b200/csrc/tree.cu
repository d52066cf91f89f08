// Usage dependency tree of the cache manager (Section 4): a virtual root, LoRA nodes on the second
// layer, and below each LoRA node a trie of KV nodes, one node per pool block of block_tokens tokens,
// labelled by those tokens.  A path from a LoRA node downwards is a conversation prefix; conversations
// that share a prefix share its nodes (Section 4.3).  Every node records where it lives (HBM or host
// memory), its block ids, its visit count and last use.  Matching (Section 4.2): the LoRA node first,
// then KV nodes depth first, block after block, until no child carries the next tokens.  Swapping
// (Section 4.2, second part): only a node without a child in HBM may leave HBM, only a node whose parent
// is in HBM (or is the virtual root) may enter, so every KV block in HBM has its whole prefix and its
// adapter in HBM too.  Host code only.
#include <string.h>
#include <new>
#include <unordered_map>
#include <vector>
#include "fastpool.h"

namespace {

struct Node {
  int32_t parent;                 // -1 = virtual root (LoRA nodes)
  int32_t kind;                   // FL_NODE_LORA / FL_NODE_KV
  int32_t lora_id;
  int32_t in_hbm;
  int32_t hbm_children;           // children resident in HBM
  double visits, last_use_s;
  std::vector<uint32_t> blocks;   // one block for a KV node, the adapter's table for a LoRA node
  std::vector<int32_t> label;     // KV node: its block_tokens tokens
  std::unordered_multimap<uint64_t, int32_t> children;   // hash of the child's label -> child node
};

uint64_t label_hash(const int32_t* tok, int n) {
  uint64_t h = 0x9E3779B97F4A7C15ull;
  for (int i = 0; i < n; ++i) {
    h ^= (uint64_t)(uint32_t)tok[i] + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2);
    h *= 0xBF58476D1CE4E5B9ull;
  }
  return h;
}

}  // namespace

struct fl_tree {
  int bt = 16;
  int dependency = 1;       // 1: Section 4.2 rules; 0: the ablation that ignores usage dependencies (any node may
                            // move); 2: adapters move freely, KV nodes keep the rules among themselves
  std::vector<Node> nodes;
  std::unordered_map<int32_t, int32_t> lora_node;   // lora id -> node
  double total_visits = 0.0;

  int32_t find_child(int32_t parent, const int32_t* tok) const {
    const Node& p = nodes[parent];
    auto range = p.children.equal_range(label_hash(tok, bt));
    for (auto it = range.first; it != range.second; ++it)
      if (memcmp(nodes[it->second].label.data(), tok, sizeof(int32_t) * bt) == 0) return it->second;
    return -1;
  }
  void touch(int32_t n, double now) {
    nodes[n].visits += 1.0;
    nodes[n].last_use_s = now;
    total_visits += 1.0;
  }
};

extern "C" {

int fl_tree_create(fl_tree** out, int block_tokens) {
  if (!out || block_tokens < 1) return FL_EINVAL;
  fl_tree* t = new (std::nothrow) fl_tree();
  if (!t) return FL_ENOMEM;
  t->bt = block_tokens;
  *out = t;
  return FL_OK;
}

int fl_tree_destroy(fl_tree* t) {
  if (!t) return FL_EINVAL;
  delete t;
  return FL_OK;
}

int fl_tree_add_lora(fl_tree* t, int32_t lora_id, const uint32_t* blocks, uint32_t n_blocks, int in_hbm, double now_s,
                     int32_t* node) {
  if (!t || (n_blocks && !blocks) || lora_id < 0) return FL_EINVAL;
  if (t->lora_node.count(lora_id)) return FL_EBADID;
  Node n;
  n.parent = -1;
  n.kind = FL_NODE_LORA;
  n.lora_id = lora_id;
  n.in_hbm = in_hbm ? 1 : 0;
  n.hbm_children = 0;
  n.visits = 0.0;
  n.last_use_s = now_s;
  n.blocks.assign(blocks, blocks + n_blocks);
  const int32_t id = (int32_t)t->nodes.size();
  t->nodes.push_back(std::move(n));
  t->lora_node[lora_id] = id;
  if (node) *node = id;
  return FL_OK;
}

int fl_tree_match(fl_tree* t, int32_t lora_id, const int32_t* tokens, int n_tokens, double now_s, int32_t* lora_node,
                  int32_t* kv_nodes, int cap, int* n_kv_nodes, int* matched_tokens) {
  if (!t || n_tokens < 0 || (n_tokens && !tokens) || !n_kv_nodes || !matched_tokens || cap < 0 || (cap && !kv_nodes)) return FL_EINVAL;
  auto it = t->lora_node.find(lora_id);
  if (it == t->lora_node.end()) return FL_EBADID;
  int32_t cur = it->second;
  if (lora_node) *lora_node = cur;
  t->touch(cur, now_s);
  int k = 0;
  for (; (k + 1) * t->bt <= n_tokens; ++k) {
    const int32_t child = t->find_child(cur, tokens + (size_t)k * t->bt);
    if (child < 0) break;
    if (k >= cap) return FL_ENOMEM;
    kv_nodes[k] = child;
    t->touch(child, now_s);
    cur = child;
  }
  *n_kv_nodes = k;
  *matched_tokens = k * t->bt;
  return FL_OK;
}

int fl_tree_insert(fl_tree* t, int32_t parent, const int32_t* tokens, int n_new_blocks, const uint32_t* block_ids,
                   double now_s, int32_t* new_nodes) {
  if (!t || parent < 0 || parent >= (int32_t)t->nodes.size() || n_new_blocks < 0 || (n_new_blocks && (!tokens || !block_ids))) return FL_EINVAL;
  if (!t->nodes[parent].in_hbm && n_new_blocks) return FL_EBUSY;    // new KV is generated in HBM, below a resident prefix
  for (int k = 0; k < n_new_blocks; ++k) {
    const int32_t* tok = tokens + (size_t)k * t->bt;
    if (t->find_child(parent, tok) >= 0) return FL_EBADID;           // that block of the conversation is cached already
    Node n;
    n.parent = parent;
    n.kind = FL_NODE_KV;
    n.lora_id = t->nodes[parent].lora_id;
    n.in_hbm = 1;
    n.hbm_children = 0;
    n.visits = 1.0;
    n.last_use_s = now_s;
    n.blocks.assign(1, block_ids[k]);
    n.label.assign(tok, tok + t->bt);
    const int32_t id = (int32_t)t->nodes.size();
    t->nodes.push_back(std::move(n));
    t->total_visits += 1.0;
    t->nodes[parent].children.emplace(label_hash(tok, t->bt), id);
    t->nodes[parent].hbm_children += 1;
    if (new_nodes) new_nodes[k] = id;
    parent = id;
  }
  return FL_OK;
}

int fl_tree_size(fl_tree* t) { return t ? (int)t->nodes.size() : 0; }

int fl_tree_node_blocks(fl_tree* t, int32_t node, uint32_t* blocks, uint32_t cap, uint32_t* n_blocks) {
  if (!t || node < 0 || node >= (int32_t)t->nodes.size() || !n_blocks) return FL_EINVAL;
  const Node& n = t->nodes[node];
  *n_blocks = (uint32_t)n.blocks.size();
  if (blocks) {
    if (cap < n.blocks.size()) return FL_EINVAL;
    if (!n.blocks.empty()) memcpy(blocks, n.blocks.data(), n.blocks.size() * sizeof(uint32_t));
  }
  return FL_OK;
}

int fl_tree_stats(fl_tree* t, fl_node_stat* out, int cap, int* n_nodes, double* total_visits, int32_t* now_lora) {
  if (!t || !n_nodes) return FL_EINVAL;
  const int n = (int)t->nodes.size();
  *n_nodes = n;
  if (total_visits) *total_visits = t->total_visits;
  int loras = 0;
  for (const Node& nd : t->nodes) loras += (nd.kind == FL_NODE_LORA && nd.in_hbm);
  if (now_lora) *now_lora = loras;
  if (!out) return FL_OK;
  if (cap < n) return FL_EINVAL;
  for (int i = 0; i < n; ++i) {
    const Node& nd = t->nodes[i];
    out[i].kind = nd.kind;
    out[i].in_hbm = nd.in_hbm;
    // swap-out candidates: HBM nodes with no child in HBM; swap-in candidates: host nodes right below HBM (or the root)
    if (t->dependency == 0 || (t->dependency == 2 && nd.kind == FL_NODE_LORA))
      out[i].candidate = 1;
    else if (nd.in_hbm)
      out[i].candidate = nd.hbm_children == 0;
    else
      out[i].candidate = nd.parent < 0 || t->nodes[nd.parent].in_hbm ||
                         (t->dependency == 2 && t->nodes[nd.parent].kind == FL_NODE_LORA);
    out[i].n_blocks = (uint32_t)nd.blocks.size();
    out[i].visits = nd.visits;
    out[i].last_use_s = nd.last_use_s;
  }
  return FL_OK;
}

int fl_tree_set_location(fl_tree* t, int32_t node, int in_hbm, const uint32_t* blocks, uint32_t n_blocks) {
  if (!t || node < 0 || node >= (int32_t)t->nodes.size() || (n_blocks && !blocks)) return FL_EINVAL;
  Node& nd = t->nodes[node];
  in_hbm = in_hbm ? 1 : 0;
  if (n_blocks != nd.blocks.size()) return FL_EINVAL;
  if (in_hbm == nd.in_hbm) return FL_EINVAL;
  if (t->dependency == 1 || (t->dependency == 2 && nd.kind == FL_NODE_KV)) {
    if (!in_hbm && nd.hbm_children != 0) return FL_EBUSY;                             // only leaves of the HBM part leave
    if (in_hbm && nd.parent >= 0 && !t->nodes[nd.parent].in_hbm &&
        !(t->dependency == 2 && t->nodes[nd.parent].kind == FL_NODE_LORA))
      return FL_EBUSY;                                                                // only roots of the host part enter
  }
  nd.in_hbm = in_hbm;
  nd.blocks.assign(blocks, blocks + n_blocks);
  if (nd.parent >= 0) t->nodes[nd.parent].hbm_children += in_hbm ? 1 : -1;
  return FL_OK;
}

int fl_tree_set_option(fl_tree* t, int option, int value) {
  if (!t) return FL_EINVAL;
  if (option != FL_TREE_OPT_DEPENDENCY || value < 0 || value > 2) return FL_EINVAL;
  t->dependency = value;
  return FL_OK;
}

int fl_tree_invalid(fl_tree* t, uint32_t* invalid_kv, uint32_t* hbm_kv) {
  if (!t || !invalid_kv || !hbm_kv) return FL_EINVAL;
  // nodes are created parents first, so one pass in id order knows every ancestor's state
  std::vector<char> usable(t->nodes.size());
  uint32_t bad = 0, all = 0;
  for (size_t i = 0; i < t->nodes.size(); ++i) {
    const Node& nd = t->nodes[i];
    usable[i] = nd.in_hbm && (nd.parent < 0 || usable[nd.parent]);
    if (nd.kind == FL_NODE_KV && nd.in_hbm) {
      ++all;
      bad += usable[i] ? 0u : 1u;
    }
  }
  *invalid_kv = bad;
  *hbm_kv = all;
  return FL_OK;
}

int fl_tree_check(fl_tree* t, int32_t* first_bad) {
  if (!t) return FL_EINVAL;
  for (int i = 0; i < (int)t->nodes.size(); ++i) {
    const Node& nd = t->nodes[i];
    int hbm_children = 0;
    for (const auto& kv : nd.children) hbm_children += t->nodes[kv.second].in_hbm;
    const bool orphan = nd.in_hbm && nd.parent >= 0 && !t->nodes[nd.parent].in_hbm;   // an invalid KV cache in HBM
    if (orphan || hbm_children != nd.hbm_children) {
      if (first_bad) *first_bad = i;
      return FL_EBADID;
    }
  }
  return FL_OK;
}

}  // extern "C"
