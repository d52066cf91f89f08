// Trace replay through the dependency tree and the cache swapper (Sections 4.2, 5.3, 6): what an arriving query
// finds usable in HBM, what has to be swapped, and what the policy variants of the paper's ablations (and the
// static LoRA/KV partition the paper argues against, Section 2.2) make of the same trace.  Host code only; it
// drives the library's own tree and swapper calls.
#include <math.h>
#include <vector>
#include "fastpool.h"

namespace {

struct Replay {
  const fl_replay_config& cfg;
  int n_lora;
  fl_tree* tree = nullptr;
  std::vector<int32_t> lora_nodes;
  uint32_t next_id[2] = {0, 0};       // host, device block ids handed out so far
  uint32_t used = 0;                  // HBM blocks in use
  uint32_t part[2] = {0, 0};          // per kind (FL_NODE_LORA, FL_NODE_KV): the static variant's partitions
  uint32_t cap[2] = {0, 0};
  fl_replay_result res = {};
  std::vector<fl_node_stat> stats;
  std::vector<int32_t> order;
  std::vector<uint32_t> ids;
  double total_visits = 0.0;
  int32_t now_lora = 0;

  explicit Replay(const fl_replay_config& c, int n) : cfg(c), n_lora(n) {}
  ~Replay() { if (tree) fl_tree_destroy(tree); }

  const uint32_t* fresh(int dev, uint32_t n) {
    ids.resize(n);
    for (uint32_t i = 0; i < n; ++i) ids[i] = next_id[dev] + i;
    next_id[dev] += n;
    return ids.data();
  }
  int take_stats() {
    int n = 0;
    int rc = fl_tree_stats(tree, nullptr, 0, &n, nullptr, nullptr);
    if (rc != FL_OK) return rc;
    stats.resize((size_t)n);
    order.resize((size_t)n + 1);
    return fl_tree_stats(tree, stats.data(), n, &n, &total_visits, &now_lora);
  }
  // one call of the swapper on the last statistics: Eq. 3 from the adapters' shares of the visits
  int decide(double now, uint32_t blocks_used, uint32_t blocks_total, uint32_t policy, double upper, double lower,
             int* n_order, int* direction) {
    std::vector<double> prob((size_t)n_lora, 0.0);
    double sum = 0.0;
    for (int a = 0; a < n_lora; ++a) sum += stats[lora_nodes[a]].visits;
    if (sum > 0.0)
      for (int a = 0; a < n_lora; ++a) prob[a] = stats[lora_nodes[a]].visits / sum;
    fl_swap_params prm;
    prm.now_s = now;
    prm.total_visits = total_visits;
    int rc = fl_expected_lora_demand(prob.data(), n_lora, cfg.batch_size, &prm.low_lora);
    if (rc != FL_OK) return rc;
    prm.now_lora = now_lora;
    prm.block_bytes = cfg.block_bytes;
    prm.link_bytes_per_s = cfg.link_bytes_per_s;
    prm.upper = upper;
    prm.lower = lower;
    return fl_swapper_decide_policy(stats.data(), (int)stats.size(), &prm, blocks_used, blocks_total, policy,
                                    order.data(), n_order, direction);
  }
  int move(int32_t node, int to_hbm) {
    const uint32_t nb = stats[node].n_blocks;
    int rc = fl_tree_set_location(tree, node, to_hbm, fresh(to_hbm ? 1 : 0, nb), nb);
    if (rc != FL_OK) return rc;
    if (to_hbm) { used += nb; part[stats[node].kind] += nb; res.swapped_in += nb; }
    else { used -= nb; part[stats[node].kind] -= nb; res.swapped_out += nb; }
    return FL_OK;
  }
  uint32_t policy() const {
    return cfg.variant == FL_REPLAY_WOS ? FL_POLICY_LRU : cfg.variant == FL_REPLAY_WOL ? FL_POLICY_NO_LORA_REWARD : 0u;
  }
  // room for `need` more blocks (of kind `kind` in the static variant), the running query's nodes held back
  int make_room(uint32_t need, int kind, const std::vector<int32_t>& pinned, double now) {
    int n_order = 0, direction = 0;
    if (cfg.variant == FL_REPLAY_STATIC) {
      // least recently used nodes of the partition leave until the request fits; the leaves change as nodes leave
      while (part[kind] + need > cap[kind]) {
        int rc = take_stats();
        if (rc != FL_OK) return rc;
        for (int32_t n : pinned) stats[n].candidate = 0;
        rc = decide(now, part[kind] + need, cap[kind],
                    FL_POLICY_LRU | (kind == FL_NODE_LORA ? FL_POLICY_ONLY_LORA : FL_POLICY_ONLY_KV), 1.0, 0.0, &n_order,
                    &direction);
        if (rc != FL_OK) return rc;
        if (direction != -1 || n_order == 0) return FL_ENOMEM;
        for (int k = 0; k < n_order; ++k)
          if ((rc = move(order[k], 0)) != FL_OK) return rc;
      }
      return FL_OK;
    }
    int rc = take_stats();
    if (rc != FL_OK) return rc;
    for (int32_t n : pinned) stats[n].candidate = 0;
    rc = decide(now, used + need, cfg.capacity, policy(), cfg.upper, cfg.lower, &n_order, &direction);
    if (rc != FL_OK) return rc;
    if (direction == -1)
      for (int k = 0; k < n_order; ++k)
        if ((rc = move(order[k], 0)) != FL_OK) return rc;
    return used + need > cfg.capacity ? FL_ENOMEM : FL_OK;
  }
};

}  // namespace

extern "C" int fl_cache_replay(const fl_replay_config* cfg, int n_lora, const int32_t* event_lora,
                               const int32_t* event_indptr, const int32_t* tokens, int n_events, fl_replay_result* out,
                               double* invalid_samples, uint32_t cap_samples) {
  if (!cfg || !out || n_lora < 1 || n_events < 0 || (n_events && (!event_lora || !event_indptr || !tokens))) return FL_EINVAL;
  if (cfg->variant < FL_REPLAY_FULL || cfg->variant > FL_REPLAY_STATIC || cfg->capacity == 0 || cfg->block_tokens < 1 ||
      cfg->tick_every < 1 || cfg->batch_size < 0 || cfg->lora_blocks == 0 || (cap_samples && !invalid_samples))
    return FL_EINVAL;
  if (cfg->variant == FL_REPLAY_STATIC && !(cfg->lora_share >= 0.0 && cfg->lora_share <= 1.0)) return FL_EINVAL;
  Replay r(*cfg, n_lora);
  int rc = fl_tree_create(&r.tree, cfg->block_tokens);
  if (rc != FL_OK) return rc;
  if (cfg->variant == FL_REPLAY_WOM) fl_tree_set_option(r.tree, FL_TREE_OPT_DEPENDENCY, 0);
  if (cfg->variant == FL_REPLAY_STATIC) {
    fl_tree_set_option(r.tree, FL_TREE_OPT_DEPENDENCY, 2);
    r.cap[FL_NODE_LORA] = (uint32_t)floor(cfg->lora_share * (double)cfg->capacity);
    r.cap[FL_NODE_KV] = cfg->capacity - r.cap[FL_NODE_LORA];
  }
  r.lora_nodes.resize((size_t)n_lora);
  for (int a = 0; a < n_lora; ++a)
    if ((rc = fl_tree_add_lora(r.tree, a, r.fresh(0, cfg->lora_blocks), cfg->lora_blocks, 0, 0.0, &r.lora_nodes[a])) != FL_OK) return rc;
  const int bt = cfg->block_tokens;
  std::vector<int32_t> path, chain;
  std::vector<char> resident;
  for (int step = 0; step < n_events; ++step) {
    const double now = cfg->t0 + cfg->dt * (double)step;
    const int32_t* tok = tokens + event_indptr[step];
    const int n_tok = event_indptr[step + 1] - event_indptr[step];
    if (n_tok < 0) return FL_EINVAL;
    path.resize((size_t)n_tok / bt + 1);
    int32_t ln = -1;
    int n_path = 0, matched = 0;
    rc = fl_tree_match(r.tree, event_lora[step], tok, n_tok, now, &ln, path.data(), (int)path.size(), &n_path, &matched);
    if (rc != FL_OK) return rc;
    chain.assign(1, ln);
    chain.insert(chain.end(), path.begin(), path.begin() + n_path);
    if ((rc = r.take_stats()) != FL_OK) return rc;
    resident.resize(chain.size());
    for (size_t k = 0; k < chain.size(); ++k) resident[k] = r.stats[chain[k]].in_hbm != 0;
    if (resident[0]) {
      int usable = 0;
      while (usable < n_path && resident[1 + usable]) ++usable;
      r.res.hit_blocks += (uint64_t)usable;
    } else {
      r.res.lora_cold += 1;
    }
    r.res.asked_blocks += (uint64_t)(n_tok / bt);
    for (size_t k = 0; k < chain.size(); ++k) {        // what the query needs comes in, root first
      if (resident[k]) continue;
      const uint32_t nb = r.stats[chain[k]].n_blocks;
      const int kind = r.stats[chain[k]].kind;
      if ((rc = r.make_room(nb, kind, chain, now)) != FL_OK) return rc;
      if ((rc = r.take_stats()) != FL_OK) return rc;
      if ((rc = r.move(chain[k], 1)) != FL_OK) return rc;
    }
    const int n_new = n_tok / bt - n_path;
    if (n_new > 0) {
      if ((rc = r.make_room((uint32_t)n_new, FL_NODE_KV, chain, now)) != FL_OK) return rc;
      rc = fl_tree_insert(r.tree, chain.back(), tok + matched, n_new, r.fresh(1, (uint32_t)n_new), now, nullptr);
      if (rc != FL_OK) return rc;
      r.used += (uint32_t)n_new;
      r.part[FL_NODE_KV] += (uint32_t)n_new;
    }
    if (step % cfg->tick_every == cfg->tick_every - 1) {
      if (cfg->variant != FL_REPLAY_STATIC) {
        if ((rc = r.take_stats()) != FL_OK) return rc;
        int n_order = 0, direction = 0;
        rc = r.decide(now, r.used, cfg->capacity, r.policy(), cfg->upper, cfg->lower, &n_order, &direction);
        if (rc != FL_OK) return rc;
        for (int k = 0; k < n_order; ++k)
          if ((rc = r.move(r.order[k], direction == 1 ? 1 : 0)) != FL_OK) return rc;
      }
      uint32_t bad = 0, total = 0;
      if ((rc = fl_tree_invalid(r.tree, &bad, &total)) != FL_OK) return rc;
      if (r.res.n_samples < cap_samples) invalid_samples[r.res.n_samples] = total ? (double)bad / (double)total : 0.0;
      r.res.n_samples += 1;
    }
  }
  r.res.used_blocks = r.used;
  r.res.n_nodes = (uint64_t)fl_tree_size(r.tree);
  *out = r.res;
  return FL_OK;
}
