// Performance-driven cache swapper (Section 5): expected adapter demand (Eq. 3), the cost model that
// ranks LoRA and KV nodes by the benefit of keeping them in HBM (Eq. 4, Eq. 5, Eq. 6), and the greedy
// selection of the monitor tick (Section 5.3).  Host code only: its output is the ordered node list
// whose blocks then go to fl_swap_out / fl_swap_in.
#include <math.h>
#include <algorithm>
#include <numeric>
#include <vector>
#include "fastpool.h"

extern "C" {

int fl_expected_lora_demand(const double* prob, int n, int batch_size, double* low_lora) {
  if (!prob || !low_lora || n < 0 || batch_size < 0) return FL_EINVAL;
  double sum = 0.0;
  for (int i = 0; i < n; ++i) {
    if (!(prob[i] >= 0.0 && prob[i] <= 1.0)) return FL_EINVAL;
    sum += 1.0 - pow(1.0 - prob[i], (double)batch_size);     // Eq. 3: fe_i
  }
  *low_lora = sum;
  return FL_OK;
}

int fl_swap_eval(const fl_node_stat* nodes, int n, const fl_swap_params* prm, double* eval) {
  if (!nodes || !prm || !eval || n < 0) return FL_EINVAL;
  if (!(prm->link_bytes_per_s > 0.0) || !(prm->total_visits > 0.0) || prm->now_lora < 0 || prm->block_bytes == 0) return FL_EINVAL;
  // Eq. 4: one coefficient for every LoRA node; KV nodes take 1
  const double lora_eval = prm->now_lora > 0 ? std::max(1.0, prm->low_lora / (double)prm->now_lora)
                                             : (prm->low_lora > 0.0 ? INFINITY : 1.0);
  for (int i = 0; i < n; ++i) {
    const fl_node_stat& nd = nodes[i];
    const double cost = (double)nd.n_blocks * (double)prm->block_bytes / prm->link_bytes_per_s;   // transfer time, seconds
    const double prob = nd.visits / prm->total_visits;
    const double t = prm->now_s - nd.last_use_s;
    const double retain = cost * prob * (1.0 - 1.0 / (1.0 + exp(-t)));                              // Eq. 5
    eval[i] = (nd.kind == FL_NODE_LORA ? lora_eval : 1.0) * retain;                                 // Eq. 6
  }
  return FL_OK;
}

int fl_swapper_decide(const fl_node_stat* nodes, int n, const fl_swap_params* prm, uint32_t blocks_used,
                      uint32_t blocks_total, int32_t* order, int* n_order, int* direction) {
  if (blocks_used > blocks_total) return FL_EINVAL;
  return fl_swapper_decide_policy(nodes, n, prm, blocks_used, blocks_total, 0u, order, n_order, direction);
}

int fl_swapper_decide_policy(const fl_node_stat* nodes, int n, const fl_swap_params* prm, uint32_t blocks_used,
                             uint32_t blocks_total, uint32_t policy, int32_t* order, int* n_order, int* direction) {
  if (!nodes || !prm || !order || !n_order || !direction || n < 0 || blocks_total == 0) return FL_EINVAL;
  if (policy & ~(uint32_t)(FL_POLICY_LRU | FL_POLICY_NO_LORA_REWARD | FL_POLICY_ONLY_LORA | FL_POLICY_ONLY_KV)) return FL_EINVAL;
  if ((policy & FL_POLICY_ONLY_LORA) && (policy & FL_POLICY_ONLY_KV)) return FL_EINVAL;
  if (!(prm->lower >= 0.0 && prm->lower <= prm->upper && prm->upper <= 1.0)) return FL_EINVAL;
  *n_order = 0;
  *direction = 0;
  const double usage = (double)blocks_used / (double)blocks_total;
  const bool out = usage > prm->upper, in = usage < prm->lower;
  if (!out && !in) return FL_OK;                       // between the thresholds: nothing moves
  std::vector<double> eval((size_t)n);
  if (policy & FL_POLICY_LRU) {
    // the ablation without the cost model: the node used longest ago leaves first, the one used last enters first
    for (int i = 0; i < n; ++i) eval[i] = nodes[i].last_use_s;
  } else {
    fl_swap_params q = *prm;
    if (policy & FL_POLICY_NO_LORA_REWARD) q.low_lora = 0.0;     // Eq. 4 coefficient = 1 for every node
    int rc = fl_swap_eval(nodes, n, &q, eval.data());
    if (rc != FL_OK) return rc;
  }
  std::vector<int32_t> cand;
  for (int i = 0; i < n; ++i)
    if (nodes[i].candidate && (nodes[i].in_hbm != 0) == out &&
        !((policy & FL_POLICY_ONLY_LORA) && nodes[i].kind != FL_NODE_LORA) &&
        !((policy & FL_POLICY_ONLY_KV) && nodes[i].kind != FL_NODE_KV))
      cand.push_back(i);
  // swap-out: ascending benefit; swap-in: descending benefit; equal values keep the lower index first
  std::stable_sort(cand.begin(), cand.end(), [&](int32_t a, int32_t b) { return out ? eval[a] < eval[b] : eval[a] > eval[b]; });
  const double upper_blocks = prm->upper * (double)blocks_total, lower_blocks = prm->lower * (double)blocks_total;
  double used = (double)blocks_used;
  int k = 0;
  for (int32_t i : cand) {
    if (out) {
      if (used <= upper_blocks) break;                 // balanced again
      used -= (double)nodes[i].n_blocks;
      order[k++] = i;
    } else {
      if (used >= lower_blocks) break;
      if (used + (double)nodes[i].n_blocks > upper_blocks) continue;   // would make the pool busy: skip this node
      used += (double)nodes[i].n_blocks;
      order[k++] = i;
    }
  }
  *n_order = k;
  *direction = out ? -1 : 1;
  return FL_OK;
}

}  // extern "C"
