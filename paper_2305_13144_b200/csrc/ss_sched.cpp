// Host scheduler: length bins, sort-and-split, variable batch size, token caps.
// Follows Sec. 4.1 of the paper (sequence scheduling, FCR, VBS, binning) with the constants
// of Sec. 4.2 supplied through ss_sched_cfg.  Pure integer host code, no CUDA.
#include "ss_internal.h"

#include <algorithm>
#include <vector>

namespace ss {

// Length -> cell: clamp to [1, max_new], then round up to the next multiple of the cell.
int32_t length_bin(int32_t x, const ss_sched_cfg& c) {
  if (x < 1) x = 1;
  if (x > c.max_new_tokens) x = c.max_new_tokens;
  if (c.bin_size <= 1) return x;
  int32_t cells = (x + c.bin_size - 1) / c.bin_size;
  return cells * c.bin_size;
}

// Power of two nearest to budget / L in linear distance; the lower one wins a tie.
static int64_t nearest_pow2_ratio(int64_t budget, int64_t L) {
  int64_t below = 1;
  while ((below << 1) * L <= budget) below <<= 1;   // below <= budget/L < 2*below (or budget/L < 1)
  int64_t above = below << 1;
  int64_t d_lo = budget - below * L;                 // both distances scaled by L
  int64_t d_hi = above * L - budget;
  return d_lo <= d_hi ? below : above;
}

int32_t batch_allowance(int32_t L, const ss_sched_cfg& c) {
  if (!c.use_vbs || L >= c.vbs_len_threshold) return c.base_batch;
  int64_t b = nearest_pow2_ratio(c.vbs_token_budget, L);
  b = std::max<int64_t>(b, c.min_batch);
  b = std::min<int64_t>(b, c.max_batch);
  return (int32_t)b;
}

int validate_sched_cfg(const ss_sched_cfg* c) {
  if (!c) return SS_ERR_ARG;
  if (c->bin_size < 1 || c->base_batch < 1 || c->max_new_tokens < 1) return SS_ERR_ARG;
  if (c->use_vbs && (c->min_batch < 1 || c->max_batch < c->min_batch || c->vbs_token_budget < 1)) return SS_ERR_ARG;
  if (c->kv_budget_bytes < 0 || c->kv_bytes_per_token < 0) return SS_ERR_ARG;
  return SS_OK;
}

int plan_first_pass(const ss_sched_cfg& c, const int32_t* prompt_len, const int32_t* pred_len,
                    const int32_t* perm, int32_t n, std::vector<int32_t>& order,
                    std::vector<ss_batch_desc>& out) {
  order.assign(n, 0);
  out.clear();
  if (c.vanilla) {
    std::vector<uint8_t> seen(n, 0);
    for (int32_t i = 0; i < n; ++i) {
      int32_t q = perm ? perm[i] : i;
      if (q < 0 || q >= n || seen[q]) return SS_ERR_ARG;
      seen[q] = 1;
      order[i] = q;
    }
    for (int32_t i = 0; i < n; i += c.base_batch)
      out.push_back({i, std::min(c.base_batch, n - i), c.max_new_tokens, 0});
    return SS_OK;
  }

  // Stable ascending order by cell.
  std::vector<int32_t> cell(n);
  for (int32_t i = 0; i < n; ++i) cell[i] = length_bin(pred_len[i], c);
  for (int32_t i = 0; i < n; ++i) order[i] = i;
  std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return cell[a] < cell[b]; });

  int32_t start = 0;
  while (start < n) {
    int32_t rows = 0, longest_prompt = 0, largest_cell = 0;
    for (;;) {
      if (start + rows >= n) break;
      const int32_t q = order[start + rows];
      const int32_t q_cap = std::min(cell[q], c.max_new_tokens);
      if (rows + 1 > batch_allowance(cell[q], c)) break;
      const int32_t lp = std::max(longest_prompt, prompt_len[q]);
      if (c.kv_budget_bytes > 0 && rows >= 1) {
        const int64_t need = (int64_t)(rows + 1) * ((int64_t)lp + q_cap) * c.kv_bytes_per_token;
        if (need > c.kv_budget_bytes) break;
      }
      ++rows;
      longest_prompt = lp;
      largest_cell = std::max(largest_cell, cell[q]);
    }
    const int32_t cap = c.use_fcr ? std::min(largest_cell, c.max_new_tokens) : c.max_new_tokens;
    out.push_back({start, rows, cap, 0});
    start += rows;
  }
  return SS_OK;
}

}  // namespace ss

// Replica dispatch (Sec. 1: micro-batches of different perceived lengths can be handed to different GPUs).
// Estimated cost of a batch = its steps (the cap) times the bytes one decode step moves: the weights once plus, per
// row, the cached keys and values at the batch's mean prompt length plus half the cap.  Batches are taken in order
// of decreasing cost (equal costs: lower index first); each goes to the replica whose total is smallest so far
// (equal totals: lowest replica).
extern "C" int ss_deal_batches(const ss_batch_desc* batches, int32_t n_batches, const int32_t* order,
                               const int32_t* prompt_len, int64_t weight_bytes, int64_t kv_bytes_per_token,
                               int32_t n_gpus, int32_t* gpu_of) {
  if (n_batches < 0 || n_gpus < 1 || weight_bytes < 0 || kv_bytes_per_token < 0) return SS_ERR_ARG;
  if (n_batches > 0 && (!batches || !order || !prompt_len || !gpu_of)) return SS_ERR_ARG;
  std::vector<int64_t> cost(n_batches);
  for (int32_t i = 0; i < n_batches; ++i) {
    const ss_batch_desc& b = batches[i];
    if (b.n_rows < 1 || b.first_row < 0 || b.cap < 1) return SS_ERR_ARG;
    int64_t prompt_sum = 0;
    for (int32_t r = 0; r < b.n_rows; ++r) prompt_sum += prompt_len[order[b.first_row + r]];
    // rows * (mean prompt + cap / 2) cached tokens, kept in integers: (2 * prompt_sum + rows * cap) / 2
    const int64_t tokens2 = 2 * prompt_sum + (int64_t)b.n_rows * b.cap;
    cost[i] = (int64_t)b.cap * (weight_bytes + tokens2 * kv_bytes_per_token / 2);
  }
  std::vector<int32_t> by_cost(n_batches);
  for (int32_t i = 0; i < n_batches; ++i) by_cost[i] = i;
  std::stable_sort(by_cost.begin(), by_cost.end(), [&](int32_t a, int32_t b) { return cost[a] > cost[b]; });
  std::vector<int64_t> load(n_gpus, 0);
  for (int32_t i : by_cost) {
    int32_t best = 0;
    for (int32_t g = 1; g < n_gpus; ++g)
      if (load[g] < load[best]) best = g;
    gpu_of[i] = best;
    load[best] += cost[i];
  }
  return SS_OK;
}

extern "C" int ss_schedule(const ss_sched_cfg* cfg, const int32_t* prompt_len, const int32_t* pred_len,
                           const int32_t* perm, int32_t n, int32_t* order, ss_batch_desc* batches,
                           int32_t batch_cap, int32_t* n_batches) {
  int rc = ss::validate_sched_cfg(cfg);
  if (rc != SS_OK) return rc;
  if (n < 0 || !n_batches || (n > 0 && (!prompt_len || !pred_len || !order))) return SS_ERR_ARG;
  std::vector<int32_t> ord;
  std::vector<ss_batch_desc> plan;
  rc = ss::plan_first_pass(*cfg, prompt_len, pred_len, perm, n, ord, plan);
  if (rc != SS_OK) return rc;
  *n_batches = (int32_t)plan.size();
  if ((int32_t)plan.size() > batch_cap || (plan.size() && !batches)) return SS_ERR_CAPACITY;
  std::copy(ord.begin(), ord.end(), order);
  std::copy(plan.begin(), plan.end(), batches);
  return SS_OK;
}
