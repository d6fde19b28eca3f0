// Block-rate selection ("Heterogeneous Block-Rate Optimization"): one hybrid rate per transformer
// block, minimal summed error under a summed-cost budget - a multiple-choice knapsack problem.
//
// Host code only.  Exact solver: the blocks are taken in order and the set of non-dominated partial
// assignments (cost, error) is carried along; a partial assignment is dropped when another one is no
// more expensive and no worse, or when it cannot be completed within the budget even with the cheapest
// rates of the remaining blocks.  Sums are taken in block order in double precision, so a cost that
// meets the budget exactly is treated the same way by any caller that adds in that order.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <new>
#include <vector>

#include "as_hybrid_attn.h"

namespace {

struct State {
  double cost, err;
  int32_t parent;   // index into the previous block's frontier
  int32_t rate;
};

constexpr size_t kMaxFrontier = size_t(1) << 22;   // states kept per block before giving up

}  // namespace

as_status_t as_select_block_rates(int32_t n_blocks, int32_t n_rates, const double* cost, const double* err,
                                  double budget, int32_t* choice_out, double* total_cost_out,
                                  double* total_err_out) {
  if (n_blocks <= 0 || n_rates <= 0 || !cost || !err || !choice_out) return AS_ERR_INVALID_ARG;
  if (std::isnan(budget)) return AS_ERR_INVALID_ARG;
  for (int64_t i = 0; i < (int64_t)n_blocks * n_rates; ++i)
    if (!std::isfinite(cost[i]) || !std::isfinite(err[i]) || cost[i] < 0.0) return AS_ERR_INVALID_ARG;
  try {
    // cheapest completion of blocks i.. (a lower bound; it is only used to drop hopeless states early,
    // with a margin for its different summation order)
    std::vector<double> tail_min((size_t)n_blocks + 1, 0.0);
    for (int i = n_blocks - 1; i >= 0; --i) {
      const double* c = cost + (size_t)i * n_rates;
      tail_min[i] = tail_min[i + 1] + *std::min_element(c, c + n_rates);
    }
    std::vector<std::vector<State>> frontier((size_t)n_blocks);
    std::vector<State> cand;
    for (int i = 0; i < n_blocks; ++i) {
      const double* c = cost + (size_t)i * n_rates;
      const double* e = err + (size_t)i * n_rates;
      cand.clear();
      const size_t n_prev = i == 0 ? 1 : frontier[i - 1].size();
      for (size_t s = 0; s < n_prev; ++s) {
        const double c0 = i == 0 ? 0.0 : frontier[i - 1][s].cost;
        const double e0 = i == 0 ? 0.0 : frontier[i - 1][s].err;
        for (int r = 0; r < n_rates; ++r) {
          const double cc = c0 + c[r];
          if (cc > budget) continue;
          const double slack = 1e-9 * (std::fabs(budget) + tail_min[i + 1]);
          if (cc + tail_min[i + 1] > budget + slack) continue;
          cand.push_back(State{cc, e0 + e[r], (int32_t)s, r});
        }
      }
      if (cand.empty()) return AS_ERR_INFEASIBLE;
      std::sort(cand.begin(), cand.end(), [](const State& a, const State& b) {
        return a.cost < b.cost || (a.cost == b.cost && a.err < b.err);
      });
      std::vector<State>& f = frontier[i];
      double best_err = INFINITY;
      for (const State& s : cand)
        if (s.err < best_err) { f.push_back(s); best_err = s.err; }   // strictly better than everything cheaper
      if (f.size() > kMaxFrontier) return AS_ERR_UNSUPPORTED;
    }
    // the last frontier is sorted by cost with strictly falling error: its last state is the optimum;
    // the sums of the last block's states are complete, so every one of them is within the budget
    const std::vector<State>& last = frontier[n_blocks - 1];
    int32_t s = (int32_t)last.size() - 1;
    if (total_cost_out) *total_cost_out = last[s].cost;
    if (total_err_out) *total_err_out = last[s].err;
    for (int i = n_blocks - 1; i >= 0; --i) {
      choice_out[i] = frontier[i][s].rate;
      s = frontier[i][s].parent;
    }
    return AS_OK;
  } catch (const std::bad_alloc&) {
    return AS_ERR_ALLOC;
  }
}
