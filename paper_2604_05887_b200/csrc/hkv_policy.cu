// Top-down budget allocation (paper Section 3.2): host arithmetic that turns a total token budget,
// the head classification and the text-centric sparsity scores into the per-head budgets that
// hkv_plan / hkv_compress take.  No device work.
#include <cmath>
#include <cstdint>

#include "hkv.h"

extern "C" hkv_status hkv_allocate_budgets(int32_t n_heads, const uint8_t* head_type, const double* scores,
                                           int64_t total_budget, double r, double alpha, uint32_t flags,
                                           int32_t* budgets_out) {
  if (n_heads < 1 || !head_type || !budgets_out) return HKV_ERR_INVALID_ARG;
  if (flags & ~HKV_BUDGET_PAD_POW2) return HKV_ERR_INVALID_ARG;
  if (total_budget < n_heads || !(r > 0.0) || !(alpha >= 0.0 && alpha <= 1.0)) return HKV_ERR_BUDGET;
  int64_t n_stat = 0, n_dyna = 0;
  double score_sum = 0.0;
  for (int32_t i = 0; i < n_heads; ++i) {
    if (head_type[i] > 1) return HKV_ERR_INVALID_ARG;
    if (head_type[i] == 0) {
      ++n_stat;
      if (scores) {
        if (!(scores[i] >= 0.0) || std::isinf(scores[i])) return HKV_ERR_INVALID_ARG;
        score_sum += scores[i];   // in head order
      }
    } else {
      ++n_dyna;
    }
  }
  // head-type level: average per-head budget, share coefficient r for the dynamic heads
  const double b_total = static_cast<double>(total_budget);
  const double b_bar = b_total / static_cast<double>(n_stat + n_dyna);
  int64_t b_dyna = 0;
  if (n_dyna > 0) {
    if (r > b_total / (b_bar * static_cast<double>(n_dyna))) return HKV_ERR_BUDGET;   // would exceed the total
    b_dyna = static_cast<int64_t>(std::ceil(r * b_bar * static_cast<double>(n_dyna)));
    if (b_dyna > total_budget) b_dyna = total_budget;
  }
  const int64_t b_stat = total_budget - b_dyna;
  if (n_stat > 0 && b_stat < n_stat) return HKV_ERR_BUDGET;   // not even one token per static head
  // individual heads
  int64_t dyn_each = 0;
  if (n_dyna > 0) {
    dyn_each = (b_dyna + n_dyna - 1) / n_dyna;   // uniform share, rounded up
    if (dyn_each < 1) dyn_each = 1;
    if (flags & HKV_BUDGET_PAD_POW2) {
      int64_t p = 1;
      while (p < dyn_each) p <<= 1;
      dyn_each = p;
    }
  }
  const double bs = static_cast<double>(b_stat);
  const double base = n_stat > 0 ? alpha * bs / static_cast<double>(n_stat) : 0.0;
  for (int32_t i = 0; i < n_heads; ++i) {
    int64_t b;
    if (head_type[i] == 0) {
      // L1-normalised score over all static heads (uniform when no scores are given or all are zero)
      const double s_norm = (scores && score_sum > 0.0) ? scores[i] / score_sum : 1.0 / static_cast<double>(n_stat);
      b = static_cast<int64_t>(std::ceil(base + (1.0 - alpha) * bs * s_norm));
      if (b < 1) b = 1;
    } else {
      b = dyn_each;
    }
    if (b > 0x7FFFFFFF) return HKV_ERR_UNSUPPORTED;
    budgets_out[i] = static_cast<int32_t>(b);
  }
  return HKV_OK;
}
