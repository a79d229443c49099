// Host-side planning steps that feed the per-layer kernels: the per-chunk token budgets of
// Section 4.3 ("Structure-Aware Budget Allocation") and the span selection of Section 4.4
// ("Span selection under budget"), whose covered tokens become the protected set (prior = 1)
// that the selection kernel keeps first.  Plain C++ on host arrays: the inputs are a few
// numbers per chunk or span, produced on the host by the program-analysis front end.
#include <math.h>

#include <algorithm>
#include <vector>

#include "codecomp.h"

extern "C" {

int cc_plan_budgets(const double* sigma, const int32_t* lens, int32_t num_chunks,
                    const cc_budget_params* p, int32_t* budgets, double* multipliers) {
  if (num_chunks < 0 || !p || (num_chunks > 0 && (!sigma || !lens || !budgets)))
    return CC_ERR_INVALID_ARG;
  if (!(p->r >= 0.0) || !(p->r_max >= 0.0) || !(p->m_max >= p->m_min) || !(p->eps > 0.0))
    return CC_ERR_INVALID_ARG;
  if (num_chunks == 0) return CC_OK;
  double lo = sigma[0], hi = sigma[0];
  for (int i = 0; i < num_chunks; ++i) {
    if (sigma[i] != sigma[i] || lens[i] < 0) return CC_ERR_INVALID_ARG;
    lo = std::min(lo, sigma[i]);
    hi = std::max(hi, sigma[i]);
  }
  for (int i = 0; i < num_chunks; ++i) {
    double st = hi == lo ? 0.5 : (sigma[i] - lo) / std::max(p->eps, hi - lo);
    st = std::min(1.0, std::max(0.0, st));
    const double m = p->m_min + (p->m_max - p->m_min) * st;
    // the same 1e-9 nudge as for B^span: products that are integers on paper stay integers
    const double b = floor((double)lens[i] * std::min(p->r_max, p->r * m) + 1e-9);
    budgets[i] = (int32_t)std::min(b, (double)lens[i]);
    if (multipliers) multipliers[i] = m;
  }
  return CC_OK;
}

int cc_select_spans(const int32_t* starts, const int32_t* ends, const float* scores,
                    const uint8_t* is_protected, int32_t num_spans, int32_t n, int32_t budget,
                    double span_ratio, int32_t span_min, float* prior_mask, int32_t* taken,
                    int32_t* num_taken) {
  if (num_spans < 0 || n < 0 || budget < 0 || !prior_mask ||
      (num_spans > 0 && (!starts || !ends || !scores || !is_protected)))
    return CC_ERR_INVALID_ARG;
  for (int i = 0; i < num_spans; ++i)
    if (starts[i] < 0 || ends[i] < starts[i] || ends[i] > n || scores[i] != scores[i])
      return CC_ERR_INVALID_ARG;
  long long cap = budget;
  if (span_ratio > 0.0) {
    const long long want = (long long)floor(span_ratio * (double)budget + 1e-9);
    cap = std::min<long long>(budget, std::max<long long>(span_min, want));
  }
  for (int j = 0; j < n; ++j) prior_mask[j] = 0.0f;
  long long covered = 0;
  int count = 0;
  auto take = [&](int i) {
    for (int j = starts[i]; j < ends[i]; ++j) {
      if (prior_mask[j] == 0.0f) ++covered;
      prior_mask[j] = 1.0f;
    }
    if (taken) taken[count] = i;
    ++count;
  };
  std::vector<int> rest;
  for (int i = 0; i < num_spans; ++i) {
    if (is_protected[i]) take(i); else rest.push_back(i);
  }
  std::stable_sort(rest.begin(), rest.end(), [&](int a, int b) {
    if (scores[a] != scores[b]) return scores[a] > scores[b];
    if (starts[a] != starts[b]) return starts[a] < starts[b];
    return a < b;
  });
  for (int i : rest) {
    if (covered >= cap) break;
    take(i);
  }
  if (num_taken) *num_taken = count;
  return CC_OK;
}

}  // extern "C"
