// Barrier step: per-layer budgets from the layers' entropies (Eq. 7, Appendix A.3; Sec. 4.4 for
// the recent : important split).  One thread block; the arithmetic is serial fp64 in thread 0
// because L is a few dozen and the result must not depend on a reduction order.
#pragma once

#include "meda_common.cuh"

namespace meda {

__global__ void allocate_budgets_kernel(const float* __restrict__ entropy, int32_t* __restrict__ budgets,
                                        int n_layers, long long total, int lo, int hi, int beta_r, int beta_i,
                                        int alloc_mode, int* status) {
  __shared__ double w[kMaxLayers];
  __shared__ double q[kMaxLayers];
  __shared__ signed char state[kMaxLayers];   // -1 clamped at lo, 0 free, +1 clamped at hi
  __shared__ unsigned char bumped[kMaxLayers];
  if (threadIdx.x != 0) return;
  const int L = n_layers;
  if (total < (long long)L * lo || total > (long long)L * hi) {
    set_status(status, MEDA_ERR_BUDGET_INFEASIBLE);
    return;
  }
  // softmax over layers (uniform in the ablation mode)
  double emax = -1e300;
  for (int l = 0; l < L; ++l) emax = fmax(emax, (double)entropy[l]);
  double sum = 0.0;
  for (int l = 0; l < L; ++l) {
    w[l] = alloc_mode == 1 ? 1.0 : exp((double)entropy[l] - emax);
    sum += w[l];
  }
  for (int l = 0; l < L; ++l) { w[l] /= sum; state[l] = 0; bumped[l] = 0; }

  // q_l = clip(lambda w_l, lo, hi) with sum q_l = total: clamp the side with the larger violation
  // until none is left; the layers on the other side can only move further inside.
  if (total == (long long)L * lo) {
    for (int l = 0; l < L; ++l) state[l] = -1;
  } else if (total == (long long)L * hi) {
    for (int l = 0; l < L; ++l) state[l] = 1;
  }
  for (int it = 0; it <= L; ++it) {
    long long clamped = 0;
    double w_free = 0.0;
    int n_free = 0;
    for (int l = 0; l < L; ++l) {
      if (state[l] == 0) { w_free += w[l]; ++n_free; }
      else clamped += state[l] < 0 ? lo : hi;
    }
    if (n_free == 0) break;
    double over = 0.0, under = 0.0;
    for (int l = 0; l < L; ++l) {
      if (state[l] != 0) continue;
      q[l] = (double)(total - clamped) * w[l] / w_free;
      if (q[l] > (double)hi) over += q[l] - hi;
      if (q[l] < (double)lo) under += lo - q[l];
    }
    if (over == 0.0 && under == 0.0) break;
    if (over >= under) {
      for (int l = 0; l < L; ++l) if (state[l] == 0 && q[l] > (double)hi) state[l] = 1;
    } else {
      for (int l = 0; l < L; ++l) if (state[l] == 0 && q[l] < (double)lo) state[l] = -1;
    }
  }
  long long assigned = 0;
  for (int l = 0; l < L; ++l) {
    long long s = state[l] < 0 ? lo : state[l] > 0 ? hi : (long long)floor(q[l]);
    budgets[l * 3] = (int32_t)s;
    assigned += s;
  }
  // largest remainder among the free layers, ties to the lowest layer
  for (long long missing = total - assigned; missing > 0; --missing) {
    int best = -1;
    double best_frac = -1.0;
    for (int l = 0; l < L; ++l) {
      if (state[l] != 0 || bumped[l]) continue;
      double frac = q[l] - floor(q[l]);
      if (frac > best_frac) { best_frac = frac; best = l; }
    }
    if (best < 0) { set_status(status, MEDA_ERR_BUDGET_INFEASIBLE); break; }
    bumped[best] = 1;
    budgets[best * 3] += 1;
  }
  for (int l = 0; l < L; ++l) {
    int32_t s = budgets[l * 3];
    int32_t m = (int32_t)(((long long)s * beta_r) / (beta_r + beta_i));
    budgets[l * 3 + 1] = m;
    budgets[l * 3 + 2] = s - m;
  }
}

}  // namespace meda
