// Phase B, selection (Eq. 9-10): per (layer, KV head) keep the last M tokens and the N best of the
// others, ranked text first (Eq. 9's boost, as an extra key bit), then by accumulated score, then
// by lowest index.  Exact radix select on the 33-bit key followed by an ordered compaction, so the
// result does not depend on thread scheduling.  One thread block per KV head.
#pragma once

#include "meda_common.cuh"

namespace meda {

constexpr int kSelThreads = 1024;

// Monotone map of (modality, score) to an unsigned key: larger key = ranked earlier.
__device__ __forceinline__ unsigned long long select_key(float score, uint8_t modality) {
  unsigned int b = __float_as_uint(score);
  b = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  return ((unsigned long long)(modality == MEDA_TEXT ? 1u : 0u) << 32) | b;
}

// Exclusive prefix count of `flag` over the block (thread order) and the block total.
__device__ __forceinline__ int block_exclusive_count(bool flag, int* warp_counts, int& total) {
  const int lane = threadIdx.x % 32, warp = threadIdx.x / 32;
  unsigned int ballot = __ballot_sync(0xffffffffu, flag);
  int in_warp = __popc(ballot & ((1u << lane) - 1u));
  __syncthreads();                      // previous users of warp_counts are done
  if (lane == 0) warp_counts[warp] = __popc(ballot);
  __syncthreads();
  int before = 0, all = 0;
  for (int x = 0; x < kSelThreads / 32; ++x) {
    int c = warp_counts[x];
    before += (x < warp) ? c : 0;
    all += c;
  }
  total = all;
  return before + in_warp;
}

__global__ void __launch_bounds__(kSelThreads)
select_topk_kernel(const float* __restrict__ scores, const uint8_t* __restrict__ modality,
                   const int32_t* __restrict__ budget_row, int32_t* __restrict__ idx_conserved,
                   int32_t* __restrict__ idx_less, int n, int cap, int* status) {
  __shared__ unsigned int hist[256];
  __shared__ int warp_counts[kSelThreads / 32];
  __shared__ unsigned long long s_prefix, s_mask;
  __shared__ int s_remaining;

  const int g = blockIdx.x;
  const int S = budget_row[0], M = budget_row[1], N = budget_row[2];
  const int n_cand = n - M;
  if (S < 0 || M < 0 || N < 0 || S != M + N || M > n || N > n_cand || S > cap) {
    if (threadIdx.x == 0) set_status(status, S > cap ? MEDA_ERR_WORKSPACE : MEDA_ERR_BUDGET_INFEASIBLE);
    return;
  }
  const float* sc = scores + (size_t)g * n;
  int32_t* out_c = idx_conserved + (size_t)g * cap;
  int32_t* out_l = idx_less + (size_t)g * n;

  // ---- the N-th largest key among the candidates, most significant digit first
  if (threadIdx.x == 0) { s_prefix = 0ull; s_mask = 0ull; s_remaining = N; }
  __syncthreads();
  if (N > 0) {
    for (int pass = 0; pass < 5; ++pass) {
      const int shift = pass == 0 ? 32 : 32 - 8 * pass;
      const unsigned int bins = pass == 0 ? 2u : 256u;
      for (int b = threadIdx.x; b < 256; b += kSelThreads) hist[b] = 0u;
      __syncthreads();
      const unsigned long long prefix = s_prefix, mask = s_mask;
      for (int j = threadIdx.x; j < n_cand; j += kSelThreads) {
        unsigned long long key = select_key(sc[j], modality[j]);
        if ((key & mask) == prefix) atomicAdd(&hist[(unsigned int)(key >> shift) & (bins - 1u)], 1u);
      }
      __syncthreads();
      if (threadIdx.x == 0) {
        int remaining = s_remaining, cum = 0;
        int digit = 0;
        for (int b = (int)bins - 1; b >= 0; --b) {
          int c = (int)hist[b];
          if (cum + c >= remaining) { digit = b; break; }
          cum += c;
        }
        s_remaining = remaining - cum;
        s_prefix = prefix | ((unsigned long long)digit << shift);
        s_mask = mask | ((unsigned long long)(bins - 1u) << shift);
      }
      __syncthreads();
    }
  }
  const unsigned long long threshold = s_prefix;
  const int take_equal = N > 0 ? s_remaining : 0;   // how many keys equal to the threshold are kept (lowest indices)

  // ---- ordered compaction in chunks of one block
  int kept_before = 0, equal_before = 0;
  for (int base = 0; base < n; base += kSelThreads) {
    const int j = base + threadIdx.x;
    bool greater = false, equal = false, recent = false;
    if (j < n_cand) {
      unsigned long long key = select_key(sc[j], modality[j]);
      greater = N > 0 && key > threshold;
      equal = N > 0 && key == threshold;
    } else if (j < n) {
      recent = true;
    }
    int equal_total, keep_total;
    int equal_rank = equal_before + block_exclusive_count(equal, warp_counts, equal_total);
    bool keep = greater || recent || (equal && equal_rank < take_equal);
    int pos = kept_before + block_exclusive_count(keep, warp_counts, keep_total);
    if (j < n) {
      if (keep) out_c[pos] = j;
      else out_l[j - pos] = j;
    }
    kept_before += keep_total;
    equal_before += equal_total;
  }
}

}  // namespace meda
