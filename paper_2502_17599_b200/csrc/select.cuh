// Phase B, selection (Eq. 9-10): per (layer, KV head) keep the last M tokens and the N best of the
// others, ranked text first (Eq. 9's boost, as an extra key bit), then by accumulated score, then
// by lowest index.  Exact radix select on the 33-bit key followed by an ordered compaction, so the
// result does not depend on thread scheduling.  One thread block per KV head.
#pragma once

#include <cooperative_groups.h>

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


// ---------------------------------------------------------------------------------------------
// The same selection with one thread-block cluster per KV head, for sequences whose keys fit the
// cluster's shared memory: the C blocks of a cluster each stage one C-th of the head's scores
// as 32-bit sort keys, so the radix passes read shared memory only; digit histograms are combined
// across the cluster through distributed shared memory, and the hardware cluster barrier is the
// only synchronisation between blocks.  Same ranking, same tie-break, same outputs as the
// single-block kernel above.  C is 8 for long prompts and smaller (4, 2, 1) when an eighth of the
// prompt would be less than one compaction step per block or when 8 blocks per head would need more
// than one wave of the GPU (see select_cluster_size).
// ---------------------------------------------------------------------------------------------
constexpr int kSelMaxClusterSize = 8;
constexpr int kSelBins = 2048;                    // 11-bit digits: 11 + 11 + 10 bits of the score key
constexpr int kSelPerThread = 16;                 // consecutive tokens per thread and round of the compaction
constexpr int kSelBlockStep = 4096;               // a block's share of the tokens is a multiple of this
constexpr int kSelMaxRounds = 4;                  // compaction rounds per block: 64K tokens, more than shared memory holds

struct SelectClusterSmem {
  int chunk;          // tokens per block
  int keys_off, hist_off, total_off, misc_off, total;
};
__host__ __device__ inline SelectClusterSmem select_cluster_smem(int n, int cluster_size) {
  SelectClusterSmem L;
  const int step = kSelBlockStep;
  L.chunk = ((n + cluster_size - 1) / cluster_size + step - 1) / step * step;
  int off = 0;
  L.keys_off = off;  off += L.chunk * 4;
  L.hist_off = off;  off += 2 * kSelBins * 4;     // two histograms, used by alternate radix passes
  L.total_off = off;
  L.misc_off = off;  off += 256;
  L.total = off;
  return L;
}

// Exclusive prefix of `v` over the block in thread order, and the block total.  `scratch` holds 33 ints.
__device__ __forceinline__ int block_exclusive_sum(int v, int* scratch, int& total) {
  const int lane = threadIdx.x % 32, warp = threadIdx.x / 32;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  __syncthreads();                      // previous users of scratch are done
  if (lane == 31) scratch[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = scratch[lane], wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int y = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += y;
    }
    scratch[lane] = wi - w;
    if (lane == 31) scratch[32] = wi;
  }
  __syncthreads();
  total = scratch[32];
  return scratch[warp] + incl - v;
}

// Blocks per head: the largest of 8, 4, 2, 1 that gives every block at least one compaction step of tokens
// and keeps all heads' clusters within one wave of `sm_count` blocks, as long as the keys of a block still
// fit `smem_limit` bytes; 0 if even eight blocks per head do not fit (the single-block kernel then runs).
inline int select_cluster_size(int n, int n_heads, int sm_count, int smem_limit) {
  if (select_cluster_smem(n, kSelMaxClusterSize).total > smem_limit) return 0;
  int c = kSelMaxClusterSize;
  while (c > 1 && ((n + c - 1) / c < kSelBlockStep || n_heads * c > sm_count) &&
         select_cluster_smem(n, c / 2).total <= smem_limit)
    c /= 2;
  return c;
}

template <int kSelClusterSize>
__global__ void __cluster_dims__(kSelClusterSize, 1, 1) __launch_bounds__(kSelThreads, 1)
select_topk_cluster_kernel(const float* __restrict__ scores, const uint8_t* __restrict__ modality,
                           const int32_t* __restrict__ budget_row, int32_t* __restrict__ idx_conserved,
                           int32_t* __restrict__ idx_less, int n, int cap, int* status) {
  namespace cg = cooperative_groups;
  extern __shared__ __align__(16) unsigned char sel_smem[];
  cg::cluster_group cluster = cg::this_cluster();
  const SelectClusterSmem L = select_cluster_smem(n, kSelClusterSize);
  unsigned int* keys = reinterpret_cast<unsigned int*>(sel_smem + L.keys_off);
  unsigned int* hist = reinterpret_cast<unsigned int*>(sel_smem + L.hist_off);
  int* misc = reinterpret_cast<int*>(sel_smem + L.misc_off);
  // misc: [0..32] scan scratch, [40] text candidates of this block, [41] kept for sure, [42] equal to the
  // threshold, [44] digit, [45] remaining
  const int rank = (int)cluster.block_rank();
  const int g = blockIdx.x / kSelClusterSize;
  const int S = budget_row[0], M = budget_row[1], N = budget_row[2];
  const int n_cand = n - M;
  if (S < 0 || M < 0 || N < 0 || S != M + N || M > n || N > n_cand || S > cap) {     // uniform over the cluster
    if (threadIdx.x == 0 && rank == 0) set_status(status, S > cap ? MEDA_ERR_WORKSPACE : MEDA_ERR_BUDGET_INFEASIBLE);
    return;
  }
  const float* sc = scores + (size_t)g * n;
  int32_t* out_c = idx_conserved + (size_t)g * cap;
  int32_t* out_l = idx_less + (size_t)g * n;
  const int lo = rank * L.chunk, hi = min(lo + L.chunk, n);

  // ---- stage the keys; count the text candidates
  int my_text = 0;
  for (int j = lo + (int)threadIdx.x; j < hi; j += kSelThreads) {
    unsigned int b = __float_as_uint(sc[j]);
    keys[j - lo] = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
    my_text += (j < n_cand && modality[j] == MEDA_TEXT) ? 1 : 0;
  }
  my_text = __reduce_add_sync(0xffffffffu, my_text);
  if (threadIdx.x == 0) misc[40] = 0;
  __syncthreads();
  if (threadIdx.x % 32 == 0 && my_text) atomicAdd(&misc[40], my_text);
  cluster.sync();
  int text_total = 0;
  for (int r = 0; r < kSelClusterSize; ++r) text_total += cluster.map_shared_rank(misc, r)[40];
  // Eq. 9 puts every text candidate ahead of every visual one: the N-th ranked candidate is a text
  // token iff N <= #text candidates; the other class is then wholly kept or wholly dropped.
  const int cls = (N <= text_total) ? MEDA_TEXT : MEDA_VISUAL;
  int remaining = (cls == MEDA_TEXT) ? N : N - text_total;

  // ---- the `remaining`-th largest key inside the class, most significant digit first
  unsigned int prefix = 0u, mask = 0u;
  if (N > 0) {
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
      const unsigned int bins = pass == 2 ? 1024u : 2048u;
      // Alternate passes count into alternate histograms: the other blocks read this block's histogram of pass p
      // before they arrive at the barrier of pass p + 1, and it is cleared again only in pass p + 2, so one
      // cluster barrier per pass is enough.
      unsigned int* h = hist + (pass & 1) * kSelBins;
      for (int b = threadIdx.x; b < kSelBins; b += kSelThreads) h[b] = 0u;
      __syncthreads();
      for (int j = lo + (int)threadIdx.x; j < min(hi, n_cand); j += kSelThreads) {
        const unsigned int key = keys[j - lo];
        if (modality[j] == cls && (key & mask) == prefix) atomicAdd(&h[(key >> shift) & (bins - 1u)], 1u);
      }
      cluster.sync();                                   // every block's histogram is complete
      // Thread t owns the bins bins - 1 - 2t and bins - 2 - 2t (from the top down), summed over the cluster; an
      // exclusive sum over the threads gives the number of keys in all bins above, and the one thread whose bins
      // hold the `remaining`-th key from the top records the digit.
      const int b0 = (int)bins - 1 - 2 * (int)threadIdx.x, b1 = b0 - 1;       // b1 is even: one 8-byte load for both
      int c0 = 0, c1 = 0;
      if (b1 >= 0) {
#pragma unroll
        for (int r = 0; r < kSelClusterSize; ++r) {
          const uint2 pair = *reinterpret_cast<const uint2*>(cluster.map_shared_rank(h, r) + b1);
          c1 += (int)pair.x;
          c0 += (int)pair.y;
        }
      }
      int all_keys;
      const int above = block_exclusive_sum(c0 + c1, misc, all_keys);
      if (above < remaining && above + c0 + c1 >= remaining) {
        if (above + c0 >= remaining) { misc[44] = b0; misc[45] = remaining - above; }
        else { misc[44] = b1; misc[45] = remaining - above - c0; }
      }
      __syncthreads();
      prefix |= (unsigned int)misc[44] << shift;
      mask |= (bins - 1u) << shift;
      remaining = misc[45];
    }
  }
  const unsigned int threshold = prefix;
  const int take_equal = N > 0 ? remaining : 0;

  // ---- classify own tokens, 16 consecutive ones per thread and round: 2 = kept for sure, 1 = equal to the
  // threshold, 0 = dropped; two bits per token, kept in registers for the compaction below
  uint32_t codes[kSelMaxRounds];
  int sure = 0, equal = 0;
#pragma unroll
  for (int r = 0; r < kSelMaxRounds; ++r) {
    codes[r] = 0u;
    const int j0 = lo + (r * kSelThreads + (int)threadIdx.x) * kSelPerThread;
    if (j0 < hi) {
      // the modality map is padded past n and j0 is a multiple of 16: one 16-byte load; keys: four
      const uint4 mv = *reinterpret_cast<const uint4*>(modality + j0);
      const uint32_t mw[4] = {mv.x, mv.y, mv.z, mv.w};
      const uint4* kp = reinterpret_cast<const uint4*>(keys + (j0 - lo));
#pragma unroll
      for (int w4 = 0; w4 < 4; ++w4) {
        const uint4 kv = kp[w4];
        const unsigned int kk[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          const int x = 4 * w4 + b, j = j0 + x;
          const int md = (int)((mw[w4] >> (8 * b)) & 0xffu);
          int c;
          if (j >= n) c = 0;
          else if (j >= n_cand) c = 2;
          else if (N == 0) c = 0;
          else if (md != cls) c = (cls == MEDA_VISUAL) ? 2 : 0;
          else c = kk[b] > threshold ? 2 : (kk[b] == threshold ? 1 : 0);
          codes[r] |= (uint32_t)c << (2 * x);
          sure += c == 2;
          equal += c == 1;
        }
      }
    }
  }
  sure = __reduce_add_sync(0xffffffffu, sure);
  equal = __reduce_add_sync(0xffffffffu, equal);
  if (threadIdx.x == 0) { misc[41] = 0; misc[42] = 0; }
  __syncthreads();
  if (threadIdx.x % 32 == 0) { atomicAdd(&misc[41], sure); atomicAdd(&misc[42], equal); }
  cluster.sync();
  int kept_before = 0, equal_before = 0;
  for (int r = 0; r < rank; ++r) {
    const int* m = cluster.map_shared_rank(misc, r);
    const int e = m[42];
    kept_before += m[41] + min(max(take_equal - equal_before, 0), e);
    equal_before += e;
  }

  // ---- ordered compaction of own tokens.  The positions are computed per thread (16 consecutive tokens), but
  // written to global memory by the whole block from shared memory, where the sort keys are no longer needed:
  // kept indices from the front of the buffer, dropped ones from its back (a block's dropped tokens are
  // contiguous in the less-important list too), so that every global store is a full line.
  int* stage = reinterpret_cast<int*>(keys);
#pragma unroll
  for (int r = 0; r < kSelMaxRounds; ++r) {
    const int r_lo = lo + r * kSelThreads * kSelPerThread;             // first token of the round
    if (r_lo >= hi) break;                                            // uniform over the block
    const int r_n = min(kSelThreads * kSelPerThread, hi - r_lo);       // tokens of the round
    const int j0 = r_lo + (int)threadIdx.x * kSelPerThread;
    const uint32_t cd = codes[r];
    // tokens equal to the threshold: code 1; kept for sure: code 2
    const uint32_t eq_bits = cd & ~(cd >> 1) & 0x55555555u, sure_bits = (cd >> 1) & 0x55555555u;
    int eq_total, keep_total;
    int eq_rank = equal_before + block_exclusive_sum(__popc(eq_bits), misc, eq_total);
    uint32_t keep_bits = sure_bits;
#pragma unroll
    for (int x = 0; x < kSelPerThread; ++x) {
      if ((eq_bits >> (2 * x)) & 1u) {
        if (eq_rank < take_equal) keep_bits |= 1u << (2 * x);
        ++eq_rank;
      }
    }
    // (the first barrier inside the sum above also orders the last reads of the keys before the stores below)
    int pos = block_exclusive_sum(__popc(keep_bits), misc, keep_total);   // kept tokens of the round before mine
#pragma unroll
    for (int x = 0; x < kSelPerThread; ++x) {
      const int j = j0 + x;
      if (j < hi) {
        if ((keep_bits >> (2 * x)) & 1u) { stage[pos] = j; ++pos; }
        else stage[r_n - 1 - ((j - r_lo) - pos)] = j;
      }
    }
    __syncthreads();
    const int drop_total = r_n - keep_total;
    int32_t* dst_c = out_c + kept_before;
    int32_t* dst_l = out_l + (r_lo - kept_before);
    for (int e = threadIdx.x; e < keep_total; e += kSelThreads) dst_c[e] = stage[e];
    for (int e = threadIdx.x; e < drop_total; e += kSelThreads) dst_l[e] = stage[r_n - 1 - e];
    kept_before += keep_total;
    equal_before += eq_total;
    __syncthreads();                                                  // the buffer is reused by the next round
  }
  cluster.sync();                                       // no block leaves while another may still read its counters
}

}  // namespace meda
