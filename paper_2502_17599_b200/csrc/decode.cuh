// After the pass: attention of one new token over a layer's cache (Eq. 3), full or compressed.
// Reads the cache once: every warp walks a strided share of the rows of one KV head, keeps an
// online softmax (max, sum, weighted value sum) per query head of the group with lane l owning
// elements [l * E, l * E + E) of the head dimension, the warps of a block and then the blocks of a
// head are merged in a fixed order.  The row count comes from the layer's budget row on the device
// (or is given by the host for a cache that was not compressed).
#pragma once

#include "group_reduce.cuh"   // load_row
#include "meda_common.cuh"

namespace meda {

constexpr int kDecWarps = 8;
constexpr int kDecMaxGroup = 16;      // query heads per KV head this kernel accepts
constexpr int kDecSplits = 74;        // blocks per KV head: with 4 KV heads two blocks per SM
constexpr int kDecBatch = 4;          // rows a warp has in flight

// partial[h][split] = (m, z, acc[D]) of the rows block `split` saw, D + 2 floats each.
// Short caches use fewer blocks (one per 32 rows), so that the partial states written and merged stay in
// proportion to the cache.
__device__ __forceinline__ int decode_active_splits(int rows) {
  return min(max((rows + kDecWarps * kDecBatch - 1) / (kDecWarps * kDecBatch), 1), kDecSplits);
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(kDecWarps * 32)
decode_partial_kernel(const T* __restrict__ q, const T* __restrict__ k_c, const T* __restrict__ v_c,
                      const int32_t* __restrict__ budget_row, int rows_given, int cap, float* __restrict__ partial,
                      float scale) {
  constexpr int E = D / 32;
  __shared__ float s_m[kDecWarps][G], s_z[kDecWarps][G];
  __shared__ float s_acc[kDecWarps][G][D];
  const int g = blockIdx.y, split = blockIdx.x, warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int rows = min(budget_row ? budget_row[0] : rows_given, cap);
  const int n_splits = decode_active_splits(rows);
  if (split >= n_splits) return;
  float qv[G][E], acc[G][E], m[G], z[G];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    load_row<T, E>(q + (size_t)(g * G + h) * D, lane, qv[h]);
    m[h] = -INFINITY;
    z[h] = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[h][e] = 0.f;
  }
  const T* kg = k_c + (size_t)g * cap * D;
  const T* vg = v_c + (size_t)g * cap * D;
  const int kStride = n_splits * kDecWarps;
  for (int r0 = split * kDecWarps + warp; r0 < rows; r0 += kStride * kDecBatch) {
    float kr[kDecBatch][E], vr[kDecBatch][E];
#pragma unroll
    for (int b = 0; b < kDecBatch; ++b) {
      const int r = min(r0 + b * kStride, rows - 1);
      load_row<T, E>(kg + (size_t)r * D, lane, kr[b]);
      load_row<T, E>(vg + (size_t)r * D, lane, vr[b]);
    }
#pragma unroll
    for (int b = 0; b < kDecBatch; ++b) {
      if (r0 + b * kStride < rows) {
#pragma unroll
        for (int h = 0; h < G; ++h) {
          float dot = 0.f;
#pragma unroll
          for (int e = 0; e < E; ++e) dot = fmaf(qv[h][e], kr[b][e], dot);
          const float s = warp_sum(dot) * scale;
          const float m_new = fmaxf(m[h], s);
          const float c_old = __expf(m[h] - m_new), p = __expf(s - m_new);
          z[h] = z[h] * c_old + p;
#pragma unroll
          for (int e = 0; e < E; ++e) acc[h][e] = fmaf(acc[h][e], c_old, p * vr[b][e]);
          m[h] = m_new;
        }
      }
    }
  }
  // warps of the block, in warp order
#pragma unroll
  for (int h = 0; h < G; ++h) {
    if (lane == 0) { s_m[warp][h] = m[h]; s_z[warp][h] = z[h]; }
#pragma unroll
    for (int e = 0; e < E; ++e) s_acc[warp][h][lane * E + e] = acc[h][e];
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
    const int h = idx / D, t = idx % D;
    float mm = -INFINITY;
    for (int w = 0; w < kDecWarps; ++w) mm = fmaxf(mm, s_m[w][h]);
    float zz = 0.f, aa = 0.f;
    for (int w = 0; w < kDecWarps; ++w) {
      const float c = s_m[w][h] == -INFINITY ? 0.f : __expf(s_m[w][h] - mm);
      zz = fmaf(s_z[w][h], c, zz);
      aa = fmaf(s_acc[w][h][t], c, aa);
    }
    float* po = partial + ((size_t)(g * G + h) * kDecSplits + split) * (D + 2);
    if (t == 0) { po[0] = mm; po[1] = zz; }
    po[2 + t] = aa;
  }
}

// out[h] = merge of the splits, in split order, divided by the normaliser.  grid = Hq, block = D.
template <int D>
__global__ void decode_combine_kernel(const float* __restrict__ partial, const int32_t* __restrict__ budget_row,
                                      int rows_given, int cap, float* __restrict__ out) {
  const int h = blockIdx.x, t = threadIdx.x;
  const int n_splits = decode_active_splits(min(budget_row ? budget_row[0] : rows_given, cap));
  const float* p = partial + (size_t)h * kDecSplits * (D + 2);
  float mm = -INFINITY;
  for (int s = 0; s < n_splits; ++s) mm = fmaxf(mm, p[s * (D + 2)]);
  float zz = 0.f, aa = 0.f;
  for (int s = 0; s < n_splits; ++s) {
    const float ms = p[s * (D + 2)];
    const float c = ms == -INFINITY ? 0.f : __expf(ms - mm);
    zz = fmaf(p[s * (D + 2) + 1], c, zz);
    aa = fmaf(p[s * (D + 2) + 2 + t], c, aa);
  }
  out[(size_t)h * D + t] = zz > 0.f ? aa / zz : 0.f;
}

}  // namespace meda
