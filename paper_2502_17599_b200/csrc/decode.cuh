// After the pass: attention of one new token over a layer's cache (Eq. 3), full or compressed.
// Reads the cache once: every warp walks a strided share of the rows of one KV head, a few rows at a
// time, keeps an online softmax (max, sum, weighted value sum) per query head of the group with lane l
// owning elements [l * E, l * E + E) of the head dimension; the warps of a block and then the blocks of
// a head are merged in a fixed order.  The row count comes from the layer's budget row on the device
// (or is given by the host for a cache that was not compressed).
#pragma once

#include "group_reduce.cuh"   // load_row
#include "meda_common.cuh"

namespace meda {

constexpr int kDecWarps = 8;
constexpr int kDecMaxGroup = 16;      // query heads per KV head this kernel accepts
constexpr int kDecSplits = 74;        // blocks per KV head: with 4 KV heads two blocks per SM
constexpr int kDecBatch = 4;          // rows per warp that one block of a short cache gets (see decode_active_splits)

// partial[h][split] = (m, z, acc[D]) of the rows block `split` saw, D + 2 floats each.
// Short caches use fewer blocks (one per 32 rows), so that the partial states written and merged stay in
// proportion to the cache.
__device__ __forceinline__ int decode_active_splits(int rows) {
  return min(max((rows + kDecWarps * kDecBatch - 1) / (kDecWarps * kDecBatch), 1), kDecSplits);
}

// Rows a warp scores at once for G query heads per KV head: G * B (row, head) pairs share one transposing
// reduction, so B is a power of two with G * B <= 32.
template <int G>
struct DecodeShape {
  static constexpr int B = G <= 4 ? 8 : 4;
  static constexpr int PAIRS = G * B;
  static constexpr int P = PAIRS <= 8 ? 8 : (PAIRS <= 16 ? 16 : 32);     // lanes of one reduction group
};

// Every lane holds P partial sums v[0 .. P); afterwards v[0] of lane l is the sum over the warp's lanes of
// v[l % P]: a transposing butterfly (P - 1 exchanges inside groups of P lanes) and, for P < 32, a plain butterfly
// over the groups.  The order of the additions is fixed.
template <int P>
__device__ __forceinline__ float transpose_reduce(float (&v)[P], int lane) {
#pragma unroll
  for (int step = P / 2; step >= 1; step >>= 1) {
    const bool upper = (lane & step) != 0;
#pragma unroll
    for (int i = 0; i < step; ++i) {
      const float send = upper ? v[i] : v[i + step];
      const float keep = upper ? v[i + step] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, step);
    }
  }
  float r = v[0];
#pragma unroll
  for (int o = P; o < 32; o <<= 1) r += __shfl_xor_sync(0xffffffffu, r, o);
  return r;
}

// One warp walks a strided share of the rows, B rows at a time.  The partial dot products of the B x G
// (row, head) pairs are reduced together, so that lane h * B + b ends up owning pair (row b, head h): it alone
// evaluates the pair's exponential (one special-function instruction per batch instead of two per pair and
// lane), the online-softmax update of head h runs inside its B lanes, and the probabilities come back to every
// lane by one shuffle each for the weighted sum of the value rows.
template <typename T, int D, int G>
__global__ void __launch_bounds__(kDecWarps * 32)
decode_partial_kernel(const T* __restrict__ q, const T* __restrict__ k_c, const T* __restrict__ v_c,
                      const int32_t* __restrict__ budget_row, int rows_given, int cap, float* __restrict__ partial,
                      float scale) {
  constexpr int E = D / 32;
  using Shape = DecodeShape<G>;
  constexpr int B = Shape::B, P = Shape::P;
  __shared__ float s_m[kDecWarps][G], s_z[kDecWarps][G];
  __shared__ float s_acc[kDecWarps][G][D];
  const int g = blockIdx.y, split = blockIdx.x, warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int rows = min(budget_row ? budget_row[0] : rows_given, cap);
  const int n_splits = decode_active_splits(rows);
  if (split >= n_splits) return;
  float qv[G][E], acc[G][E];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    load_row<T, E>(q + (size_t)(g * G + h) * D, lane, qv[h]);
#pragma unroll
    for (int e = 0; e < E; ++e) {
      qv[h][e] *= scale;
      acc[h][e] = 0.f;
    }
  }
  // lane h * B + b owns pair (b, h); the running (max, sum) of head h lives, identically, in its B lanes
  const int pair = lane % P;
  const int my_h = pair / B, my_b = pair % B;
  const bool owner = pair < Shape::PAIRS;
  float m_run = -INFINITY, z_run = 0.f;
  const T* kg = k_c + (size_t)g * cap * D;
  const T* vg = v_c + (size_t)g * cap * D;
  const int kStride = n_splits * kDecWarps;
  for (int r0 = split * kDecWarps + warp; r0 < rows; r0 += kStride * B) {
    float kr[B][E], vr[B][E];
#pragma unroll
    for (int b = 0; b < B; ++b) {
      const int r = min(r0 + b * kStride, rows - 1);
      load_row<T, E>(kg + (size_t)r * D, lane, kr[b]);
      load_row<T, E>(vg + (size_t)r * D, lane, vr[b]);
    }
    float part[P];
#pragma unroll
    for (int i = 0; i < P; ++i) part[i] = 0.f;
#pragma unroll
    for (int h = 0; h < G; ++h)
#pragma unroll
      for (int b = 0; b < B; ++b) {
        float dot = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) dot = fmaf(qv[h][e], kr[b][e], dot);
        part[h * B + b] = dot;
      }
    float s = transpose_reduce<P>(part, lane);                      // this lane's pair: q_h . k_b / sqrt(d)
    if (!owner || r0 + my_b * kStride >= rows) s = -INFINITY;
    float m_new = s;                                                // maximum over the head's B rows, then the running one
#pragma unroll
    for (int o = 1; o < B; o <<= 1) m_new = fmaxf(m_new, __shfl_xor_sync(0xffffffffu, m_new, o));
    m_new = fmaxf(m_new, m_run);
    const float pr = m_new == -INFINITY ? 0.f : __expf(s - m_new);
    const float c_old = m_new == -INFINITY ? 1.f : __expf(m_run - m_new);
    float psum = pr;
#pragma unroll
    for (int o = 1; o < B; o <<= 1) psum += __shfl_xor_sync(0xffffffffu, psum, o);
    z_run = z_run * c_old + psum;
    m_run = m_new;
#pragma unroll
    for (int h = 0; h < G; ++h) {
      const float c = __shfl_sync(0xffffffffu, c_old, h * B);
#pragma unroll
      for (int e = 0; e < E; ++e) acc[h][e] *= c;
#pragma unroll
      for (int b = 0; b < B; ++b) {
        const float w = __shfl_sync(0xffffffffu, pr, h * B + b);
#pragma unroll
        for (int e = 0; e < E; ++e) acc[h][e] = fmaf(w, vr[b][e], acc[h][e]);
      }
    }
  }
  float m[G], z[G];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    m[h] = __shfl_sync(0xffffffffu, m_run, h * B);
    z[h] = __shfl_sync(0xffffffffu, z_run, h * B);
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
