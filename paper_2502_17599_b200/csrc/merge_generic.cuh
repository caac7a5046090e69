// Phase B, merging (Eq. 11-12), dtype-generic CUDA-core kernels: inverse norms of the conserved
// keys and nearest conserved key of every less-important key (cosine similarity, first maximum).
// These are the fp32 path and the path for head dimensions the tensor-core kernel does not cover.
#pragma once

#include "meda_common.cuh"

namespace meda {

// inv_norm[g][s] = 1 / max(|k[c_s]|, eps).  One warp per conserved slot.
template <typename T>
__global__ void conserved_inv_norm_kernel(const T* __restrict__ k, const int32_t* __restrict__ idx_conserved,
                                          const int32_t* __restrict__ budget_row, float* __restrict__ inv_norm,
                                          int n, int d, int cap, int inv_stride) {
  const int g = blockIdx.y;
  const int S = min(budget_row[0], cap);
  const int slot = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
  if (slot >= S) return;
  const int lane = threadIdx.x % 32;
  int row = idx_conserved[(size_t)g * cap + slot];
  row = min(max(row, 0), n - 1);
  const T* kr = k + ((size_t)g * n + row) * d;
  float ss = 0.f;
  for (int t = lane; t < d; t += 32) { float x = to_f32<T>(kr[t]); ss = fmaf(x, x, ss); }
  ss = warp_sum(ss);
  if (lane == 0) inv_norm[(size_t)g * inv_stride + slot] = 1.f / fmaxf(sqrtf(ss), kCosEps);
}

// target[g][p] = argmax over slots s of k[less_p] . k[c_s] * inv_norm[s]  (the row's own norm is a
// positive factor common to all s, so it does not move the arg-max), first maximum in slot order.
// Tile: 64 less rows x 64 slots per step, 16x16 threads, 4x4 outputs each.
constexpr int kNnTile = 64;
constexpr int kNnDk = 32;

template <typename T>
__global__ void __launch_bounds__(256)
nearest_generic_kernel(const T* __restrict__ k, const int32_t* __restrict__ idx_conserved,
                       const int32_t* __restrict__ idx_less, const int32_t* __restrict__ budget_row,
                       const float* __restrict__ inv_norm, int32_t* __restrict__ target, int n, int d, int cap,
                       int inv_stride) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* a_s = reinterpret_cast<float*>(smem_raw);               // [64][d + 1]
  float* b_s = a_s + kNnTile * (d + 1);                          // [64][kNnDk + 1]
  const int g = blockIdx.y;
  const int S = min(budget_row[0], cap);
  const int n_less = n - S;
  const int r0 = blockIdx.x * kNnTile;
  if (r0 >= n_less || S <= 0) return;
  const T* k_g = k + (size_t)g * n * d;
  const int32_t* less = idx_less + (size_t)g * n;
  const int32_t* cons = idx_conserved + (size_t)g * cap;
  const float* inv = inv_norm + (size_t)g * inv_stride;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;

  for (int e = threadIdx.x; e < kNnTile * d; e += 256) {
    int r = e / d, c = e - r * d;
    int p = r0 + r;
    float x = 0.f;
    if (p < n_less) { int row = min(max(less[p], 0), n - 1); x = to_f32<T>(k_g[(size_t)row * d + c]); }
    a_s[r * (d + 1) + c] = x;
  }
  float best[4];
  int best_slot[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) { best[r] = -INFINITY; best_slot[r] = 0; }

  for (int c0 = 0; c0 < S; c0 += kNnTile) {
    float acc[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;
    for (int t0 = 0; t0 < d; t0 += kNnDk) {
      __syncthreads();
      for (int e = threadIdx.x; e < kNnTile * kNnDk; e += 256) {
        int r = e / kNnDk, c = e - r * kNnDk;
        int s = c0 + r;
        float x = 0.f;
        if (s < S) { int row = min(max(cons[s], 0), n - 1); x = to_f32<T>(k_g[(size_t)row * d + t0 + c]); }
        b_s[r * (kNnDk + 1) + c] = x;
      }
      __syncthreads();
#pragma unroll 4
      for (int t = 0; t < kNnDk; ++t) {
        float av[4], bv[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) av[r] = a_s[(ty * 4 + r) * (d + 1) + t0 + t];
#pragma unroll
        for (int c = 0; c < 4; ++c) bv[c] = b_s[(tx * 4 + c) * (kNnDk + 1) + t];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
          for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(av[r], bv[c], acc[r][c]);
      }
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      int s = c0 + tx * 4 + c;
      if (s < S) {
        float w = inv[s];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          float u = acc[r][c] * w;
          if (u > best[r]) { best[r] = u; best_slot[r] = s; }
        }
      }
    }
  }
  // combine the 16 column owners of each row: larger value wins, equal values -> lower slot
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    float b = best[r];
    int s = best_slot[r];
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
      float b2 = __shfl_xor_sync(0xffffffffu, b, o);
      int s2 = __shfl_xor_sync(0xffffffffu, s, o);
      if (b2 > b || (b2 == b && s2 < s)) { b = b2; s = s2; }
    }
    int p = r0 + ty * 4 + r;
    if (tx == 0 && p < n_less) target[(size_t)g * n + p] = s;
  }
}

}  // namespace meda
