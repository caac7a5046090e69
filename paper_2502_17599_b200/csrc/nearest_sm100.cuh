// Phase B, merge step 1 for bf16 / head_dim 128 on the 5th-generation tensor cores (Eq. 11 and the
// arg-max that follows it): for every token row i of a KV head, the conserved slot s maximising
// k_i . k_{c_s} / |k_{c_s}|  (the row's own norm is a positive factor common to all slots).
//
// The similarity matrix is never stored.  A persistent block owns 256 consecutive token rows (two
// 128-row UMMA tiles, loaded once by TMA straight from the caller's key cache) and sweeps all
// conserved slots in tiles of 128 columns (TMA from the gathered conserved keys).  Accumulators
// live in tensor memory, double buffered; eight epilogue warps read them back with tcgen05.ld,
// scale each column by its inverse norm in fp32 and keep a running (value, first slot) maximum per
// row.  All token rows are swept, the conserved ones included (their result is ignored): that
// wastes S/n of the contraction but needs no row gather for the large operand.
#pragma once

#include "umma_stream.cuh"

namespace meda {

// Gathers the conserved keys of every KV head into a dense operand and computes their inverse
// norms: kc[g][s][:] = k[g][c_s][:], inv_norm[g][s] = 1 / max(|k[g][c_s]|, eps).  One warp per slot.
__global__ void __launch_bounds__(256)
gather_conserved_bf16_kernel(const __nv_bfloat16* __restrict__ k, const int32_t* __restrict__ idx_conserved,
                             const int32_t* __restrict__ budget_row, __nv_bfloat16* __restrict__ kc,
                             float* __restrict__ inv_norm, int n, int cap, int kc_rows, int inv_stride) {
  const int g = blockIdx.y;
  const int S = min(budget_row[0], cap);
  const int slot = blockIdx.x * 8 + threadIdx.x / 32;
  if (slot >= S) return;
  const int lane = threadIdx.x % 32;
  int row = idx_conserved[(size_t)g * cap + slot];
  row = min(max(row, 0), n - 1);
  const uint2* src = reinterpret_cast<const uint2*>(k + ((size_t)g * n + row) * kFastDim);
  uint2 x = src[lane];
  reinterpret_cast<uint2*>(kc + ((size_t)g * kc_rows + slot) * kFastDim)[lane] = x;
  float2 a = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&x.x));
  float2 b = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&x.y));
  float ss = a.x * a.x + a.y * a.y + b.x * b.x + b.y * b.y;
  ss = warp_sum(ss);
  if (lane == 0) inv_norm[(size_t)g * inv_stride + slot] = 1.f / fmaxf(sqrtf(ss), kCosEps);
}

// target[g][p] = token_target[g][less[p]]: from per-token results to the less-important list order.
__global__ void remap_targets_kernel(const int32_t* __restrict__ token_target, const int32_t* __restrict__ idx_less,
                                     const int32_t* __restrict__ budget_row, int32_t* __restrict__ target, int n,
                                     int cap) {
  const int g = blockIdx.y;
  const int S = min(budget_row[0], cap);
  const int p = blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= n - S) return;
  int row = min(max(idx_less[(size_t)g * n + p], 0), n - 1);
  target[(size_t)g * n + p] = token_target[(size_t)g * n + row];
}

// Policy of the streaming UMMA pipeline: resident block = 256 token rows of one KV head, streamed
// tiles = 128 conserved slots each, epilogue = running (value, first slot) maximum per token row.
struct NearestPolicy {
  struct Params {
    const float* inv_norm;
    const int32_t* budget_row;
    int32_t* token_target;
    int n, n_heads, cap, inv_stride;
  };
  static constexpr int kABuffers = 1;
  static constexpr int kBStages = 4;
  static constexpr uint32_t kExtraBytes = kUsEpilogueWarps * 128 * 4;   // one inverse-norm slice per epilogue warp

  __device__ static int slots(const Params& p) { return min(p.budget_row[0], p.cap); }
  __device__ static bool active(const Params& p) {
    const int S = slots(p);
    return S > 0 && S < p.n;                       // otherwise there is nothing to merge
  }
  __device__ static bool get_item(const Params& p, int it, StreamItem& o) {
    const int m_blocks = (p.n + 255) / 256;
    const int idx = blockIdx.x + it * gridDim.x;
    if (idx >= m_blocks * p.n_heads) return false;
    const int S = slots(p);
    o.a_head = o.b_head = idx / m_blocks;
    o.a_row = (idx % m_blocks) * 256;
    o.b_row = 0;
    o.n_tiles = (S + 127) / 128;
    o.last_n = 128;
    o.m_tiles = (p.n - o.a_row > 128) ? 2 : 1;
    o.u0 = S;
    o.u1 = 0;
    return true;
  }

  struct Epilogue {
    float* inv_t;
    int lane, row_in_block;
    float best;
    int best_slot;
    __device__ void init(const Params&, unsigned char* extra, int ewarp, int lane_) {
      inv_t = reinterpret_cast<float*>(extra) + ewarp * 128;
      lane = lane_;
      row_in_block = (ewarp / 4) * 128 + ((ewarp + 2) % 4) * 32 + lane_;   // (ewarp + 2) % 4 == warp % 4
    }
    __device__ void item_begin(const Params&, const StreamItem&) {
      best = -INFINITY;
      best_slot = 0;
    }
    __device__ void tile(const Params& p, const StreamItem& it, int tile, uint32_t taddr) {
      const int S = it.u0;
      const int c0 = tile * 128;
      // this warp's private copy of the tile's 128 inverse norms (the array is padded so that a
      // whole slice can always be read)
      const float* inv_g = p.inv_norm + (size_t)it.b_head * p.inv_stride;
      __syncwarp();
      reinterpret_cast<float4*>(inv_t)[lane] = __ldg(reinterpret_cast<const float4*>(inv_g + c0) + lane);
      __syncwarp();
      const bool ragged = c0 + 128 > S;
#pragma unroll 1
      for (int chunk = 0; chunk < 4; ++chunk) {
        float v[32];
        sm100::tmem_ld_32x32(taddr + chunk * 32u, v);
        const float4* inv4 = reinterpret_cast<const float4*>(inv_t + chunk * 32);
#pragma unroll
        for (int x = 0; x < 8; ++x) {
          const float4 w = inv4[x];
          v[4 * x + 0] *= w.x; v[4 * x + 1] *= w.y; v[4 * x + 2] *= w.z; v[4 * x + 3] *= w.w;
        }
        if (ragged) {
#pragma unroll
          for (int x = 0; x < 32; ++x) if (c0 + chunk * 32 + x >= S) v[x] = -INFINITY;
        }
        float cmax = -INFINITY;
#pragma unroll
        for (int x = 0; x < 32; ++x) cmax = fmaxf(cmax, v[x]);
        if (cmax > best) {
          int first = 31;
#pragma unroll
          for (int x = 31; x >= 0; --x) if (v[x] == cmax) first = x;
          best = cmax;
          best_slot = c0 + chunk * 32 + first;
        }
      }
    }
    __device__ void item_end(const Params& p, const StreamItem& it) {
      const int token = it.a_row + row_in_block;
      if (token < p.n) p.token_target[(size_t)it.a_head * p.n + token] = best_slot;
    }
  };
};

}  // namespace meda
