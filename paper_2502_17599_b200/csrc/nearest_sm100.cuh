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
  const int lane = threadIdx.x % 32;
  // the grid is sized on the host for the largest possible S: walk the slots with a stride
  for (int slot = blockIdx.x * 8 + threadIdx.x / 32; slot < S; slot += gridDim.x * 8) {
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
  static constexpr uint32_t kItemExtraBytes = 0;
  static constexpr int kEpilogueGroups = 1;

  __device__ static int slots(const Params& p) { return min(p.budget_row[0], p.cap); }
  __device__ static bool active(const Params& p) {
    const int S = slots(p);
    return S > 0 && S < p.n;                       // otherwise there is nothing to merge
  }
  // Token rows [n - M, n) are the recent window: always conserved, never merged, so the 256-row
  // blocks that lie wholly inside it are not swept.
  __device__ static int rows_swept(const Params& p) {
    const int m = min(max(p.budget_row[1], 0), p.n);
    return p.n - m;
  }
  __device__ static bool get_item(const Params& p, int it, StreamItem& o) {
    const int m_blocks = (rows_swept(p) + 255) / 256;
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
    __device__ void item_begin(const Params&, const StreamItem&, const unsigned char*) {
      best = -INFINITY;
      best_slot = 0;
    }
    // One chunk = this thread's row against 32 consecutive slots: scale by the slots' inverse norms
    // (two products per instruction), reduce with three-input maxima, and only when the chunk
    // beats the running best look for the first slot that attains it.
    __device__ __forceinline__ void chunk(const uint32_t (&r)[32], int chunk_idx, int c0, int S, bool ragged) {
      const ulonglong2* inv2 = reinterpret_cast<const ulonglong2*>(inv_t + chunk_idx * 32);
      float v[32];
#pragma unroll
      for (int x = 0; x < 8; ++x) {
        const ulonglong2 w = inv2[x];
        sm100::mul_f32x2(sm100::pack_f32x2(r[4 * x + 0], r[4 * x + 1]), w.x, v[4 * x + 0], v[4 * x + 1]);
        sm100::mul_f32x2(sm100::pack_f32x2(r[4 * x + 2], r[4 * x + 3]), w.y, v[4 * x + 2], v[4 * x + 3]);
      }
      const int s0 = c0 + chunk_idx * 32;
      if (ragged) {
#pragma unroll
        for (int x = 0; x < 32; ++x) if (s0 + x >= S) v[x] = -INFINITY;
      }
      float t[12];
#pragma unroll
      for (int x = 0; x < 10; ++x) t[x] = sm100::fmax3(v[3 * x], v[3 * x + 1], v[3 * x + 2]);
      t[10] = v[30];
      t[11] = v[31];
      const float u0 = sm100::fmax3(t[0], t[1], t[2]), u1 = sm100::fmax3(t[3], t[4], t[5]);
      const float u2 = sm100::fmax3(t[6], t[7], t[8]), u3 = sm100::fmax3(t[9], t[10], t[11]);
      const float cmax = fmaxf(sm100::fmax3(u0, u1, u2), u3);
      if (cmax > best) {
        int first = 31;
#pragma unroll
        for (int x = 30; x >= 0; --x) if (v[x] == cmax) first = x;
        best = cmax;
        best_slot = s0 + first;
      }
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
      // two register buffers: the load of chunk c + 1 is in flight while chunk c is reduced
      uint32_t ra[32], rb[32];
      sm100::tmem_ld_32x32_issue(taddr, ra);
      sm100::tmem_ld_wait();
      sm100::tmem_ld_pin(ra);
      sm100::tmem_ld_32x32_issue(taddr + 32u, rb);
      chunk(ra, 0, c0, S, ragged);
      sm100::tmem_ld_wait();
      sm100::tmem_ld_pin(rb);
      sm100::tmem_ld_32x32_issue(taddr + 64u, ra);
      chunk(rb, 1, c0, S, ragged);
      sm100::tmem_ld_wait();
      sm100::tmem_ld_pin(ra);
      sm100::tmem_ld_32x32_issue(taddr + 96u, rb);
      chunk(ra, 2, c0, S, ragged);
      sm100::tmem_ld_wait();
      sm100::tmem_ld_pin(rb);
      chunk(rb, 3, c0, S, ragged);
    }
    __device__ void item_end(const Params& p, const StreamItem& it) {
      const int token = it.a_row + row_in_block;
      if (token < p.n) p.token_target[(size_t)it.a_head * p.n + token] = best_slot;
    }
  };
};

}  // namespace meda
