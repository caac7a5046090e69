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

#include "meda_common.cuh"
#include "sm100_primitives.cuh"

namespace meda {

constexpr int kFastDim = 128;            // head_dim of the tcgen05 paths
constexpr int kNnBlockM = 256;           // token rows per work item
constexpr int kNnTileN = 128;            // conserved slots per accumulator tile
constexpr int kNnStages = 4;             // B-operand ring
constexpr int kNnThreads = 320;          // warp 0: TMA, warp 1: UMMA issue + TMEM owner, warps 2-9: epilogue
constexpr int kNnEpilogueThreads = 256;
constexpr uint32_t kNnABytes = kNnBlockM * kFastDim * 2;
constexpr uint32_t kNnBBytes = kNnTileN * kFastDim * 2;
constexpr uint32_t kNnHalfTile = 128 * 64 * 2;   // one 128-row x 64-column bf16 box (16 KB)
constexpr uint32_t kNnTmemCols = 512;

struct NnShared {
  // offsets from the 1024-byte aligned base of dynamic shared memory
  static constexpr uint32_t a_off = 0;
  static constexpr uint32_t b_off = a_off + kNnABytes;
  static constexpr uint32_t inv_off = b_off + kNnStages * kNnBBytes;
  static constexpr uint32_t bar_off = inv_off + (kNnEpilogueThreads / 32) * kNnTileN * 4;   // one slice per epilogue warp
  static constexpr uint32_t n_bars = 2 + 2 * kNnStages + 4;
  static constexpr uint32_t misc_off = bar_off + n_bars * 8;
  static constexpr uint32_t total = misc_off + 16;
  static constexpr uint32_t alloc = total + 1024;   // slack for the manual 1024-byte alignment
};

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

__global__ void __launch_bounds__(kNnThreads, 1)
nearest_sm100_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_kc,
                     const float* __restrict__ inv_norm, const int32_t* __restrict__ budget_row,
                     int32_t* __restrict__ token_target, int n, int n_heads, int cap, int inv_stride, int* status) {
  using namespace sm100;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* a_smem = smem + NnShared::a_off;
  unsigned char* b_smem = smem + NnShared::b_off;
  float* inv_smem = reinterpret_cast<float*>(smem + NnShared::inv_off);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + NnShared::bar_off);
  uint64_t* a_full = bars + 0;
  uint64_t* a_empty = bars + 1;
  uint64_t* b_full = bars + 2;
  uint64_t* b_empty = bars + 2 + kNnStages;
  uint64_t* t_full = bars + 2 + 2 * kNnStages;
  uint64_t* t_empty = t_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + NnShared::misc_off);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + NnShared::misc_off + 4);

  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int S = min(budget_row[0], cap);
  if (S <= 0 || S >= n) return;                      // nothing to merge (uniform across the grid)
  const int n_tiles = (S + kNnTileN - 1) / kNnTileN;
  const int m_blocks = (n + kNnBlockM - 1) / kNnBlockM;
  const int n_items = m_blocks * n_heads;

  if (threadIdx.x == 0) {
    mbar_init(a_full, 1);
    mbar_init(a_empty, 1);
    for (int s = 0; s < kNnStages; ++s) { mbar_init(b_full + s, 1); mbar_init(b_empty + s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(t_full + b, 1); mbar_init(t_empty + b, kNnEpilogueThreads / 32); }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kNnTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_descriptor(&map_k);
      tma_prefetch_descriptor(&map_kc);
      uint32_t b_count = 0, item_count = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++item_count) {
        const int g = item / m_blocks, m0 = (item % m_blocks) * kNnBlockM;
        ok = mbar_wait(a_empty, (item_count & 1u) ^ 1u, abort_flag);
        if (!ok) break;
        mbar_expect_tx(a_full, kNnABytes);
        for (int t = 0; t < 2; ++t)
          for (int kh = 0; kh < 2; ++kh)
            tma_load_3d(a_smem + (t * 2 + kh) * kNnHalfTile, &map_k, a_full, kh * 64, m0 + t * 128, g);
        for (int tile = 0; tile < n_tiles; ++tile, ++b_count) {
          const uint32_t stage = b_count % kNnStages, phase = (b_count / kNnStages) & 1u;
          ok = mbar_wait(b_empty + stage, phase ^ 1u, abort_flag);
          if (!ok) break;
          mbar_expect_tx(b_full + stage, kNnBBytes);
          for (int kh = 0; kh < 2; ++kh)
            tma_load_3d(b_smem + stage * kNnBBytes + kh * kNnHalfTile, &map_kc, b_full + stage, kh * 64,
                        tile * kNnTileN, g);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(128, kNnTileN);
      uint32_t b_count = 0, item_count = 0, t_count = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++item_count) {
        ok = mbar_wait(a_full, item_count & 1u, abort_flag);
        if (!ok) break;
        for (int tile = 0; tile < n_tiles; ++tile, ++b_count, ++t_count) {
          const uint32_t stage = b_count % kNnStages, phase = (b_count / kNnStages) & 1u;
          const uint32_t buf = t_count & 1u, tphase = (t_count >> 1) & 1u;
          ok = mbar_wait(b_full + stage, phase, abort_flag) && mbar_wait(t_empty + buf, tphase ^ 1u, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t b_addr = smem_u32(b_smem + stage * kNnBBytes);
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            const uint32_t d_tmem = tmem_base + buf * 256u + t * 128u;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              const uint32_t kh = kk / 4, koff = (kk % 4) * 32;
              const uint64_t da = umma_desc_k_sw128(smem_u32(a_smem + (t * 2 + kh) * kNnHalfTile), koff);
              const uint64_t db = umma_desc_k_sw128(b_addr + kh * kNnHalfTile, koff);
              umma_bf16(d_tmem, da, db, idesc, kk > 0 ? 1u : 0u);
            }
          }
          umma_commit(b_empty + stage);     // the B stage may be refilled once these UMMAs have read it
          umma_commit(t_full + buf);        // the accumulators of this tile are complete
        }
        if (ok) umma_commit(a_empty);       // the A block may be replaced once the item's UMMAs are done
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue: running arg-max
    const int quarter = warp % 4;                 // TMEM lanes this warp may read: 32 * (warp % 4) ..
    const int t = (warp - 2) / 4;                 // which 128-row UMMA tile
    const int row_in_block = t * 128 + quarter * 32 + lane;
    uint32_t t_count = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      const int g = item / m_blocks, m0 = (item % m_blocks) * kNnBlockM;
      const float* inv_g = inv_norm + (size_t)g * inv_stride;
      float best = -INFINITY;
      int best_slot = 0;
      for (int tile = 0; tile < n_tiles; ++tile, ++t_count) {
        const uint32_t buf = t_count & 1u, tphase = (t_count >> 1) & 1u;
        const int c0 = tile * kNnTileN;
        // this warp's private copy of the tile's 128 inverse norms (no cross-warp barrier needed);
        // the array is padded so that a whole slice can always be read
        float* inv_t = inv_smem + (warp - 2) * kNnTileN;
        reinterpret_cast<float4*>(inv_t)[lane] = __ldg(reinterpret_cast<const float4*>(inv_g + c0) + lane);
        __syncwarp();
        ok = mbar_wait(t_full + buf, tphase, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after_sync();
        const bool ragged = c0 + kNnTileN > S;
#pragma unroll 1
        for (int chunk = 0; chunk < kNnTileN / 32; ++chunk) {
          float v[32];
          tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * 256u + t * 128u + chunk * 32u, v);
          const float4* inv4 = reinterpret_cast<const float4*>(inv_t + chunk * 32);
          float cmax = -INFINITY;
#pragma unroll
          for (int x = 0; x < 8; ++x) {
            const float4 w = inv4[x];
            v[4 * x + 0] *= w.x; v[4 * x + 1] *= w.y; v[4 * x + 2] *= w.z; v[4 * x + 3] *= w.w;
          }
          if (ragged) {
#pragma unroll
            for (int x = 0; x < 32; ++x) if (c0 + chunk * 32 + x >= S) v[x] = -INFINITY;
          }
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
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(t_empty + buf);
      }
      const int token = m0 + row_in_block;
      if (ok && token < n) token_target[(size_t)g * n + token] = best_slot;
    }
  }

  // ------------------------------------------------------------------ common exit
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kNnTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag != 0) set_status(status, MEDA_ERR_TIMEOUT);
}

}  // namespace meda
