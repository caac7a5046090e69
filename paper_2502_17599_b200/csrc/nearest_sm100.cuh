// Phase B, merge step 1 for bf16 / head_dim 128 (Eq. 11 and the arg-max that follows it), with the
// token rows held in TENSOR MEMORY as the A operand of the UMMAs.
//
// The contraction is only K = 128 deep, so every accumulator is read back after eight instructions
// and the read-back (tcgen05.ld), the inverse-norm loads and the UMMAs' shared-memory operand reads
// all go through the same per-SM data path.  With both operands in shared memory that path
// saturates at well under half the tensor rate.  Here a persistent block owns 256 consecutive entries
// of a head's less-important list (two 128-row UMMA tiles): every epilogue thread reads half of its
// own row straight from the caller's key cache, by index, so the large operand needs no gather pass
// and no conserved row is swept, and stores it with tcgen05.st; the rows stay in tensor memory for the whole
// sweep over the conserved slots, and the UMMAs read only the 96-slot B tiles (TMA from the
// gathered conserved keys, a six-stage ring) from shared memory.
//
//   tensor memory (512 columns): [0, 128) A, 64 columns per 128-row tile; then two accumulator
//   buffers of 2 x 96 columns.
//   warp 0: TMA producer; warps 1 and 2: UMMA issuers, one per 128-row tile (a single thread cannot
//   issue these short instructions as fast as the tensor pipe retires them); warps 3..18: epilogue,
//   two groups of eight.  Group g
//   reads accumulator buffer g, i.e. every other tile, so two tiles are being reduced at any time;
//   the groups' running maxima are combined through shared memory at the end of each row block.
#pragma once

#include "meda_common.cuh"
#include "sm100_primitives.cuh"

namespace meda {

constexpr int kNtDim = 128;                             // head_dim of this path
constexpr int kNtTileN = 96;                            // conserved slots per streamed tile (UMMA N)
constexpr int kNtStages = 6;
constexpr int kNtGroupWarps = 8;                        // epilogue warps per accumulator buffer
constexpr int kNtEpilogueWarps = 2 * kNtGroupWarps;
constexpr int kNtFirstEpilogueWarp = 3;                 // warp 0 TMA, warps 1 and 2 UMMA (one per row tile)
constexpr int kNtThreads = 32 * (kNtFirstEpilogueWarp + kNtEpilogueWarps);
constexpr uint32_t kNtHalf = kNtTileN * 64 * 2;         // one 96-row x 64-column bf16 TMA box (12 KB)
constexpr uint32_t kNtStageBytes = 2 * kNtHalf;
constexpr uint32_t kNtTmemCols = 512;
constexpr uint32_t kNtAccBase = 128;                    // first accumulator column
constexpr uint32_t kNtAccBuf = 2 * kNtTileN;            // columns per accumulator buffer
// Layers that keep at most this many slots take the streaming kernel of nearest_small_sm100.cuh instead: with
// one to three slot tiles per row block, loading the rows by index into tensor memory dominates here.  Beyond
// that the streaming kernel loses: its UMMAs read both operands from shared memory (measured break-even
// between 350 and 600 slots, depending on the number of KV heads).
constexpr int kNearestSmallMaxS = 384;

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
    const uint2* src = reinterpret_cast<const uint2*>(k + ((size_t)g * n + row) * kNtDim);
    uint2 x = src[lane];
    reinterpret_cast<uint2*>(kc + ((size_t)g * kc_rows + slot) * kNtDim)[lane] = x;
    float2 a = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&x.x));
    float2 b = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&x.y));
    float ss = a.x * a.x + a.y * a.y + b.x * b.x + b.y * b.y;
    ss = warp_sum(ss);
    if (lane == 0) inv_norm[(size_t)g * inv_stride + slot] = 1.f / fmaxf(sqrtf(ss), kCosEps);
  }
}

struct NearestParams {
  const __nv_bfloat16* k;        // [heads][n][128]
  const float* inv_norm;         // [heads][inv_stride]
  const int32_t* budget_row;     // (S, M, N) of the layer
  const int32_t* idx_less;       // [heads][n]: the n - S less-important token rows of every head
  int32_t* target;               // [heads][n]: slot chosen for idx_less[g][p]
  int n, n_heads, cap, inv_stride;
};

struct NearestSmem {
  static constexpr uint32_t b_off = 0;
  static constexpr uint32_t inv_off = b_off + kNtStages * kNtStageBytes;
  static constexpr uint32_t comb_off = inv_off + kNtEpilogueWarps * kNtTileN * 4;   // [2][256] (value, slot)
  static constexpr uint32_t bar_off = comb_off + 2 * 256 * 8;
  static constexpr uint32_t n_bars = 2 * kNtStages + 7;
  static constexpr uint32_t misc_off = bar_off + n_bars * 8;
  static constexpr uint32_t total = misc_off + 16;
  static constexpr uint32_t alloc = total + 1024;       // slack for the manual 1024-byte alignment
};

// Running arg-max of one token row over the slots it has seen.
struct NearestRow {
  float best;
  int best_slot;
  // One chunk = this thread's row against 32 consecutive slots starting at s0: scale by the slots'
  // inverse norms (two products per instruction), reduce with three-input maxima, and only when the
  // chunk beats the running best look for the first slot that attains it.
  __device__ __forceinline__ void chunk(const uint32_t (&r)[32], const float* inv32, int s0, int S, bool ragged) {
    const ulonglong2* inv2 = reinterpret_cast<const ulonglong2*>(inv32);
    float v[32];
#pragma unroll
    for (int x = 0; x < 8; ++x) {
      const ulonglong2 w = inv2[x];
      sm100::mul_f32x2(sm100::pack_f32x2(r[4 * x + 0], r[4 * x + 1]), w.x, v[4 * x + 0], v[4 * x + 1]);
      sm100::mul_f32x2(sm100::pack_f32x2(r[4 * x + 2], r[4 * x + 3]), w.y, v[4 * x + 2], v[4 * x + 3]);
    }
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
      // First slot that attains the maximum.  The four sub-maxima of the reduction tree say which
      // nine-column group holds it, so only that group is scanned; the few lanes that improve in a
      // chunk rarely sit in more than one or two groups, which is what the warp pays for.
      int first;
      if (u0 == cmax) {
        first = 8;
#pragma unroll
        for (int x = 7; x >= 0; --x) if (v[x] == cmax) first = x;
      } else if (u1 == cmax) {
        first = 17;
#pragma unroll
        for (int x = 16; x >= 9; --x) if (v[x] == cmax) first = x;
      } else if (u2 == cmax) {
        first = 26;
#pragma unroll
        for (int x = 25; x >= 18; --x) if (v[x] == cmax) first = x;
      } else {
        first = 31;
#pragma unroll
        for (int x = 30; x >= 27; --x) if (v[x] == cmax) first = x;
      }
      best = cmax;
      best_slot = s0 + first;
    }
  }
};

__global__ void __launch_bounds__(kNtThreads, 1)
nearest_kernel(const __grid_constant__ CUtensorMap map_kc, const NearestParams p, int* status) {
  using namespace sm100;
  using SH = NearestSmem;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* b_smem = smem + SH::b_off;
  float* inv_smem = reinterpret_cast<float*>(smem + SH::inv_off);
  float2* comb = reinterpret_cast<float2*>(smem + SH::comb_off);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SH::bar_off);
  uint64_t* b_full = bars;
  uint64_t* b_empty = b_full + kNtStages;
  uint64_t* t_full = b_empty + kNtStages;
  uint64_t* t_empty = t_full + 2;
  uint64_t* a_full = t_empty + 2;
  uint64_t* a_empty = a_full + 1;
  uint64_t* c_full = a_empty + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + SH::misc_off);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SH::misc_off + 4);

  // work of this launch, from the layer's budget row (uniform over the grid)
  const int S = min(p.budget_row[0], p.cap);
  if (S <= kNearestSmallMaxS || S >= p.n) return;                  // nothing to merge, or the streaming kernel's layer
  // only the less-important rows are swept: a row block is 256 consecutive entries of the head's list
  const int n_less = p.n - S;
  const int m_blocks = (n_less + 255) / 256;
  const int n_items = m_blocks * p.n_heads;
  const int n_tiles = (S + kNtTileN - 1) / kNtTileN;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;

  if (threadIdx.x == 0) {
    // two UMMA issuers: whatever they release takes one commit from each
    for (int s = 0; s < kNtStages; ++s) { mbar_init(b_full + s, 1); mbar_init(b_empty + s, 2); }
    for (int b = 0; b < 2; ++b) { mbar_init(t_full + b, 2); mbar_init(t_empty + b, kNtGroupWarps); }
    mbar_init(a_full, kNtEpilogueWarps);
    mbar_init(a_empty, 2);
    mbar_init(c_full, kNtGroupWarps);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kNtTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (B tiles)
    if (lane == 0) {
      tma_prefetch_descriptor(&map_kc);
      uint32_t b_count = 0;
      bool ok = true;
      for (int idx = blockIdx.x; ok && idx < n_items; idx += gridDim.x) {
        const int head = idx / m_blocks;
        for (int tile = 0; tile < n_tiles; ++tile, ++b_count) {
          const uint32_t stage = b_count % kNtStages, phase = (b_count / kNtStages) & 1u;
          ok = mbar_wait(b_empty + stage, phase ^ 1u, abort_flag);
          if (!ok) break;
          mbar_expect_tx(b_full + stage, kNtStageBytes);
          for (int kh = 0; kh < 2; ++kh)
            tma_load_3d(b_smem + stage * kNtStageBytes + kh * kNtHalf, &map_kc, b_full + stage, kh * 64,
                        tile * kNtTileN, head);
        }
      }
    }
  } else if (warp < kNtFirstEpilogueWarp) {
    // ------------------------------------------------------------------ UMMA issuers: warp 1 + t issues row tile t
    if (lane == 0) {
      const int t = warp - 1;
      uint32_t b_count = 0, t_count = 0, item = 0;
      const uint32_t idesc = umma_idesc_bf16(128, kNtTileN);
      bool ok = true;
      for (int idx = blockIdx.x; ok && idx < n_items; idx += gridDim.x, ++item) {
        const int a_row = (idx % m_blocks) * 256;
        const int m_tiles = (n_less - a_row > 128) ? 2 : 1;
        ok = mbar_wait(a_full, item & 1u, abort_flag);              // the rows are in tensor memory
        if (!ok) break;
        for (int tile = 0; tile < n_tiles; ++tile, ++b_count, ++t_count) {
          const uint32_t stage = b_count % kNtStages, phase = (b_count / kNtStages) & 1u;
          const uint32_t buf = t_count & 1u, tphase = (t_count >> 1) & 1u;
          ok = mbar_wait(b_full + stage, phase, abort_flag) && mbar_wait(t_empty + buf, tphase ^ 1u, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t b_lo = umma_desc_lo_sw128(smem_u32(b_smem + stage * kNtStageBytes));
          if (t < m_tiles) {
            const uint32_t d_tmem = tmem_base + kNtAccBase + buf * kNtAccBuf + (uint32_t)t * kNtTileN;
            const uint32_t a_tmem = tmem_base + (uint32_t)t * 64u;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              // K slice kk: half kk / 4 of the tile, 32-byte step (kk % 4) inside the 128-byte swizzled row
              const uint32_t off = (uint32_t)(kk / 4) * (kNtHalf >> 4) + (uint32_t)(kk % 4) * 2u;
              umma_bf16_a_tmem_lohi(d_tmem, a_tmem + (uint32_t)kk * 8u, b_lo + off, idesc, kk > 0 ? 1u : 0u);
            }
          }
          umma_commit(b_empty + stage);     // the B stage may be refilled once these UMMAs have read it
          umma_commit(t_full + buf);        // the accumulators of this tile are complete
        }
        if (ok) umma_commit(a_empty);       // the rows may be replaced once the item's UMMAs are done
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (and A loader)
    // Inside a group, warp e covers the 32 tensor-memory lanes (warp % 4) * 32.. of row tile e / 4.
    const int ewarp = warp - kNtFirstEpilogueWarp;
    const int group = ewarp / kNtGroupWarps;
    const int quarter = warp % 4;
    const int t = (ewarp % kNtGroupWarps) / 4;
    const int row_in_block = t * 128 + quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    float* inv_t = inv_smem + ewarp * kNtTileN;
    NearestRow row;
    uint32_t t_count = 0, item = 0;
    bool ok = true;
    for (int idx = blockIdx.x; ok && idx < n_items; idx += gridDim.x, ++item) {
      const int head = idx / m_blocks;
      const int a_row = (idx % m_blocks) * 256;
      const int m_tiles = (n_less - a_row > 128) ? 2 : 1;
      const int pos = a_row + row_in_block;          // position in the less-important list
      const bool live = t < m_tiles && pos < n_less;
      // ---- half of this thread's key row -> tensor memory (once the previous item's UMMAs are done
      // with it): group g stores elements [64 g, 64 g + 64), tensor-memory columns [32 g, 32 g + 32)
      ok = mbar_wait(a_empty, (item & 1u) ^ 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      if (t < m_tiles) {
        uint32_t a[32];
        if (live) {
          const int token = min(max(p.idx_less[(size_t)head * p.n + pos], 0), p.n - 1);
          const uint4* src = reinterpret_cast<const uint4*>(p.k + ((size_t)head * p.n + token) * kNtDim) + group * 8;
#pragma unroll
          for (int x = 0; x < 8; ++x) {
            const uint4 q = __ldg(src + x);
            a[4 * x + 0] = q.x; a[4 * x + 1] = q.y; a[4 * x + 2] = q.z; a[4 * x + 3] = q.w;
          }
        } else {
#pragma unroll
          for (int x = 0; x < 32; ++x) a[x] = 0u;
        }
        tmem_st_32x32(lane_addr + (uint32_t)t * 64u + (uint32_t)group * 32u, a);
        tmem_st_wait();
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(a_full);
      // ---- sweep of the conserved slots: this group's tiles
      row.best = -INFINITY;
      row.best_slot = 0;
      const float* inv_g = p.inv_norm + (size_t)head * p.inv_stride;
      for (int tile = 0; tile < n_tiles; ++tile, ++t_count) {
        if ((int)(t_count & 1u) != group) continue;
        const uint32_t tphase = (t_count >> 1) & 1u;
        const int c0 = tile * kNtTileN;
        // this warp's private copy of the tile's inverse norms (the array is padded so that a whole
        // slice can always be read); loaded while the UMMAs of the tile are still running
        __syncwarp();
        if (lane < kNtTileN / 4)
          reinterpret_cast<float4*>(inv_t)[lane] = __ldg(reinterpret_cast<const float4*>(inv_g + c0) + lane);
        __syncwarp();
        ok = mbar_wait(t_full + group, tphase, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after_sync();
        if (t < m_tiles) {
          const uint32_t taddr = lane_addr + kNtAccBase + (uint32_t)group * kNtAccBuf + (uint32_t)t * kNtTileN;
          const bool ragged = c0 + kNtTileN > S;
          // two register buffers: the load of chunk c + 1 is in flight while chunk c is reduced
          uint32_t ra[32], rb[32];
          tmem_ld_32x32_issue(taddr, ra);
          tmem_ld_wait();
          tmem_ld_pin(ra);
          tmem_ld_32x32_issue(taddr + 32u, rb);
          row.chunk(ra, inv_t, c0, S, ragged);
          tmem_ld_wait();
          tmem_ld_pin(rb);
          tmem_ld_32x32_issue(taddr + 64u, ra);
          row.chunk(rb, inv_t + 32, c0 + 32, S, ragged);
          tmem_ld_wait();
          tmem_ld_pin(ra);
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(t_empty + group);   // the accumulators are in registers: release them early
          row.chunk(ra, inv_t + 64, c0 + 64, S, ragged);
        } else {
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(t_empty + group);
        }
      }
      if (!ok) break;
      // ---- the two groups saw disjoint tiles: group 1 hands its result over, group 0 keeps the larger
      // value (equal values: the lower slot) and writes the row's target
      float2* cb = comb + (item & 1u) * 256;
      if (group == 1) {
        cb[row_in_block] = make_float2(row.best, __int_as_float(row.best_slot));
        __syncwarp();
        if (lane == 0) mbar_arrive(c_full);
      } else {
        ok = mbar_wait(c_full, item & 1u, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const float2 other = cb[row_in_block];
        const int oslot = __float_as_int(other.y);
        if (other.x > row.best || (other.x == row.best && oslot < row.best_slot)) row.best_slot = oslot;
        if (live) p.target[(size_t)head * p.n + pos] = row.best_slot;
      }
    }
  }

  // ------------------------------------------------------------------ common exit
  tc_fence_before_sync();
  __syncthreads();
  drain_after_abort(abort_flag);
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kNtTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag != 0) set_status(status, MEDA_ERR_TIMEOUT);
}

}  // namespace meda
