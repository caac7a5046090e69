// Phase A, sweep 1 for bf16 / head_dim 128 / window 32 or 64 (Eq. 4 and Eq. 8 need, for every window
// row, the softmax normalisers over all visible keys and over the visible visual keys).
//
// One persistent block per SM.  An item is (KV group, block of up to 256 query rows, run of 128-key tiles).
//
//  * The query rows are the A operand of the UMMAs and live in TENSOR MEMORY for the whole item (each
//    epilogue thread loads half of its row once and stores it with tcgen05.st): the tensor pipe then reads only
//    the streamed key tile from shared memory.  With both operands in shared memory the operand reads of a
//    128 x 128 x 16 instruction take as long as its arithmetic, and the kernel with an empty epilogue already
//    ran well above the time the keys need to arrive.
//  * Key tiles (128 keys) arrive by TMA through a six-stage ring.
//  * Accumulators are handed over per UNIT = (128-row tile, key tile), 128 columns each, through three
//    rotating slots of tensor memory.  Epilogue group t (eight warps: two per lane quarter, each taking two of
//    the unit's four 32-key chunks) owns row tile t and therefore every other unit; with three slots the tensor
//    pipe always has a free slot to fill while both groups are reducing.  Four epilogue warps per scheduler:
//    while one waits for its accumulators the others keep the special-function unit busy (with two per
//    scheduler a warp's chunk took 650 cycles against the 512 the unit needs for two warps' exponentials).
//  * Every epilogue thread owns one query row for two chunks of every unit and keeps online (max, sum of exp2)
//    over visual and over text keys.  Per 32-key chunk: the chunk maximum by three-input maxima, then one
//    exponential per logit on the special-function unit.  A share of the exponentials can be moved to the FMA
//    pipes (exp2_poly_pair: round-to-nearest split of the exponent, degree-5 polynomial in packed pairs,
//    exponent added as an integer; relative error 2.4e-7, the special-function unit's own is 1.7e-7).  That paid
//    with two epilogue warps per scheduler (a quarter of the exponentials: 5 %); with four the sweep is short of
//    issue slots rather than of exponentials and the share is zero (a quarter: +4 % time, half: +12 %).
//  * The two warps that share a row add their states through shared memory at the end of an item (they meet on
//    an mbarrier with a bounded wait, like every other hand-over here).  The
//    partial normalisers of an item go to global memory, run-major; the pair of warps that completes a set of 32
//    rows over all key runs (counted with one atomic per pair and item) merges them, each warp half of the
//    runs, in run order, and writes the rows' final normalisers together with the per-column constants the
//    second sweep reads.  Which pair does it depends on timing; what it computes does not.
//
// Logits are kept in base-2 units: t = (q.k) * scale * log2(e).
#pragma once

#include "attn_sm100.cuh"
#include "meda_common.cuh"
#include "sm100_primitives.cuh"

namespace meda {

constexpr int kWsStages = 6;
constexpr int kWsEpilogueWarps = 16;                      // two groups of eight: group t reduces row tile t
constexpr int kWsThreads = 32 * (2 + kWsEpilogueWarps);   // warp 0 TMA, warp 1 UMMA issue
constexpr uint32_t kWsStageBytes = 2 * kUsHalfTile;       // 128 keys x 128 dims, bf16, two 64-column halves
constexpr uint32_t kWsTmemCols = 512;
constexpr uint32_t kWsAccBase = 128;                      // columns [0, 128): the query rows, 64 per row tile
constexpr uint32_t kWsSlots = 3;                          // accumulator slots of 128 columns
constexpr int kWsMaxChunks = 64;                          // key runs per (KV group, row block): at most this many partials per row
constexpr int kWsPolyOf8 = 0;                             // exponentials per 8 that take the FMA pipes (none: see below)

struct WinStatsParams {
  const __nv_bfloat16* q;        // [Hq * w][128]: window rows, head-major
  const uint8_t* modality;       // padded to a multiple of 128 with the value 2 (= no key)
  const uint32_t* tile_class;    // per 128-key tile: one byte per 32-key chunk: 0 all text, 1 all visual, 2 mixed / padding
  float* partial;                // [chunks][Hq * w][4]: run-major, a warp's 32 rows of one run are contiguous
  float* row_stats;              // [Hq][w][4]  (written by the merging warps)
  float2* coef_vis;              // [Hq * w]    per-column constants of the second sweep, or null
  float2* coef_text;             // [Hq * w]
  int coef_paired;               // 0: (ref, ratio) per column; 1: (-ref, -ref', ratio, ratio') per pair of columns
  unsigned int* counters;        // [n_groups * row_blocks * 8], zero between launches
  int n, hq, group, w, cols;     // cols = group * w query rows per KV group
  int row_blocks;                // ceil(cols / 256)
  int chunks, tiles_per_chunk, tiles_total;
  float sc2;                     // scale * log2(e)
};

struct WinStatsSmem {
  static constexpr uint32_t b_off = 0;
  static constexpr uint32_t bar_off = b_off + kWsStages * kWsStageBytes;
  static constexpr uint32_t n_bars = 2 * kWsStages + 2 * kWsSlots + 2 + 8;     // + one per pair of warps sharing 32 rows
  static constexpr uint32_t misc_off = bar_off + n_bars * 8;
  static constexpr uint32_t pair_off = misc_off + 16;                  // row states handed from a warp to its partner
  static constexpr uint32_t total = pair_off + 8 * 32 * 16 + 8 * 4;
  static constexpr uint32_t alloc = total + 1024;         // slack for the manual 1024-byte alignment
};

struct WinStatsItem {
  int g, rb, kc;          // KV group, row block, key run
  int b_row;              // first key
  int n_tiles, m_tiles;
};

__device__ __forceinline__ bool win_stats_item(const WinStatsParams& p, int it, WinStatsItem& o) {
  const int idx = blockIdx.x + it * gridDim.x;
  const int per_group = p.row_blocks * p.chunks;
  const int n_groups = p.hq / p.group;
  if (idx >= per_group * n_groups) return false;
  o.g = idx / per_group;
  o.rb = (idx / p.chunks) % p.row_blocks;
  o.kc = idx % p.chunks;
  o.b_row = o.kc * p.tiles_per_chunk * 128;
  o.n_tiles = min(p.tiles_per_chunk, p.tiles_total - o.kc * p.tiles_per_chunk);
  o.m_tiles = (p.cols - o.rb * 256 > 128) ? 2 : 1;
  return o.n_tiles > 0;
}

// 2^t for a pair of non-positive arguments on the FMA pipes: n = round(t) by the magic-number addition,
// f = t - n in [-0.5, 0.5], 2^f by a degree-5 polynomial, 2^n by adding n to the exponent field.
__device__ __forceinline__ uint64_t exp2_poly_pair(uint64_t t2) {
  float t0, t1;
  f32x2_split(t2, t0, t1);
  t0 = fmaxf(t0, -125.f);                               // keeps the exponent field positive; 2^-125 is nothing next to a sum >= 1
  t1 = fmaxf(t1, -125.f);
  const uint64_t t = f32x2(t0, t1);
  constexpr float kMagic = 12582912.f;                  // 1.5 * 2^23: the sum's low mantissa bits hold round(t)
  const uint64_t r = add_f32x2(t, f32x2(kMagic, kMagic));
  const uint64_t n = add_f32x2(r, f32x2(-kMagic, -kMagic));
  const uint64_t f = fma_f32x2(n, f32x2(-1.f, -1.f), t);
  uint64_t y = fma_f32x2(f32x2(1.3400433e-3f, 1.3400433e-3f), f, f32x2(9.6760374e-3f, 9.6760374e-3f));
  y = fma_f32x2(y, f, f32x2(5.5503272e-2f, 5.5503272e-2f));
  y = fma_f32x2(y, f, f32x2(2.4022107e-1f, 2.4022107e-1f));
  y = fma_f32x2(y, f, f32x2(6.9314718e-1f, 6.9314718e-1f));
  y = fma_f32x2(y, f, f32x2(1.0000001f, 1.0000001f));
  float y0, y1, r0, r1;
  f32x2_split(y, y0, y1);
  f32x2_split(r, r0, r1);
  y0 = __int_as_float(__float_as_int(y0) + (__float_as_int(r0) << 23));
  y1 = __int_as_float(__float_as_int(y1) + (__float_as_int(r1) << 23));
  return f32x2(y0, y1);
}

// Online-softmax state of one query row: running (max, sum of exp2) in base-2 logit units, visual and text keys.
struct WinStatsRow {
  float mv, zv, mt, zt;
  __device__ __forceinline__ void reset() {
    mv = mt = -INFINITY;
    zv = zt = 0.f;
  }
  __device__ __forceinline__ static void absorb(float& m, float& z, float t) {
    if (t > m) { z = z * fast_exp2(m - t) + 1.f; m = t; }
    else z += fast_exp2(t - m);
  }
  // 32 consecutive keys of one modality, all visible: the chunk maximum first, then one exponential per key.
  __device__ __forceinline__ void uniform_chunk(const uint32_t (&r)[32], float sc2, bool visual) {
    // four independent chains of three-input maxima
    float u0 = __uint_as_float(r[0]), u1 = __uint_as_float(r[1]), u2 = __uint_as_float(r[2]), u3 = __uint_as_float(r[3]);
#pragma unroll
    for (int x = 4; x < 28; x += 8) {
      u0 = sm100::fmax3(u0, __uint_as_float(r[x]), __uint_as_float(r[x + 1]));
      u1 = sm100::fmax3(u1, __uint_as_float(r[x + 2]), __uint_as_float(r[x + 3]));
      u2 = sm100::fmax3(u2, __uint_as_float(r[x + 4]), __uint_as_float(r[x + 5]));
      u3 = sm100::fmax3(u3, __uint_as_float(r[x + 6]), __uint_as_float(r[x + 7]));
    }
    u0 = sm100::fmax3(u0, __uint_as_float(r[28]), __uint_as_float(r[29]));
    u1 = sm100::fmax3(u1, __uint_as_float(r[30]), __uint_as_float(r[31]));
    const float cm = fmaxf(sm100::fmax3(u0, u1, u2), u3);
    float& m = visual ? mv : mt;
    float& z = visual ? zv : zt;
    const float m_new = fmaxf(m, cm * sc2);
    const uint64_t sc2x2 = f32x2(sc2, sc2), ref2 = f32x2(-m_new, -m_new);
    uint64_t a01 = f32x2(0.f, 0.f), a23 = a01;
#pragma unroll
    for (int x = 0; x < 32; x += 8) {
      // eight logits as four pairs: the last kWsPolyOf8 / 2 pairs on the FMA pipes, the others on the special-function unit
#pragma unroll
      for (int pr = 0; pr < 4; ++pr) {
        const uint64_t tp = fma_f32x2(sm100::pack_f32x2(r[x + 2 * pr], r[x + 2 * pr + 1]), sc2x2, ref2);
        uint64_t e;
        if (pr >= 4 - kWsPolyOf8 / 2) {
          e = exp2_poly_pair(tp);
        } else {
          float t0, t1;
          f32x2_split(tp, t0, t1);
          e = f32x2(fast_exp2(t0), fast_exp2(t1));
        }
        if (pr & 1) a23 = add_f32x2(a23, e); else a01 = add_f32x2(a01, e);
      }
      // the sums so far are complete here: keeps the compiler from issuing all 32 exponentials before the first
      // addition, which needs more registers than a thread of this block can have
      asm volatile("" : "+l"(a01), "+l"(a23));
    }
    float a0, a1, a2, a3;
    f32x2_split(a01, a0, a1);
    f32x2_split(a23, a2, a3);
    z = z * fast_exp2(m - m_new) + ((a0 + a1) + (a2 + a3));
    m = m_new;
  }
};

// (max, sum of exp2) of two disjoint key sets of a row, in base-2 logit units.
__device__ __forceinline__ void merge_mz2(float& m, float& z, float m2, float z2) {
  const float mn = fmaxf(m, m2);
  if (mn == -INFINITY) { m = mn; z = 0.f; return; }
  z = z * fast_exp2(m - mn) + z2 * fast_exp2(m2 - mn);
  m = mn;
}

// Any chunk: per key modality (2 = no key) and visibility.  Only the few chunks where text and visual tokens
// meet, the prompt's last keys (causal boundary) and the padding take this path.  It reads the chunk's
// accumulators itself, eight columns at a time and twice (the maxima of the chunk's visible visual and text keys
// first, then one exponential per key against its modality's maximum), in rolled loops: little code, few
// registers, nothing in local memory.  (Taken key after key with a branch each, or through an array in local
// memory, a single such chunk at the head of the prompt held its block back by a sixth of the sweep.)
// Warp-wide: every lane must call it (tensor-memory loads are .sync.aligned); `valid` lanes update their row.
// `vis_keys` / `text_keys`: bit x set when key j0 + x is a visual / text key (the same for every row); the row's
// own causal limit masks them.
__device__ __forceinline__ void win_stats_mixed_chunk(WinStatsRow& s, bool valid, uint32_t taddr, float sc2, uint32_t vis_keys,
                                                      uint32_t text_keys, int j0, int last_visible) {
  const int n_seen = min(max(last_visible - j0 + 1, 0), 32);
  const uint32_t seen = n_seen >= 32 ? 0xffffffffu : ((1u << n_seen) - 1u);
  const uint32_t vis = valid ? vis_keys & seen : 0u, text = valid ? text_keys & seen : 0u;
  // maxima on the raw accumulators (the scale is positive), scaled once
  float rv = -INFINITY, rt = -INFINITY;
#pragma unroll 1
  for (int x0 = 0; x0 < 32; x0 += 8) {
    uint32_t r[8];
    sm100::tmem_ld_32x8_issue(taddr + (uint32_t)x0, r);
    sm100::tmem_ld_wait();
    sm100::tmem_ld_pin_n<8>(r);
#pragma unroll
    for (int x = 0; x < 8; ++x) {
      rv = fmaxf(rv, (vis >> (x0 + x)) & 1u ? __uint_as_float(r[x]) : -INFINITY);
      rt = fmaxf(rt, (text >> (x0 + x)) & 1u ? __uint_as_float(r[x]) : -INFINITY);
    }
  }
  const float mv = fmaxf(s.mv, rv * sc2), mt = fmaxf(s.mt, rt * sc2);
  float zv = 0.f, zt = 0.f;
#pragma unroll 1
  for (int x0 = 0; x0 < 32; x0 += 8) {
    uint32_t r[8];
    sm100::tmem_ld_32x8_issue(taddr + (uint32_t)x0, r);
    sm100::tmem_ld_wait();
    sm100::tmem_ld_pin_n<8>(r);
#pragma unroll
    for (int x = 0; x < 8; ++x) {
      const bool v = (vis >> (x0 + x)) & 1u, tx = (text >> (x0 + x)) & 1u;
      const float e = (v || tx) ? fast_exp2(fmaf(__uint_as_float(r[x]), sc2, v ? -mv : -mt)) : 0.f;
      zv += v ? e : 0.f;
      zt += tx ? e : 0.f;
    }
  }
  // a modality without a key so far keeps (-inf, 0): its old sum is 0 and is not rescaled
  s.zv = (s.zv > 0.f ? s.zv * fast_exp2(s.mv - mv) : 0.f) + zv;
  s.zt = (s.zt > 0.f ? s.zt * fast_exp2(s.mt - mt) : 0.f) + zt;
  s.mv = mv;
  s.mt = mt;
}

#ifndef WS_MERGE_BATCH
#define WS_MERGE_BATCH 8
#endif
// Partial normalisers of one query row over the key runs [c0, c1), merged in run order: a few runs at a time, their
// maxima first and then the sums against that maximum, so that the exponentials of a batch do not wait for each
// other.  `part` points at the row's entry of run 0; consecutive runs are `stride` entries apart (the layout is
// run-major: the 32 rows of a warp read 512 contiguous bytes per run).  Natural-log units.
// Returns (m, z, m_vis, z_vis).
__device__ __forceinline__ float4 win_stats_merge_runs(const float4* part, size_t stride, int c0, int c1) {
  float m = -INFINITY, mv = -INFINITY, z = 0.f, zv = 0.f;
  constexpr int kBatch = WS_MERGE_BATCH;
#pragma unroll 1
  for (int cb = c0; cb < c1; cb += kBatch) {
    float4 x[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u)
      x[u] = (cb + u < c1) ? __ldcg(part + (size_t)(cb + u) * stride) : make_float4(-INFINITY, 0.f, -INFINITY, 0.f);
    float mb = -INFINITY, mvb = -INFINITY;
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      mb = fmaxf(mb, x[u].x);
      mvb = fmaxf(mvb, x[u].z);
    }
    float zb = 0.f, zvb = 0.f;
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      // a run without a visible (visual) key has the sum 0 and the maximum -inf
      zb += x[u].y > 0.f ? x[u].y * __expf(x[u].x - mb) : 0.f;
      zvb += x[u].w > 0.f ? x[u].w * __expf(x[u].z - mvb) : 0.f;
    }
    merge_mz(m, z, mb, zb);
    merge_mz(mv, zv, mvb, zvb);
  }
  return make_float4(m, z, mv, zv);
}

// Writes a row's final normalisers and the two pairs of constants the second sweep uses for the row's column:
//   vis  = (m_vis * log2e + log2(z_vis * Hq),  Hq * z_vis * exp(m_vis - m_all) / z_all)   for visual keys
//   text = (m_all * log2e,                     1 / z_all)                                 for text keys
// (a row that sees no visual key gets (+huge, 0): its exponentials are 0).
__device__ __forceinline__ void win_stats_write_row(const WinStatsParams& p, int h, int i, float m, float z, float mv,
                                                    float zv) {
  const size_t row = (size_t)h * p.w + i;
  reinterpret_cast<float4*>(p.row_stats)[row] = make_float4(m, z, mv, zv);
  if (p.coef_vis) {
    float2 a = make_float2(1e30f, 0.f);
    if (zv > 0.f) {
      a.x = fmaf(mv, kLog2e, log2f(zv * (float)p.hq));
      a.y = (float)p.hq * zv * expf(mv - m) / z;
    }
    store_sweep_coef(p.coef_vis, row, a, p.coef_paired != 0);
    store_sweep_coef(p.coef_text, row, make_float2(m * kLog2e, 1.f / z), p.coef_paired != 0);
  }
}

__global__ void __launch_bounds__(kWsThreads, 1)
window_stats_kernel(const __grid_constant__ CUtensorMap map_k, const WinStatsParams p, int* status) {
  using namespace sm100;
  using SH = WinStatsSmem;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* b_smem = smem + SH::b_off;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SH::bar_off);
  uint64_t* b_full = bars;
  uint64_t* b_empty = b_full + kWsStages;
  uint64_t* s_full = b_empty + kWsStages;
  uint64_t* s_empty = s_full + kWsSlots;
  uint64_t* a_ready = s_empty + kWsSlots;       // the item's query rows are in tensor memory
  uint64_t* a_free = a_ready + 1;               // the item's UMMAs are done with them
  uint64_t* pair_bar = a_free + 1;              // [8]: the two warps that share 32 rows meet here (bounded waits)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + SH::misc_off);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SH::misc_off + 4);
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kWsStages; ++s) { mbar_init(b_full + s, 1); mbar_init(b_empty + s, 1); }
    for (uint32_t s = 0; s < kWsSlots; ++s) { mbar_init(s_full + s, 1); mbar_init(s_empty + s, kWsEpilogueWarps / 2); }
    mbar_init(a_ready, kWsEpilogueWarps);
    mbar_init(a_free, 1);
    for (int s = 0; s < 8; ++s) mbar_init(pair_bar + s, 2);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kWsTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (key tiles)
    if (lane == 0) {
      tma_prefetch_descriptor(&map_k);
      uint32_t b_count = 0;
      WinStatsItem it;
      bool ok = true;
      for (int i = 0; ok && win_stats_item(p, i, it); ++i) {
        for (int tile = 0; tile < it.n_tiles; ++tile, ++b_count) {
          const uint32_t stage = b_count % kWsStages, phase = (b_count / kWsStages) & 1u;
          ok = mbar_wait(b_empty + stage, phase ^ 1u, abort_flag);
          if (!ok) break;
          mbar_expect_tx(b_full + stage, kWsStageBytes);
          for (int kh = 0; kh < 2; ++kh)
            tma_load_3d(b_smem + stage * kWsStageBytes + kh * kUsHalfTile, &map_k, b_full + stage, kh * 64,
                        it.b_row + tile * 128, it.g);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      uint32_t b_count = 0, unit = 0, item = 0;
      const uint32_t idesc = umma_idesc_bf16(128, 128);
      WinStatsItem it;
      bool ok = true;
      for (int i = 0; ok && win_stats_item(p, i, it); ++i, ++item) {
        ok = mbar_wait(a_ready, item & 1u, abort_flag);
        if (!ok) break;
        for (int tile = 0; tile < it.n_tiles; ++tile, ++b_count) {
          const uint32_t stage = b_count % kWsStages, phase = (b_count / kWsStages) & 1u;
          ok = mbar_wait(b_full + stage, phase, abort_flag);
          if (!ok) break;
          const uint32_t b_lo = umma_desc_lo_sw128(smem_u32(b_smem + stage * kWsStageBytes));
          for (int t = 0; t < it.m_tiles; ++t, ++unit) {
            const uint32_t slot = unit % kWsSlots, sphase = (unit / kWsSlots) & 1u;
            ok = mbar_wait(s_empty + slot, sphase ^ 1u, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + kWsAccBase + slot * 128u;
            const uint32_t a_tmem = tmem_base + (uint32_t)t * 64u;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              // K slice kk: half kk / 4 of the key tile, 32-byte step (kk % 4) inside the 128-byte swizzled row
              const uint32_t off = (uint32_t)(kk / 4) * (kUsHalfTile >> 4) + (uint32_t)(kk % 4) * 2u;
              umma_bf16_a_tmem_lohi(d_tmem, a_tmem + (uint32_t)kk * 8u, b_lo + off, idesc, kk > 0 ? 1u : 0u);
            }
            umma_commit(s_full + slot);
          }
          if (!ok) break;
          umma_commit(b_empty + stage);     // the key tile may be replaced once these UMMAs have read it
        }
        if (ok) umma_commit(a_free);        // the query rows may be replaced once the item's UMMAs are done
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (and loader of the query rows)
    // Warp (t, quarter, half): row tile t, tensor-memory lanes of `quarter`, chunks 2 half and 2 half + 1 of every
    // unit.  Four epilogue warps per scheduler: while one waits for its accumulators the others keep the
    // special-function unit busy.
    const int ewarp = warp - 2;
    const int t = (ewarp / 4) & 1;              // row tile = epilogue group
    const int half = ewarp / 8;                 // which two of a unit's four 32-key chunks
    const int quarter = warp % 4;               // tensor-memory lanes this warp may touch: 32 * (warp % 4) ..
    const int set = t * 4 + ewarp % 4;          // the 32 rows this warp shares with its partner (the other half)
    const int row_in_block = t * 128 + quarter * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    WinStatsRow row;
    uint32_t unit_base = 0, item = 0, pair_uses = 0;
    // The two warps of a pair meet (and see each other's shared-memory writes) through an mbarrier, not a named
    // barrier: like every other wait of the kernel this one gives up when the block is being aborted, so a warp
    // whose partner has left the loop after a failed wait does not wait for it for ever.
    auto pair_sync = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(pair_bar + set);
      bool good = mbar_wait(pair_bar + set, pair_uses & 1u, abort_flag);
      ++pair_uses;
      return __all_sync(0xffffffffu, good);
    };
    WinStatsItem it;
    bool ok = true;
    for (int i = 0; ok && win_stats_item(p, i, it); ++i, ++item) {
      const int r = it.rb * 256 + row_in_block;     // query row inside the KV group
      const bool mine = t < it.m_tiles;
      const bool valid = mine && r < p.cols;
      // ---- half of this thread's query row -> tensor memory, once the previous item's UMMAs are done with it
      ok = mbar_wait(a_free, (item & 1u) ^ 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      if (mine) {
        const uint4* src = reinterpret_cast<const uint4*>(p.q + ((size_t)it.g * p.cols + min(r, p.cols - 1)) * kFastDim);
        uint32_t a[32];
#pragma unroll
        for (int x = 0; x < 8; ++x) {
          const uint4 v = valid ? __ldg(src + half * 8 + x) : make_uint4(0u, 0u, 0u, 0u);
          a[4 * x + 0] = v.x; a[4 * x + 1] = v.y; a[4 * x + 2] = v.z; a[4 * x + 3] = v.w;
        }
        tmem_st_32x32(lane_addr + (uint32_t)t * 64u + (uint32_t)half * 32u, a);
        tmem_st_wait();
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(a_ready);

      // ---- the item's units of this group
      row.reset();
      const int i_win = r % p.w;
      const int last_visible = p.n - p.w + i_win;     // causal: keys j <= last_visible
      if (mine) {
        const int tile0 = it.b_row / 128;
        uint32_t cls = __ldg(p.tile_class + tile0);
        for (int tile = 0; tile < it.n_tiles; ++tile) {
          const uint32_t unit = unit_base + (uint32_t)(tile * it.m_tiles + t);
          const uint32_t slot = unit % kWsSlots, sphase = (unit / kWsSlots) & 1u;
          const uint32_t cls_now = cls;
          if (tile + 1 < it.n_tiles) cls = __ldg(p.tile_class + tile0 + tile + 1);   // in flight during this unit
          ok = mbar_wait(s_full + slot, sphase, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t taddr = lane_addr + kWsAccBase + slot * 128u + (uint32_t)half * 64u;
          const int c0 = it.b_row + tile * 128 + half * 64;
          uint32_t ra[32];
#pragma unroll 1
          for (int c = 0; c < 2; ++c) {
            const uint32_t cl = (cls_now >> (8 * (2 * half + c))) & 0xffu;
            const int j0 = c0 + 32 * c;
            // uniform over the warp: the branches below hold warp-wide (.sync.aligned) tensor-memory loads
            const bool fast = __all_sync(0xffffffffu, !valid || (cl < 2u && j0 + 31 <= last_visible));
            if (fast) {
              tmem_ld_32x32_issue(taddr + 32u * c, ra);
              tmem_ld_wait();
              tmem_ld_pin(ra);
            } else {
              const int md = p.modality[j0 + lane];          // the map is padded: 2 = no key
              const uint32_t vis_keys = __ballot_sync(0xffffffffu, md == MEDA_VISUAL);
              const uint32_t text_keys = __ballot_sync(0xffffffffu, md == MEDA_TEXT);
              win_stats_mixed_chunk(row, valid, taddr + 32u * c, p.sc2, vis_keys, text_keys, j0, last_visible);
            }
            if (c == 1) {
              // this warp's share of the unit has been read: hand the slot back before the last chunk is reduced
              tc_fence_before_sync();
              __syncwarp();
              if (lane == 0) mbar_arrive(s_empty + slot);
            }
            if (fast && valid) row.uniform_chunk(ra, p.sc2, cl == 1u);
          }
        }
      }
      if (!ok) break;
      unit_base += (uint32_t)(it.n_tiles * it.m_tiles);

      // ---- the two halves of a row meet in the half-0 warp (through shared memory)
      float4* pair_state = reinterpret_cast<float4*>(smem + SH::pair_off) + set * 32 + lane;
      volatile int* pair_flag = reinterpret_cast<volatile int*>(smem + SH::pair_off + 8 * 32 * 16) + set;
      if (half == 1) *pair_state = make_float4(row.mv, row.zv, row.mt, row.zt);
      ok = pair_sync();
      if (!ok) break;
      if (half == 0) {
        const float4 o = *pair_state;
        merge_mz2(row.mv, row.zv, o.x, o.y);
        merge_mz2(row.mt, row.zt, o.z, o.w);
      }

      // ---- partial normalisers of the item; the pair of warps that completes its 32 rows merges them
      const size_t rows_total = (size_t)p.hq * p.w;
      const int h = it.g * p.group + min(r, p.cols - 1) / p.w;
      float4* my_part = reinterpret_cast<float4*>(p.partial) + (size_t)h * p.w + i_win;     // run 0 of this row
      bool last = false;
      if (mine && half == 0) {
        if (valid) {
          const float m_all = fmaxf(row.mv, row.mt);
          float z_all = 0.f;
          if (m_all > -INFINITY) z_all = row.zv * fast_exp2(row.mv - m_all) + row.zt * fast_exp2(row.mt - m_all);
          my_part[(size_t)it.kc * rows_total] = make_float4(m_all * kLn2, z_all, row.mv * kLn2, row.zv);
        }
        __threadfence();
        __syncwarp();
        unsigned int ticket = 0;
        if (lane == 0) ticket = atomicAdd(p.counters + ((size_t)(it.g * p.row_blocks + it.rb) * 8 + set), 1u);
        ticket = __shfl_sync(0xffffffffu, ticket, 0);
        last = ticket == (unsigned int)p.chunks - 1u;      // every key run of these rows has been written
        if (lane == 0) *pair_flag = last ? 1 : 0;
      }
      ok = pair_sync();
      if (!ok) break;
      last = *pair_flag != 0;                              // uniform over the pair of warps
      if (last) {
        // each warp of the pair merges half of the key runs, the half-0 warp joins the halves and writes the row
        __threadfence();
        const int c_mid = (p.chunks + 1) / 2;
        float4 mine4 = make_float4(-INFINITY, 0.f, -INFINITY, 0.f);
        if (valid) mine4 = win_stats_merge_runs(my_part, rows_total, half ? c_mid : 0, half ? p.chunks : c_mid);
        if (half == 1) *pair_state = mine4;
        ok = pair_sync();
        if (!ok) break;
        if (half == 0) {
          if (valid) {
            const float4 o = *pair_state;
            merge_mz(mine4.x, mine4.y, o.x, o.y);
            merge_mz(mine4.z, mine4.w, o.z, o.w);
            win_stats_write_row(p, h, i_win, mine4.x, mine4.y, mine4.z, mine4.w);
          }
          if (lane == 0) p.counters[(size_t)(it.g * p.row_blocks + it.rb) * 8 + set] = 0u;     // ready for the next launch
        }
      }
    }
  }

  // ------------------------------------------------------------------ common exit
  tc_fence_before_sync();
  __syncthreads();
  drain_after_abort(abort_flag);
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kWsTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag != 0) set_status(status, MEDA_ERR_TIMEOUT);
}

}  // namespace meda
