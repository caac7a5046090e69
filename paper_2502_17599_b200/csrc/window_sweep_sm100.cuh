// Phase A, sweep 2 for bf16 / head_dim 128 / window 32 or 64 when a KV head serves several query heads
// (129 .. 256 query rows per KV group): per-key accumulated scores (Eq. 8) and the cross-modal entropy
// (Eq. 4-6) from the row normalisers of sweep 1.
//
// One persistent block per SM walks 256-key blocks; for a block it visits the KV heads one after the other,
// so that the head-averaged text-to-vision attention of a key (Eq. 4 averages over ALL query heads) is
// complete inside the threads that own the key.
//
//  * Keys are the A operand (two 128-key tiles per block and KV head, TMA, ring of stages), the KV group's
//    query rows the B operand (one TMA tile of up to 256 rows, double buffered; the rows' softmax constants
//    travel with it on the same barrier).  One UMMA per K step covers ALL query columns (N = columns), so a
//    128-key unit costs eight instructions; its accumulators fill one of two 256-column halves of tensor
//    memory, and the tensor pipe fills one half while the epilogue reduces the other.
//  * Sixteen epilogue warps, four per scheduler, all on the same unit: warp (q, k) owns the tensor-memory
//    lanes of quarter q (32 keys) and the window rows [k W/4, (k+1) W/4) of every query head.  A thread
//    therefore owns a key for a quarter of the window rows: it keeps that quarter of the key's head-averaged
//    attention across the KV heads (Sum_i a_i ln a_i splits by row, so the four owners never have to meet)
//    and a partial score; the four partial scores of a key are added through shared memory by the k = 0 warp.
//  * One exponential per logit serves both softmaxes (the visual normaliser sits in the exponent's
//    reference, see sweep_coef).  The arithmetic around it works on pairs of window rows with packed fp32
//    instructions (the constants of a pair of columns are stored as one 16-byte entry whose halves are packed
//    operands as they come out of shared memory): the sweep is bound by the instructions it issues before the
//    special-function unit saturates, and for the same reason no exponential is moved to the FMA pipes here
//    (a quarter of them as polynomials made the sweep 6 % slower, half of them 15 %).
//  * The block that finishes last adds the entropy partials of all blocks in a fixed order.
#pragma once

#include <type_traits>

#include "attn_sm100.cuh"
#include "window_stats_sm100.cuh"

namespace meda {

constexpr int kSwEpilogueWarps = 16;
constexpr int kSwThreads = 32 * (2 + kSwEpilogueWarps);
constexpr uint32_t kSwAStage = 2 * kUsHalfTile;            // 128 keys x 128 dims
constexpr uint32_t kSwTmemCols = 512;
constexpr int kSwMaxCols = 256;
constexpr int kSwPartDepth = 4;                            // partial-score buffers in flight

struct WinSweepParams {
  const uint8_t* modality;     // padded to a multiple of 256 (+128) with the value 2
  const float2* vis;           // [Hq * w] per-column constants in the paired layout, see store_sweep_coef
  const float2* text;          // [Hq * w]
  const float* row_stats;      // [Hq][w][4] (the entropy's row count comes from it)
  float* scores;               // [Hkv][n] or null
  float* ent_partial;          // [ceil(n / 128) * 16] or null: one slot per 128-key tile and epilogue warp
  float* entropy_out;          // entropy[layer] or null
  unsigned int* done_counter;  // zero between launches
  int n, hkv, cols;            // cols = group * W
  int n_blocks;                // ceil(n / 256)
  int a_stages;                // key-tile stages that fit beside the query tiles
  float sc2;
  float ln_hq;
};

// Shared memory: key stages, two query buffers (two K halves of cols x 64 each), two constant buffers,
// partial scores, barriers.  Offsets depend on `cols`, so they are computed, not constants.
struct WinSweepSmem {
  uint32_t a_off, b_off, b_bytes, c_off, c_bytes, part_off, bar_off, misc_off, total;
  __host__ __device__ WinSweepSmem(int cols, int a_stages) {
    a_off = 0;
    b_off = a_off + (uint32_t)a_stages * kSwAStage;
    b_bytes = 2u * (uint32_t)cols * 128u;
    c_off = b_off + 2u * b_bytes;
    c_bytes = (uint32_t)cols * 16u;
    part_off = c_off + 2u * c_bytes;
    bar_off = part_off + kSwPartDepth * 3u * 128u * 4u;
    misc_off = bar_off + 8u * (2u * 3u + 2u * 2u + 2u * 2u + kSwPartDepth);
    total = misc_off + 32u;
  }
  __host__ __device__ uint32_t alloc() const { return total + 1024u; }
};

__host__ __device__ inline int win_sweep_a_stages(int cols) { return cols <= 224 ? 3 : 2; }

// Work of one block of the grid, in order.  Whole 256-key blocks are dealt round-robin while every block of the
// grid gets one; the blocks left over for a last, partial round are dealt out in halves (one 128-key tile each),
// so that the grid ends within half a block of each other instead of a whole one.
struct WinSweepItem {
  int blk;        // 256-key block
  int t0, nt;     // first key tile of the block this item covers, and how many (0: nothing, skip)
};
__device__ __forceinline__ bool win_sweep_item(const WinSweepParams& p, int it, WinSweepItem& o) {
  const int grid = (int)gridDim.x;
  const int full_rounds = p.n_blocks / grid;
  if (it < full_rounds) {
    o.blk = (int)blockIdx.x + it * grid;
    o.t0 = 0;
    o.nt = (p.n - o.blk * 256 > 128) ? 2 : 1;
    return true;
  }
  const int left = p.n_blocks - full_rounds * grid;
  const int h = (int)blockIdx.x + (it - full_rounds) * grid;
  if (h >= 2 * left) return false;
  o.blk = full_rounds * grid + h / 2;
  o.t0 = h & 1;
  o.nt = (o.t0 == 0 || p.n - o.blk * 256 > 128) ? 1 : 0;
  return true;
}

template <int W, int MODE>
__global__ void __launch_bounds__(kSwThreads, 1)
window_sweep_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_q,
                    const WinSweepParams p, int* status) {
  using namespace sm100;
  constexpr int R = W / 4;                       // window rows per epilogue thread
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const WinSweepSmem L(p.cols, p.a_stages);
  unsigned char* a_smem = smem + L.a_off;
  unsigned char* b_smem = smem + L.b_off;
  unsigned char* c_smem = smem + L.c_off;
  float* part = reinterpret_cast<float*>(smem + L.part_off);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L.bar_off);
  uint64_t* a_full = bars;
  uint64_t* a_empty = a_full + 3;
  uint64_t* b_full = a_empty + 3;
  uint64_t* b_empty = b_full + 2;
  uint64_t* t_full = b_empty + 2;
  uint64_t* t_empty = t_full + 2;
  uint64_t* x_full = t_empty + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L.misc_off);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L.misc_off + 4);
  int* last_flag = reinterpret_cast<int*>(smem + L.misc_off + 8);
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const uint32_t a_stages = (uint32_t)p.a_stages;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 3; ++s) { mbar_init(a_full + s, 1); mbar_init(a_empty + s, 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(b_full + b, 1);
      mbar_init(b_empty + b, 1 + kSwEpilogueWarps);      // the UMMAs and every epilogue warp (constants) are done with it
      mbar_init(t_full + b, 1);
      mbar_init(t_empty + b, kSwEpilogueWarps);
    }
    for (int d = 0; d < kSwPartDepth; ++d) mbar_init(x_full + d, 12);
    *abort_flag = 0;
    *last_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kSwTmemCols);
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
      tma_prefetch_descriptor(&map_q);
      uint32_t a_cnt = 0, b_cnt = 0;
      bool ok = true;
      WinSweepItem item;
      for (int it = 0; ok && win_sweep_item(p, it, item); ++it) {
        if (item.nt == 0) continue;
        const int blk = item.blk;
        for (int g = 0; ok && g < p.hkv; ++g, ++b_cnt) {
          const uint32_t buf = b_cnt & 1u, bphase = (b_cnt >> 1) & 1u;
          ok = mbar_wait(b_empty + buf, bphase ^ 1u, abort_flag);
          if (!ok) break;
          mbar_expect_tx(b_full + buf, L.b_bytes + L.c_bytes);
          for (int kh = 0; kh < 2; ++kh)
            tma_load_3d(b_smem + buf * L.b_bytes + kh * (L.b_bytes / 2), &map_q, b_full + buf, kh * 64, g * p.cols, 0);
          bulk_load(c_smem + buf * L.c_bytes, p.vis + (size_t)g * p.cols, (uint32_t)p.cols * 8u, b_full + buf);
          bulk_load(c_smem + buf * L.c_bytes + (uint32_t)p.cols * 8u, p.text + (size_t)g * p.cols, (uint32_t)p.cols * 8u,
                    b_full + buf);
          for (int t = item.t0; t < item.t0 + item.nt; ++t, ++a_cnt) {
            const uint32_t stage = a_cnt % a_stages, aphase = (a_cnt / a_stages) & 1u;
            ok = mbar_wait(a_empty + stage, aphase ^ 1u, abort_flag);
            if (!ok) break;
            mbar_expect_tx(a_full + stage, kSwAStage);
            for (int kh = 0; kh < 2; ++kh)
              tma_load_3d(a_smem + stage * kSwAStage + kh * kUsHalfTile, &map_k, a_full + stage, kh * 64,
                          blk * 256 + t * 128, g);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      uint32_t a_cnt = 0, b_cnt = 0, unit = 0;
      const uint32_t idesc = umma_idesc_bf16(128, p.cols);
      const uint32_t b_half16 = (L.b_bytes / 2) >> 4;
      bool ok = true;
      WinSweepItem item;
      for (int it = 0; ok && win_sweep_item(p, it, item); ++it) {
        if (item.nt == 0) continue;
        const int m_tiles = item.nt;
        for (int g = 0; ok && g < p.hkv; ++g, ++b_cnt) {
          const uint32_t buf = b_cnt & 1u, bphase = (b_cnt >> 1) & 1u;
          ok = mbar_wait(b_full + buf, bphase, abort_flag);
          if (!ok) break;
          const uint32_t b_lo = umma_desc_lo_sw128(smem_u32(b_smem + buf * L.b_bytes));
          for (int t = 0; t < m_tiles; ++t, ++a_cnt, ++unit) {
            const uint32_t stage = a_cnt % a_stages, aphase = (a_cnt / a_stages) & 1u;
            const uint32_t slot = unit & 1u, tphase = (unit >> 1) & 1u;
            ok = mbar_wait(a_full + stage, aphase, abort_flag) && mbar_wait(t_empty + slot, tphase ^ 1u, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t a_lo = umma_desc_lo_sw128(smem_u32(a_smem + stage * kSwAStage));
            const uint32_t d_tmem = tmem_base + slot * 256u;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              // K slice kk: half kk / 4 of both tiles, 32-byte step (kk % 4) inside the 128-byte swizzled row
              const uint32_t step = (uint32_t)(kk % 4) * 2u;
              umma_bf16_lohi(d_tmem, a_lo + (uint32_t)(kk / 4) * (kUsHalfTile >> 4) + step,
                             b_lo + (uint32_t)(kk / 4) * b_half16 + step, idesc, kk > 0 ? 1u : 0u);
            }
            umma_commit(a_empty + stage);
            umma_commit(t_full + slot);
          }
          if (ok) umma_commit(b_empty + buf);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int ewarp = warp - 2;
    const int quarter = warp % 4;                 // tensor-memory lanes this warp may read
    const int k = ewarp / 4;                      // quarter of the window rows this warp owns
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const int heads = p.cols / W;                 // query heads per KV head
    // this thread's share of two keys' head-averaged attention, as packed pairs of window rows
    uint64_t abar[2][R / 2];
    float plogp = 0.f;                            // MODE 1
#pragma unroll
    for (int x = 0; x < R / 2; ++x) abar[0][x] = abar[1][x] = f32x2(0.f, 0.f);
    uint32_t b_cnt = 0, unit = 0;
    bool ok = true;

    // One unit: key tile T (0 or 1) of the block against every query column of KV head g.
    auto run_unit = [&](auto tile_tag, int blk, int g, int md, const float4* cvis, const float4* ctext) -> bool {
      constexpr int T = decltype(tile_tag)::value;
      const uint32_t slot = unit & 1u, tphase = (unit >> 1) & 1u;
      const int key_in_tile = quarter * 32 + lane;
      const int j = blk * 256 + T * 128 + key_in_tile;
      const bool valid = j < p.n;
      const int first_row = j - (p.n - W);                   // causal: window rows i >= first_row see key j
      // keys past the prompt's end (zero rows of the last tile) take the masked path too: their exponentials are 0
      const bool masked = __any_sync(0xffffffffu, !valid || first_row > k * R);
      bool good = mbar_wait(t_full + slot, tphase, abort_flag);
      good = __all_sync(0xffffffffu, good);
      if (!good) return false;
      tc_fence_after_sync();
      const uint32_t taddr = lane_addr + slot * 256u + (uint32_t)(k * R);
      auto load = [&](uint32_t (&r)[R], int hl) {
        if constexpr (R == 8) tmem_ld_32x8_issue(taddr + (uint32_t)(hl * W), r);
        else tmem_ld_32x16_issue(taddr + (uint32_t)(hl * W), r);
      };
      // A text key takes the text constants and contributes nothing to the text-to-vision attention.
      // The constants of a pair of columns are one 16-byte entry (-ref, -ref', ratio, ratio'): both halves are
      // operands of packed fp32 instructions as they come out of shared memory.
      const float4* coef = (md == MEDA_VISUAL) ? cvis : ctext;
      const float vf = (valid && md == MEDA_VISUAL) ? 1.f : 0.f;
      const uint64_t vflag = f32x2(vf, vf), sc2x2 = f32x2(p.sc2, p.sc2);
      uint64_t score2 = f32x2(0.f, 0.f);
      // The heads are software-pipelined by hand: the exponentials of head h are issued, then the sums of head
      // h - 1 (whose exponentials have completed meanwhile) are taken, then the columns of head h + 1 are fetched.
      // Issued in program order instead (exponentials, then their sums), every warp would stall on its own
      // special-function results with the unit idle behind it: the four warps of a scheduler leave a barrier
      // together and run in phase, so they cannot cover for each other.
      // The loop is unrolled to its maximum with a uniform branch per head: every offset is a constant.
      // All sums are packed pairs (two window rows per instruction): the sweep is short of issue slots.
      uint32_t ra[R];
      uint64_t e_prev[R / 2];
      float t_prev[MODE == 1 ? R : 1];
      auto consume = [&](int c0) {                           // c0: pair index of the consumed head's first column
#pragma unroll
        for (int x = 0; x < R / 2; ++x) {
          const float4 c = coef[c0 + x];                      // read again rather than kept: registers are short
          score2 = fma_f32x2(e_prev[x], f32x2(c.z, c.w), score2);
          if (MODE == 0) {
            abar[T][x] = fma_f32x2(e_prev[x], vflag, abar[T][x]);
          } else {
            float e0, e1;
            f32x2_split(e_prev[x], e0, e1);
            plogp = fmaf(e0 * vf, fmaf(t_prev[2 * x], kLn2, p.ln_hq), plogp);
            plogp = fmaf(e1 * vf, fmaf(t_prev[2 * x + 1], kLn2, p.ln_hq), plogp);
          }
        }
      };
      load(ra, 0);
#pragma unroll
      for (int hl = 0; hl < kSwMaxCols / W; ++hl) {
        if (hl < heads) {
          tmem_ld_wait();
          tmem_ld_pin_n<R>(ra);
          if (masked) {
#pragma unroll
            for (int x = 0; x < R; ++x) if (!valid || k * R + x < first_row) ra[x] = __float_as_uint(-1e30f);
          }
          uint64_t e_new[R / 2];
          const int c0 = (hl * W + k * R) / 2;               // pair index of this head's first column
#pragma unroll
          for (int x = 0; x < R / 2; ++x) {
            const float4 c = coef[c0 + x];                    // (-ref, -ref', ratio, ratio') of columns 2x and 2x + 1
            float t0, t1;
            f32x2_split(fma_f32x2(sm100::pack_f32x2(ra[2 * x], ra[2 * x + 1]), sc2x2, f32x2(c.x, c.y)), t0, t1);
            e_new[x] = f32x2(fast_exp2(t0), fast_exp2(t1));
            if (MODE == 1) { t_prev[2 * x] = t0; t_prev[2 * x + 1] = t1; }
          }
          if (hl + 1 < heads) load(ra, hl + 1);              // the accumulators of this head are consumed
          if (MODE == 0) {
            if (hl > 0) consume(c0 - W / 2);
#pragma unroll
            for (int x = 0; x < R / 2; ++x) e_prev[x] = e_new[x];
          } else {
            // the per-head entropies need the exponents as well: this mode (not the paper's default) takes
            // its sums at once rather than keep a second set of eight values for one head
#pragma unroll
            for (int x = 0; x < R / 2; ++x) e_prev[x] = e_new[x];
            consume(c0);
          }
        }
      }
      if (MODE == 0) consume(((heads - 1) * W + k * R) / 2);
      float score;
      {
        float s0, s1;
        f32x2_split(score2, s0, s1);
        score = s0 + s1;
      }
      // every column of the unit has been read: hand the accumulators back
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(t_empty + slot);
      // the key's four partial scores meet in the k = 0 warp
      const uint32_t pd = unit % kSwPartDepth, xphase = (unit / kSwPartDepth) & 1u;
      float* pbuf = part + pd * (3 * 128);
      if (k != 0) {
        pbuf[(k - 1) * 128 + key_in_tile] = score;
        __syncwarp();
        if (lane == 0) mbar_arrive(x_full + pd);
      } else {
        good = mbar_wait(x_full + pd, xphase, abort_flag);
        good = __all_sync(0xffffffffu, good);
        if (!good) return false;
        score = ((score + pbuf[key_in_tile]) + pbuf[128 + key_in_tile]) + pbuf[256 + key_in_tile];
        if (p.scores && valid) p.scores[(size_t)g * p.n + j] = score;
      }
      ++unit;
      return true;
    };

    // The modality of this thread's two keys of a block, fetched one block ahead: a load from global memory
    // in front of every unit would stall all sixteen warps for its whole latency.
    const uint8_t* my_mod = p.modality + quarter * 32 + lane;         // the padded map covers whole blocks
    int md_next = 0x0202;                                             // low byte: key tile 0, next byte: key tile 1
    WinSweepItem cur;
    if (win_sweep_item(p, 0, cur)) md_next = my_mod[(size_t)cur.blk * 256] | (my_mod[(size_t)cur.blk * 256 + 128] << 8);
    for (int it = 0; ok && win_sweep_item(p, it, cur); ++it) {
      const int blk = cur.blk;
      const int md_pair = md_next;
      {
        WinSweepItem nxt;
        if (win_sweep_item(p, it + 1, nxt)) md_next = my_mod[(size_t)nxt.blk * 256] | (my_mod[(size_t)nxt.blk * 256 + 128] << 8);
      }
      if (cur.nt == 0) continue;
      for (int g = 0; ok && g < p.hkv; ++g, ++b_cnt) {
        const uint32_t buf = b_cnt & 1u, bphase = (b_cnt >> 1) & 1u;
        ok = mbar_wait(b_full + buf, bphase, abort_flag);           // the constants have landed
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const float4* cvis = reinterpret_cast<const float4*>(c_smem + buf * L.c_bytes);
        const float4* ctext = reinterpret_cast<const float4*>(c_smem + buf * L.c_bytes + (uint32_t)p.cols * 8u);
        if (cur.t0 == 0) ok = run_unit(std::integral_constant<int, 0>(), blk, g, md_pair & 0xff, cvis, ctext);
        if (ok && cur.t0 + cur.nt > 1) ok = run_unit(std::integral_constant<int, 1>(), blk, g, md_pair >> 8, cvis, ctext);
        if (!ok) break;
        __syncwarp();
        if (lane == 0) mbar_arrive(b_empty + buf);                  // this warp no longer reads the constants
      }
      if (!ok) break;
      // all KV heads of the block are in: this warp's share of the entropy sum
      float acc = plogp;
      if (MODE == 0) {
#pragma unroll
        for (int tt = 0; tt < 2; ++tt)
#pragma unroll
          for (int x = 0; x < R / 2; ++x) {
            float a0, a1;
            f32x2_split(abar[tt][x], a0, a1);
            if (a0 > 0.f) acc = fmaf(a0, __logf(a0), acc);
            if (a1 > 0.f) acc = fmaf(a1, __logf(a1), acc);
            abar[tt][x] = f32x2(0.f, 0.f);
          }
      }
      plogp = 0.f;
      acc = warp_sum(acc);
      if (p.ent_partial && lane == 0) {
        // one slot per 128-key tile and warp: an item's sum goes to its first tile, a zero to its second
        p.ent_partial[(size_t)(2 * blk + cur.t0) * kSwEpilogueWarps + ewarp] = acc;
        if (cur.nt > 1) p.ent_partial[(size_t)(2 * blk + 1) * kSwEpilogueWarps + ewarp] = 0.f;
      }
    }
    // once, after the last item (a fence after every item cost a twentieth of the sweep): the partials must be
    // visible to the block that adds them up
    if (p.ent_partial && lane == 0) __threadfence();
  }

  // ------------------------------------------------------------------ common exit
  tc_fence_before_sync();
  __syncthreads();
  drain_after_abort(abort_flag);
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kSwTmemCols);
  }
  const bool aborted = *abort_flag != 0;
  if (threadIdx.x == 0 && aborted) set_status(status, MEDA_ERR_TIMEOUT);
  if (!p.entropy_out || aborted) return;                 // uniform over the block

  // ------------------------------------------------------------------ the last block adds the entropy partials
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned int ticket = atomicAdd(p.done_counter, 1u);
    if (ticket == gridDim.x - 1) {
      *last_flag = 1;
      *p.done_counter = 0u;                              // ready for the next launch
    }
  }
  __syncthreads();
  if (*last_flag == 0) return;
  __threadfence();
  // entropy = -(1 / rows) * sum of the partials, added in a fixed order (thread-strided, then a tree), so that
  // repeated runs give identical bits; rows = window rows that see at least one visual key
  double* red = reinterpret_cast<double*>(smem);         // the key stages are idle by now
  const int n_partials = ((p.n + 127) / 128) * kSwEpilogueWarps;
  double acc = 0.0;
  for (int e = threadIdx.x; e < n_partials; e += kSwThreads) acc += (double)__ldcg(p.ent_partial + e);
  red[threadIdx.x] = acc;
  for (int e = kSwThreads + threadIdx.x; e < 1024; e += kSwThreads) red[e] = 0.0;
  const int rows = __syncthreads_count((int)threadIdx.x < W && p.row_stats[threadIdx.x * 4 + 3] > 0.f);
  for (int o = 512; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *p.entropy_out = rows > 0 ? (float)(-red[0] / (double)rows) : 0.f;
}

}  // namespace meda
