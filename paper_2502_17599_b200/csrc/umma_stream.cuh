// Persistent "resident block x streamed tiles" tcgen05 pipeline shared by the tensor-core kernels.
//
// A work item is a block of up to 256 operand-A rows (two 128-row UMMA tiles, bf16, 128 columns,
// loaded once by TMA) contracted against a run of operand-B tiles of up to 128 rows each (streamed
// by TMA through a ring).  Accumulators (fp32, 128 lanes x up to 128 columns per UMMA tile) live in
// tensor memory and are double buffered, so the UMMAs of tile i+1 overlap the epilogue of tile i.
//
//   warp 0      : TMA producer (one elected lane)
//   warp 1      : tensor-memory owner and UMMA issuer (one elected lane)
//   warps 2..9  : epilogue; warp e reads the 32 TMEM lanes (warp % 4) * 32.. of UMMA tile (e / 4)
//   warps 10..17: (policies with kEpilogueGroups = 2) a second epilogue group with the same lane map.
//                 Group g then reduces accumulator buffer g, i.e. every other streamed tile, so two
//                 tiles are in the epilogue at any time; the policy combines what the two groups hold.
//
// What an item is and what the epilogue does with the accumulators is supplied by a policy type:
//
//   struct Policy {
//     struct Params;                                  // trivially copyable kernel argument
//     static constexpr int kABuffers, kBStages;       // resident-block buffers (1 or 2), B ring depth
//     static constexpr int kEpilogueGroups;           // 1 or 2 groups of eight epilogue warps
//     static constexpr uint32_t kExtraBytes;          // policy-owned shared memory
//     static constexpr uint32_t kItemExtraBytes;      // per-item side data (multiple of 128), or 0; when
//                                                     // non-zero it is bulk-copied next to the resident
//                                                     // block, one copy per A buffer, and released with it:
//     static uint32_t item_extra_bytes(const Params&, const StreamItem&);              // bytes of this item
//     static void item_extra_issue(const Params&, const StreamItem&, unsigned char* dst, uint64_t* bar);
//     static bool active(const Params&);              // false: the whole grid returns at once
//     static bool get_item(const Params&, int it, StreamItem&);   // it-th item of this block, or false
//     struct Epilogue {                               // one object per epilogue thread
//       void init(const Params&, unsigned char* extra, int ewarp, int lane);   // ewarp 0..8 * groups - 1
//       void item_begin(const Params&, const StreamItem&, const unsigned char* item_extra);
//       void tile(const Params&, const StreamItem&, int tile, uint32_t taddr);   // taddr: this warp's lanes
//       void item_end(const Params&, const StreamItem&);
//     };
//   };
//
// Every wait is bounded (see sm100_primitives.cuh): when one runs out all roles leave their loops,
// tensor memory is released and MEDA_ERR_TIMEOUT is recorded.
#pragma once

#include "meda_common.cuh"
#include "sm100_primitives.cuh"

namespace meda {

constexpr int kFastDim = 128;                         // head_dim of the tensor-core paths
constexpr int kUsEpilogueWarps = 8;                   // per epilogue group
template <class P>
constexpr int us_threads() { return 64 + 32 * kUsEpilogueWarps * P::kEpilogueGroups; }
constexpr uint32_t kUsHalfTile = 128 * 64 * 2;        // one 128-row x 64-column bf16 TMA box (16 KB)
constexpr uint32_t kUsABlock = 4 * kUsHalfTile;       // 2 UMMA tiles x 2 K halves
constexpr uint32_t kUsBStage = 2 * kUsHalfTile;       // 1 tile x 2 K halves
constexpr uint32_t kUsTmemCols = 512;

struct StreamItem {
  int a_row, a_head;      // TMA coordinates of the resident block: rows a_row .. a_row + 128 * m_tiles
  int b_row, b_head;      // first row of streamed tile 0; tile t starts at b_row + 128 * t
  int n_tiles;            // streamed tiles of this item (>= 1)
  int last_n;             // UMMA N of the last tile (multiple of 16, <= 128); the others use 128
  int m_tiles;            // 1 or 2 UMMA tiles of the resident block are used
  int u0, u1;             // policy-defined
};

template <class P>
struct StreamShared {
  static constexpr uint32_t a_off = 0;
  static constexpr uint32_t b_off = a_off + P::kABuffers * kUsABlock;
  static constexpr uint32_t extra_off = b_off + P::kBStages * kUsBStage;
  static constexpr uint32_t item_extra_off = extra_off + ((P::kExtraBytes + 127u) / 128u) * 128u;
  static constexpr uint32_t bar_off = item_extra_off + P::kABuffers * P::kItemExtraBytes;
  static constexpr uint32_t n_bars = 2 * P::kABuffers + 2 * P::kBStages + 4;
  static constexpr uint32_t misc_off = bar_off + n_bars * 8;
  static constexpr uint32_t total = misc_off + 16;
  static constexpr uint32_t alloc = total + 1024;     // slack for the manual 1024-byte alignment
};

template <class P>
__global__ void __launch_bounds__(us_threads<P>(), 1)
umma_stream_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                   const typename P::Params prm, int* status) {
  using namespace sm100;
  using SH = StreamShared<P>;
  extern __shared__ unsigned char smem_raw[];
  // aligned to 1024 bytes by pointer arithmetic on the shared array, so that every pointer derived from
  // it is still known to point into shared memory
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* a_smem = smem + SH::a_off;
  unsigned char* b_smem = smem + SH::b_off;
  unsigned char* extra = smem + SH::extra_off;
  unsigned char* item_extra = smem + SH::item_extra_off;
  constexpr bool kHasItemExtra = P::kItemExtraBytes > 0;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SH::bar_off);
  uint64_t* a_full = bars;
  uint64_t* a_empty = a_full + P::kABuffers;
  uint64_t* b_full = a_empty + P::kABuffers;
  uint64_t* b_empty = b_full + P::kBStages;
  uint64_t* t_full = b_empty + P::kBStages;
  uint64_t* t_empty = t_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + SH::misc_off);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + SH::misc_off + 4);

  if (!P::active(prm)) return;                       // uniform across the grid
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;

  if (threadIdx.x == 0) {
    // with per-item side data the epilogue warps read the A buffer's slot too and release it with the UMMAs
    for (int i = 0; i < P::kABuffers; ++i) {
      mbar_init(a_full + i, 1);
      mbar_init(a_empty + i, kHasItemExtra ? 1 + kUsEpilogueWarps * P::kEpilogueGroups : 1);
    }
    for (int s = 0; s < P::kBStages; ++s) { mbar_init(b_full + s, 1); mbar_init(b_empty + s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(t_full + b, 1); mbar_init(t_empty + b, kUsEpilogueWarps); }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kUsTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_descriptor(&map_a);
      tma_prefetch_descriptor(&map_b);
      uint32_t b_count = 0;
      StreamItem it;
      bool ok = true;
      for (int i = 0; ok && P::get_item(prm, i, it); ++i) {
        const uint32_t abuf = (uint32_t)i % P::kABuffers, aphase = ((uint32_t)i / P::kABuffers) & 1u;
        ok = mbar_wait(a_empty + abuf, aphase ^ 1u, abort_flag);
        if (!ok) break;
        uint32_t side_bytes = 0;
        if constexpr (kHasItemExtra) side_bytes = P::item_extra_bytes(prm, it);
        mbar_expect_tx(a_full + abuf, 2 * kUsHalfTile * it.m_tiles + side_bytes);
        for (int t = 0; t < it.m_tiles; ++t)
          for (int kh = 0; kh < 2; ++kh)
            tma_load_3d(a_smem + abuf * kUsABlock + (t * 2 + kh) * kUsHalfTile, &map_a, a_full + abuf, kh * 64,
                        it.a_row + t * 128, it.a_head);
        if constexpr (kHasItemExtra)
          P::item_extra_issue(prm, it, item_extra + abuf * P::kItemExtraBytes, a_full + abuf);
        for (int tile = 0; tile < it.n_tiles; ++tile, ++b_count) {
          const uint32_t stage = b_count % P::kBStages, phase = (b_count / P::kBStages) & 1u;
          ok = mbar_wait(b_empty + stage, phase ^ 1u, abort_flag);
          if (!ok) break;
          mbar_expect_tx(b_full + stage, kUsBStage);
          for (int kh = 0; kh < 2; ++kh)
            tma_load_3d(b_smem + stage * kUsBStage + kh * kUsHalfTile, &map_b, b_full + stage, kh * 64,
                        it.b_row + tile * 128, it.b_head);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      uint32_t b_count = 0, t_count = 0;
      StreamItem it;
      bool ok = true;
      for (int i = 0; ok && P::get_item(prm, i, it); ++i) {
        const uint32_t abuf = (uint32_t)i % P::kABuffers, aphase = ((uint32_t)i / P::kABuffers) & 1u;
        ok = mbar_wait(a_full + abuf, aphase, abort_flag);
        if (!ok) break;
        const uint32_t a_lo = umma_desc_lo_sw128(smem_u32(a_smem + abuf * kUsABlock));
        for (int tile = 0; tile < it.n_tiles; ++tile, ++b_count, ++t_count) {
          const uint32_t stage = b_count % P::kBStages, phase = (b_count / P::kBStages) & 1u;
          const uint32_t buf = t_count & 1u, tphase = (t_count >> 1) & 1u;
          ok = mbar_wait(b_full + stage, phase, abort_flag) && mbar_wait(t_empty + buf, tphase ^ 1u, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t b_lo = umma_desc_lo_sw128(smem_u32(b_smem + stage * kUsBStage));
          const uint32_t idesc = umma_idesc_bf16(128, tile == it.n_tiles - 1 ? it.last_n : 128);
          for (int t = 0; t < it.m_tiles; ++t) {
            const uint32_t d_tmem = tmem_base + buf * 256u + t * 128u;
            const uint32_t at_lo = a_lo + (uint32_t)t * ((2 * kUsHalfTile) >> 4);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              // K slice kk: half kk / 4 of the tile, 32-byte step (kk % 4) inside the 128-byte swizzled row
              constexpr uint32_t kHalfStep = kUsHalfTile >> 4;
              const uint32_t off = (uint32_t)(kk / 4) * kHalfStep + (uint32_t)(kk % 4) * 2u;
              umma_bf16_lohi(d_tmem, at_lo + off, b_lo + off, idesc, kk > 0 ? 1u : 0u);
            }
          }
          umma_commit(b_empty + stage);     // the B stage may be refilled once these UMMAs have read it
          umma_commit(t_full + buf);        // the accumulators of this tile are complete
        }
        if (ok) umma_commit(a_empty + abuf);   // the resident block may be replaced once the item's UMMAs are done
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int ewarp = warp - 2;
    const int group = ewarp / kUsEpilogueWarps;
    const int quarter = warp % 4;                 // TMEM lanes this warp may read: 32 * (warp % 4) ..
    const int t = (ewarp % kUsEpilogueWarps) / 4; // which UMMA tile of the resident block
    typename P::Epilogue ep;
    ep.init(prm, extra, ewarp, lane);
    uint32_t t_count = 0;
    StreamItem it;
    bool ok = true;
    for (int i = 0; ok && P::get_item(prm, i, it); ++i) {
      const uint32_t abuf = (uint32_t)i % P::kABuffers, aphase = ((uint32_t)i / P::kABuffers) & 1u;
      if constexpr (kHasItemExtra) {
        ok = mbar_wait(a_full + abuf, aphase, abort_flag);          // the side data has landed
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      ep.item_begin(prm, it, item_extra + abuf * P::kItemExtraBytes);
      for (int tile = 0; tile < it.n_tiles; ++tile, ++t_count) {
        const uint32_t buf = t_count & 1u, tphase = (t_count >> 1) & 1u;
        if (P::kEpilogueGroups == 2 && (int)buf != group) continue;   // the other group's tile
        ok = mbar_wait(t_full + buf, tphase, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after_sync();
        if (t < it.m_tiles)
          ep.tile(prm, it, tile, tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * 256u + (uint32_t)t * 128u);
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(t_empty + buf);
      }
      if (ok) ep.item_end(prm, it);
      if constexpr (kHasItemExtra) {
        __syncwarp();
        if (ok && lane == 0) mbar_arrive(a_empty + abuf);          // this warp no longer reads the side data
      }
    }
  }

  // ------------------------------------------------------------------ common exit
  tc_fence_before_sync();
  __syncthreads();
  drain_after_abort(abort_flag);
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kUsTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag != 0) set_status(status, MEDA_ERR_TIMEOUT);
}

// Exercises the give-up path of the bounded waits on its own: one block waits on a barrier that
// nothing ever arrives on, with the given cycle limit.  The wait returns false, the block records
// MEDA_ERR_TIMEOUT exactly like the pipelines above do on their exit path, and returns; nothing is
// left waiting and no product kernel is involved.
__global__ void wait_timeout_selftest_kernel(long long limit_cycles, int* status) {
  using namespace sm100;
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    fence_barrier_init();
  }
  __syncthreads();
  // every thread waits, as the roles of a pipeline would: the first to run out raises the flag,
  // the others see it and leave too
  const bool ok = mbar_wait(&bar, 0u, &abort_flag, limit_cycles);
  __syncthreads();
  if (threadIdx.x == 0 && (!ok || abort_flag != 0)) set_status(status, MEDA_ERR_TIMEOUT);
}

}  // namespace meda
