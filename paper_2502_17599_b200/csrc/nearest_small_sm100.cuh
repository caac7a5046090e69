// Phase B, merge step 1 (Eq. 11 and its arg-max) for layers whose budget is small (S <= kNearestSmallMaxS):
// the same arithmetic as nearest_kernel on the streaming UMMA pipeline.
//
// With a handful of conserved slots there is one slot tile (or a few) per block of token rows, and what the
// row-gathering kernel spends per block (rows fetched by index into tensor memory, nothing to overlap them
// with) is most of its time.  Here the token rows are NOT gathered: a block takes 256 consecutive rows of the
// key cache by TMA (double buffered, so the next block's rows arrive during this block's UMMAs) against the
// S gathered conserved keys, for every row of the prompt, kept ones included (S of n rows: little waste for
// these layers).  Each epilogue thread owns a row, scales by the slots' inverse norms and keeps the first
// maximum exactly like NearestRow in nearest_kernel; a row's place in the less-important list is its index
// minus the number of kept rows before it (a binary search in the ascending kept list), so the result
// lands in list order like nearest_kernel's.
#pragma once

#include "nearest_sm100.cuh"
#include "umma_stream.cuh"

namespace meda {

struct NearestSmallPolicy {
  struct Params {
    const float* inv_norm;         // [heads][inv_stride]
    const int32_t* budget_row;     // (S, M, N) of the layer
    const int32_t* idx_conserved;  // [heads][cap]: the S kept token rows of every head, ascending
    int32_t* target;               // [heads][n]: slot chosen for the p-th less-important row of the head
    int n, n_heads, cap, inv_stride;
    int row_blocks;                // ceil(n / 256)
  };
  static constexpr int kABuffers = 2;
  static constexpr int kBStages = 2;
  static constexpr int kEpilogueGroups = 1;
  static constexpr uint32_t kExtraBytes = 0;
  static constexpr uint32_t kItemExtraBytes = 0;

  __device__ static int slots(const Params& p) { return min(p.budget_row[0], p.cap); }
  __device__ static bool active(const Params& p) {
    const int S = slots(p);
    return S > 0 && S < p.n && S <= kNearestSmallMaxS;
  }
  __device__ static bool get_item(const Params& p, int it, StreamItem& o) {
    const int idx = blockIdx.x + it * gridDim.x;
    if (idx >= p.row_blocks * p.n_heads) return false;
    const int g = idx / p.row_blocks, blk = idx % p.row_blocks;
    const int S = slots(p);
    o.a_row = blk * 256;
    o.a_head = g;
    o.b_row = 0;
    o.b_head = g;
    o.n_tiles = (S + 127) / 128;
    o.last_n = ((S - (o.n_tiles - 1) * 128 + 15) / 16) * 16;       // UMMA N: a multiple of 16 covering the last slots
    o.m_tiles = (p.n - o.a_row > 128) ? 2 : 1;
    o.u0 = g;
    o.u1 = S;
    return true;
  }

  struct Epilogue {
    NearestRow row;
    int row_in_block;
    const float* inv;
    __device__ void init(const Params&, unsigned char*, int ewarp, int lane) {
      row_in_block = (ewarp / 4) * 128 + ((ewarp + 2) % 4) * 32 + lane;
    }
    __device__ void item_begin(const Params& p, const StreamItem& it, const unsigned char*) {
      row.best = -INFINITY;
      row.best_slot = 0;
      inv = p.inv_norm + (size_t)it.u0 * p.inv_stride;
    }
    __device__ void tile(const Params& p, const StreamItem& it, int tile, uint32_t taddr) {
      const int S = it.u1;
      const bool valid = it.a_row + row_in_block < p.n;
      const int n_chunks = (min(S - tile * 128, 128) + 31) / 32;
      // columns past the UMMA's N hold an earlier tile's values; they are slots >= S, which chunk() masks
      uint32_t ra[32], rb[32];
      sm100::tmem_ld_32x32_issue(taddr, ra);
#pragma unroll 1
      for (int c = 0; c < n_chunks; c += 2) {
        const int s0 = tile * 128 + 32 * c;
        sm100::tmem_ld_wait();
        sm100::tmem_ld_pin(ra);
        if (c + 1 < n_chunks) sm100::tmem_ld_32x32_issue(taddr + 32u * (c + 1), rb);
        if (valid) row.chunk(ra, inv + s0, s0, S, s0 + 32 > S);
        if (c + 1 < n_chunks) {
          sm100::tmem_ld_wait();
          sm100::tmem_ld_pin(rb);
          if (c + 2 < n_chunks) sm100::tmem_ld_32x32_issue(taddr + 32u * (c + 2), ra);
          if (valid) row.chunk(rb, inv + s0 + 32, s0 + 32, S, s0 + 64 > S);
        }
      }
    }
    __device__ void item_end(const Params& p, const StreamItem& it) {
      const int r = it.a_row + row_in_block;
      if (r >= p.n) return;
      // kept rows before r: the first position of the kept list whose row is >= r
      const int32_t* kept = p.idx_conserved + (size_t)it.u0 * p.cap;
      int lo = 0, hi = it.u1;
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(kept + mid) < r) lo = mid + 1; else hi = mid;
      }
      if (lo < it.u1 && __ldg(kept + lo) == r) return;           // a kept row: it has no target
      p.target[(size_t)it.u0 * p.n + (r - lo)] = row.best_slot;
    }
  };
};

}  // namespace meda
