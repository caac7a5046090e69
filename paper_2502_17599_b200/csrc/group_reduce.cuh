// Phase B, merge step 2 (Eq. 12): average every conserved row with the less-important rows
// assigned to it, for keys and values, deterministically.
//
// All n token rows are first grouped by slot with a stable least-significant-digit radix sort
// (9-bit digits): the list being sorted is the S kept rows (slot s, row c_s) followed by the n - S
// less-important rows (their target slot, their row), so after the sort every slot's rows are
// contiguous, the kept row first, then its members in ascending token order (stability).  Warps then
// walk fixed 128-row chunks of the sorted list, summing in fp32 in list order: no row needs a
// look-up of its own, every load address comes from the list (32 entries per coalesced load, handed
// round by shuffle; batches of 8 rows inside one slot's segment are added without a branch, two
// batches in flight).  A slot whose rows lie inside one chunk
// is finished on the spot (one division, one rounding), pieces of slots that cross chunk borders are
// parked as partial sums and added up in chunk order by a second small kernel.
// No floating-point atomics anywhere: two runs give identical bits.
#pragma once

#include "meda_common.cuh"

namespace meda {

constexpr int kSortBits = 9;
constexpr int kSortBins = 1 << kSortBits;
constexpr int kSortWarps = 8;
constexpr int kSortWarpItems = 256;                          // elements ranked by one warp
constexpr int kSortBlockItems = kSortWarps * kSortWarpItems; // elements of one block = one column of the digit table
constexpr int kSegChunk = 128;        // sorted rows walked by one warp
constexpr int kSegWarps = 2;         // small blocks: more of them fit, also beside a resident tensor-core block

// ---- stable radix pass: histogram, scatter ----------------------------------------------------
// The keys are slots < S, so the pass over the digit at `shift` orders nothing when S <= 2^shift: its three
// kernels return at once (the host enqueues the passes the prompt length may need; the layer's budget is only
// known on the device) and the consumer picks the buffer the last executed pass wrote.
__device__ __forceinline__ bool sort_pass_needed(int S, int shift) { return shift == 0 || S > (1 << shift); }
// Passes executed for a layer with S slots, of the `max_passes` the host enqueued.
__device__ __forceinline__ int sort_passes_done(int S, int max_passes) {
  int done = 1;
  while (done < max_passes && sort_pass_needed(S, done * kSortBits)) ++done;
  return done;
}

// Entry q of the list a pass reads.  The first pass (shift 0) reads the kept rows followed by the
// less-important ones straight from the caller's arrays: q < S is (slot q, row idx_conserved[q]),
// q >= S is (target[q - S], idx_less[q - S]); later passes read the previous pass's output.
__device__ __forceinline__ int sort_key_at(const int32_t* __restrict__ keys, int q, int S, int shift) {
  return shift == 0 ? (q < S ? q : keys[q - S]) : keys[q];
}
__device__ __forceinline__ int sort_row_at(const int32_t* __restrict__ rows, const int32_t* __restrict__ kept, int q,
                                           int S, int shift) {
  return shift == 0 ? (q < S ? kept[q] : rows[q - S]) : rows[q];
}

// table[g][bin][block] <- number of keys of block `block` whose digit is `bin`.
__global__ void __launch_bounds__(kSortWarps * 32)
sort_hist_kernel(const int32_t* __restrict__ keys, const int32_t* __restrict__ budget_row, int32_t* __restrict__ table,
                 int n, int cap, int shift, int n_blocks) {
  __shared__ int cnt[kSortBins];
  const int g = blockIdx.y, blk = blockIdx.x;
  const int S = min(budget_row[0], cap);
  if (!sort_pass_needed(S, shift)) return;
  for (int b = threadIdx.x; b < kSortBins; b += blockDim.x) cnt[b] = 0;
  __syncthreads();
  const int32_t* kg = keys + (size_t)g * n;
#pragma unroll
  for (int r = 0; r < kSortBlockItems / (kSortWarps * 32); ++r) {
    const int q = blk * kSortBlockItems + r * (kSortWarps * 32) + (int)threadIdx.x;
    if (q < n) atomicAdd(&cnt[(sort_key_at(kg, q, S, shift) >> shift) & (kSortBins - 1)], 1);
  }
  __syncthreads();
  int32_t* tg = table + (size_t)g * kSortBins * n_blocks;
  for (int b = threadIdx.x; b < kSortBins; b += blockDim.x) tg[(size_t)b * n_blocks + blk] = cnt[b];
}

// Stable scatter of (key, row) pairs by the digit at `shift`.  A block's first output position for a digit is
// the number of keys with a smaller digit anywhere plus the number with this digit in earlier blocks: every
// block takes both from the digit table itself (512 rows of one count per block, 128 KB per head, resident in L2:
// a row's total and its prefix up to this block, then a block-wide exclusive scan of the totals), so there is no
// scan kernel between the histogram and the scatter.  Inside a block the eight warps own consecutive runs of 256
// elements: each first counts its digits, the counts are turned into per-warp start offsets (block base + the
// earlier warps' counts), then every warp ranks its elements in index order.
// `n_blocks` (the table's row length) is a multiple of 8.
__global__ void __launch_bounds__(kSortWarps * 32)
sort_scatter_kernel(const int32_t* __restrict__ keys_in, const int32_t* __restrict__ rows_in,
                    const int32_t* __restrict__ kept, const int32_t* __restrict__ budget_row,
                    const int32_t* __restrict__ table,
                    int32_t* __restrict__ keys_out, int32_t* __restrict__ rows_out, int n, int cap, int shift,
                    int n_blocks) {
  __shared__ int cnt[kSortWarps][kSortBins];
  __shared__ int base[kSortBins];                         // row totals, then this block's first position per digit
  __shared__ int warp_tot[kSortWarps];
  static_assert(kSortBins == 2 * kSortWarps * 32, "two digits per thread");
  const int g = blockIdx.y, blk = blockIdx.x, warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int S_layer = min(budget_row[0], cap);
  if (!sort_pass_needed(S_layer, shift)) return;
  if (blk * kSortBlockItems >= n) return;                 // uniform over the block
  // ---- this block's base per digit, from the raw digit table (thread t owns digits 2t and 2t + 1)
  const int32_t* tg = table + (size_t)g * kSortBins * n_blocks;
  int before[2], total[2];
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int4* row = reinterpret_cast<const int4*>(tg + (size_t)(2 * threadIdx.x + u) * n_blocks);
    int all = 0, pre = 0;
    for (int v4 = 0; v4 < n_blocks / 4; ++v4) {
      const int4 x = row[v4];
      const int b0 = 4 * v4;
      all += x.x + x.y + x.z + x.w;
      pre += (b0 < blk ? x.x : 0) + (b0 + 1 < blk ? x.y : 0) + (b0 + 2 < blk ? x.z : 0) + (b0 + 3 < blk ? x.w : 0);
    }
    total[u] = all;
    before[u] = pre;
  }
  {
    const int mine = total[0] + total[1];
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    int lower = incl - mine;                               // digits below this thread's, all blocks
    for (int w = 0; w < warp; ++w) lower += warp_tot[w];
    base[2 * threadIdx.x] = lower + before[0];
    base[2 * threadIdx.x + 1] = lower + total[0] + before[1];
  }
  const int32_t* kg = keys_in + (size_t)g * n;
  const int32_t* rg = rows_in + (size_t)g * n;
  const int32_t* kept_g = kept + (size_t)g * cap;
  int32_t* ko = keys_out + (size_t)g * n;
  int32_t* ro = rows_out + (size_t)g * n;
  const int q0 = blk * kSortBlockItems + warp * kSortWarpItems;
  constexpr int kRounds = kSortWarpItems / 32;
  int key[kRounds];
  for (int b = lane; b < kSortBins; b += 32) cnt[warp][b] = 0;
  __syncwarp();
#pragma unroll
  for (int r = 0; r < kRounds; ++r) {
    const int q = q0 + r * 32 + lane;
    key[r] = q < n ? sort_key_at(kg, q, S_layer, shift) : -1;
    if (key[r] >= 0) atomicAdd(&cnt[warp][(key[r] >> shift) & (kSortBins - 1)], 1);
  }
  __syncthreads();
  for (int b = threadIdx.x; b < kSortBins; b += blockDim.x) {
    int run = base[b];
#pragma unroll
    for (int w = 0; w < kSortWarps; ++w) {
      const int c = cnt[w][b];
      cnt[w][b] = run;
      run += c;
    }
  }
  __syncthreads();
  const unsigned int lt = (1u << lane) - 1u;
#pragma unroll
  for (int r = 0; r < kRounds; ++r) {
    const int q = q0 + r * 32 + lane;
    const bool valid = key[r] >= 0;
    const int digit = (key[r] >> shift) & (kSortBins - 1);
    const int row = valid ? sort_row_at(rg, kept_g, q, S_layer, shift) : 0;
    const unsigned int peers = __match_any_sync(0xffffffffu, valid ? digit : kSortBins + lane);
    const int leader = __ffs(peers) - 1;
    int base = 0;
    if (valid && lane == leader) {
      base = cnt[warp][digit];
      cnt[warp][digit] = base + __popc(peers);
    }
    base = __shfl_sync(0xffffffffu, base, leader);
    if (valid) {
      const int pos = min(base + __popc(peers & lt), n - 1);
      ko[pos] = key[r];
      ro[pos] = row;
    }
    __syncwarp();
  }
}

// ---- segmented average ---------------------------------------------------------------------------
// Layout of the parked partial sums: piece `which` (0 = head: the slot started in an earlier chunk,
// 1 = tail: it started here and continues) of chunk c of head g holds 2*D floats (keys then values).
template <int D>
__device__ __forceinline__ float* carry_ptr(float* carry, int g, int chunk, int which, int n_chunks) {
  return carry + (((size_t)g * n_chunks + chunk) * 2 + which) * (2 * D);
}

template <typename T, int E>
__device__ __forceinline__ void load_row(const T* p, int lane, float (&x)[E]);

template <>
__device__ __forceinline__ void load_row<__nv_bfloat16, 2>(const __nv_bfloat16* p, int lane, float (&x)[2]) {
  float2 a = __bfloat1622float2(reinterpret_cast<const __nv_bfloat162*>(p)[lane]);
  x[0] = a.x; x[1] = a.y;
}
template <>
__device__ __forceinline__ void load_row<__nv_bfloat16, 4>(const __nv_bfloat16* p, int lane, float (&x)[4]) {
  uint2 u = reinterpret_cast<const uint2*>(p)[lane];
  float2 a = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&u.x));
  float2 b = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&u.y));
  x[0] = a.x; x[1] = a.y; x[2] = b.x; x[3] = b.y;
}
template <>
__device__ __forceinline__ void load_row<__nv_bfloat16, 8>(const __nv_bfloat16* p, int lane, float (&x)[8]) {
  uint4 u = reinterpret_cast<const uint4*>(p)[lane];
  float2 a = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&u.x));
  float2 b = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&u.y));
  float2 c = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&u.z));
  float2 d = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&u.w));
  x[0] = a.x; x[1] = a.y; x[2] = b.x; x[3] = b.y; x[4] = c.x; x[5] = c.y; x[6] = d.x; x[7] = d.y;
}
template <>
__device__ __forceinline__ void load_row<float, 2>(const float* p, int lane, float (&x)[2]) {
  float2 a = reinterpret_cast<const float2*>(p)[lane];
  x[0] = a.x; x[1] = a.y;
}
template <>
__device__ __forceinline__ void load_row<float, 4>(const float* p, int lane, float (&x)[4]) {
  float4 a = reinterpret_cast<const float4*>(p)[lane];
  x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
}
template <>
__device__ __forceinline__ void load_row<float, 8>(const float* p, int lane, float (&x)[8]) {
  float4 a = reinterpret_cast<const float4*>(p)[2 * lane], b = reinterpret_cast<const float4*>(p)[2 * lane + 1];
  x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}

// Lane `lane` owns elements [lane * E, lane * E + E) of a row.
template <typename T, int E>
__device__ __forceinline__ void store_row(T* p, int lane, const float (&x)[E], float count) {
#pragma unroll
  for (int e = 0; e < E; ++e) p[lane * E + e] = from_f32<T>(x[e] / count);
}

// A lane's share of a row as loaded (E elements, not yet widened), and its addition to fp32 sums.
template <typename T, int E> struct RawRow;
template <> struct RawRow<__nv_bfloat16, 2> { uint32_t u; };
template <> struct RawRow<__nv_bfloat16, 4> { uint2 u; };
template <> struct RawRow<__nv_bfloat16, 8> { uint4 u; };
template <int E> struct RawRow<float, E> { float f[E]; };

__device__ __forceinline__ void add_bf16x2(float& lo, float& hi, uint32_t u) {
  lo += __uint_as_float(u << 16);
  hi += __uint_as_float(u & 0xffff0000u);
}
__device__ __forceinline__ void raw_load(RawRow<__nv_bfloat16, 2>& r, const char* p) { r.u = *reinterpret_cast<const uint32_t*>(p); }
__device__ __forceinline__ void raw_load(RawRow<__nv_bfloat16, 4>& r, const char* p) { r.u = *reinterpret_cast<const uint2*>(p); }
__device__ __forceinline__ void raw_load(RawRow<__nv_bfloat16, 8>& r, const char* p) { r.u = *reinterpret_cast<const uint4*>(p); }
template <int E>
__device__ __forceinline__ void raw_load(RawRow<float, E>& r, const char* p) {
#pragma unroll
  for (int e = 0; e < E; ++e) r.f[e] = reinterpret_cast<const float*>(p)[e];
}
__device__ __forceinline__ void raw_add(float (&a)[2], const RawRow<__nv_bfloat16, 2>& r) { add_bf16x2(a[0], a[1], r.u); }
__device__ __forceinline__ void raw_add(float (&a)[4], const RawRow<__nv_bfloat16, 4>& r) {
  add_bf16x2(a[0], a[1], r.u.x);
  add_bf16x2(a[2], a[3], r.u.y);
}
__device__ __forceinline__ void raw_add(float (&a)[8], const RawRow<__nv_bfloat16, 8>& r) {
  add_bf16x2(a[0], a[1], r.u.x);
  add_bf16x2(a[2], a[3], r.u.y);
  add_bf16x2(a[4], a[5], r.u.z);
  add_bf16x2(a[6], a[7], r.u.w);
}
template <int E>
__device__ __forceinline__ void raw_add(float (&a)[E], const RawRow<float, E>& r) {
#pragma unroll
  for (int e = 0; e < E; ++e) a[e] += r.f[e];
}

template <int E> struct SegSums { float a[E]; };

// End of a piece of a slot's segment inside a chunk.  A segment that starts and ends in the chunk is finished here
// (one division, one rounding; a slot without members keeps its row as it is); a piece of a segment that crosses
// the chunk's border is parked for seg_border_kernel.  The walker calls this from rolled loops only, so that it
// holds few copies of this code: with one copy per row of an unrolled batch it outgrew the instruction cache and
// ran at half speed wherever most slots have no members (a call out of line was slower too: the batches in
// flight had to be saved around it).
template <typename T, int E>
__device__ __forceinline__ void seg_end_piece(SegSums<E> sums, int members, bool whole, T* out_row, float* park_row,
                                           int32_t* count_out, int lane) {
  if (whole) {
    if (members == 1) {
#pragma unroll
      for (int e = 0; e < E; ++e) out_row[lane * E + e] = from_f32<T>(sums.a[e]);
    } else {
      store_row<T, E>(out_row, lane, sums.a, (float)members);
    }
  } else {
#pragma unroll
    for (int e = 0; e < E; ++e) park_row[lane * E + e] = sums.a[e];
  }
  if (count_out != nullptr) *count_out = members;
}

// grid = (chunks / kSegWarps, heads, 2): blockIdx.z picks the tensor (0 keys, 1 values), so that twice
// as many warps keep rows in flight; the z = 0 warps also record segment bounds and counts.  Every slot
// has at least one row in the list (its kept row), so every slot's bounds get written.
template <typename T, int D>
__global__ void __launch_bounds__(kSegWarps * 32, 10)
seg_reduce_kernel(const T* __restrict__ k, const T* __restrict__ v, const int32_t* __restrict__ keys_a,
                  const int32_t* __restrict__ rows_a, const int32_t* __restrict__ keys_b,
                  const int32_t* __restrict__ rows_b, int max_passes, const int32_t* __restrict__ budget_row, T* __restrict__ k_out, T* __restrict__ v_out,
                  int32_t* __restrict__ counts, int32_t* __restrict__ seg_start, int32_t* __restrict__ seg_end,
                  float* __restrict__ carry, int32_t* __restrict__ carry_cnt, int n, int cap, int n_chunks) {
  constexpr int E = D / 32;
  const int g = blockIdx.y, warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int tensor = blockIdx.z;
  const bool book = tensor == 0 && lane == 0;            // the one lane that writes bounds and counts
  // The list's last chunks first: slots are in token order, so the recent window's slots (most of them without
  // members: one segment per row, the slowest chunks) come last in the list and would otherwise form the tail.
  const int chunk = n_chunks - 1 - ((int)blockIdx.x * kSegWarps + warp);
  const int S = min(budget_row[0], cap);
  const int q0 = chunk * kSegChunk;
  if (S <= 0 || chunk < 0 || q0 >= n) return;
  const int q1 = min(q0 + kSegChunk, n);
  // the grouped list is in the buffer the last executed sort pass wrote: pass p writes buffer p % 2
  const bool in_b = ((sort_passes_done(S, max_passes) - 1) & 1) != 0;
  const int32_t* kg = (in_b ? keys_b : keys_a) + (size_t)g * n;
  const int32_t* rg = (in_b ? rows_b : rows_a) + (size_t)g * n;
  const char* x_bytes = reinterpret_cast<const char*>((tensor == 0 ? k : v) + (size_t)g * n * D) + lane * (E * sizeof(T));
  T* out_g = (tensor == 0 ? k_out : v_out) + (size_t)g * cap * D;
  int32_t* st = seg_start + (size_t)g * n;
  int32_t* en = seg_end + (size_t)g * n;

  SegSums<E> acc;
  int members = 0;                  // rows of the slot summed so far, the kept row included
  int cur = min(max(kg[q0], 0), S - 1);
  bool started_here = (q0 == 0) || (kg[q0 - 1] != kg[q0]);

  auto begin_segment = [&](int slot, bool fresh, int q) {
    members = 0;
#pragma unroll
    for (int e = 0; e < E; ++e) acc.a[e] = 0.f;
    if (fresh && book) st[slot] = q;
  };
  auto end_piece = [&](int slot, bool fresh, bool ended, int q_end) {
    if (ended && book) en[slot] = q_end;
    const bool whole = fresh && ended;
    const int which = fresh ? 1 : 0;
    int32_t* count_out = !book ? nullptr
                         : whole ? counts + (size_t)g * cap + slot
                                 : carry_cnt + ((size_t)g * n_chunks + chunk) * 2 + which;
    seg_end_piece<T, E>(acc, members, whole, out_g + (size_t)slot * D,
                        carry_ptr<D>(carry, g, chunk, which, n_chunks) + tensor * D, count_out, lane);
  };

  begin_segment(cur, started_here, q0);
  // Rounds of 32 list entries: lane l holds entry qb + l (one coalesced load per array and round, the next round's
  // in flight during this one) and the entries reach the other lanes by shuffle.  A round is cut into batches of
  // 8 rows (fewer for wide rows), two batches in flight.  A batch that lies inside the current slot's segment (the common case wherever slots
  // have many members) is summed without a branch; the others go row by row.
  using Raw = RawRow<T, E>;
  constexpr int kBatch = sizeof(Raw) <= 8 ? 8 : (sizeof(Raw) <= 16 ? 4 : 2);      // two batches of 64 bytes per lane in flight
  int key_l, row_l;
  {
    const int q = min(q0 + lane, q1 - 1);
    key_l = kg[q];
    row_l = rg[q];
  }
#pragma unroll 1
  for (int qb = q0; qb < q1; qb += 32) {
    const int key_r = min(max(key_l, 0), S - 1);
    const uint32_t off_r = (uint32_t)min(max(row_l, 0), n - 1) * (uint32_t)(D * sizeof(T));
    const bool live = qb + lane < q1;
    if (qb + 32 < q1) {
      const int q = min(qb + 32 + lane, q1 - 1);
      key_l = kg[q];
      row_l = rg[q];
    }
    auto fetch = [&](Raw (&x)[kBatch], int b0) {
#pragma unroll
      for (int b = 0; b < kBatch; ++b) raw_load(x[b], x_bytes + __shfl_sync(0xffffffffu, off_r, b0 + b));
    };
    auto consume = [&](const Raw (&x)[kBatch], int b0) {
      const unsigned int brk = (__ballot_sync(0xffffffffu, !live || key_r != cur) >> b0) & ((1u << kBatch) - 1u);
      if (brk == 0u) {
#pragma unroll
        for (int b = 0; b < kBatch; ++b) raw_add(acc.a, x[b]);
        members += kBatch;
      } else {
        // row by row, one copy of the code: the rows are read again (they are in the first-level cache, the
        // batch's loads brought them), the next row's load in flight while this row is handled
        Raw nxt;
        raw_load(nxt, x_bytes + __shfl_sync(0xffffffffu, off_r, b0));
#pragma unroll 1
        for (int b = 0; b < kBatch; ++b) {
          const Raw now = nxt;
          raw_load(nxt, x_bytes + __shfl_sync(0xffffffffu, off_r, min(b0 + b + 1, 31)));
          const int key_b = __shfl_sync(0xffffffffu, key_r, b0 + b);
          if (qb + b0 + b < q1) {
            if (key_b != cur) {
              end_piece(cur, started_here, true, qb + b0 + b);
              cur = key_b;
              started_here = true;
              begin_segment(cur, true, qb + b0 + b);
            }
            raw_add(acc.a, now);
            ++members;
          }
        }
      }
    };
    // entries past the chunk's end repeat its last entry: their loads are in bounds and their rows are not added
    Raw xa[kBatch], xb[kBatch];
    fetch(xa, 0);
#pragma unroll 1
    for (int h = 0; h < 32; h += 2 * kBatch) {
      fetch(xb, h + kBatch);
      consume(xa, h);
      if (h + 2 * kBatch < 32) fetch(xa, h + 2 * kBatch);
      consume(xb, h + kBatch);
    }
  }
  const bool ended = (q1 == n) || (min(max(kg[q1], 0), S - 1) != cur);
  end_piece(cur, started_here, ended, q1);
}

// Finishes the slots whose rows span several chunks: one warp per (chunk border, tensor).  The slot that
// crosses border b (the last row of chunk b - 1 and the first row of chunk b belong to it) is finished
// by the warp of the FIRST border it crosses: the piece parked by the chunk where it starts, then the
// pieces of the following chunks in chunk order (loaded eight at a time, added one by one), one division,
// one rounding.  Everything else was finished by the walker.  grid = (blocks of 8 borders, heads, 2).
template <typename T, int D>
__global__ void __launch_bounds__(256)
seg_border_kernel(const int32_t* __restrict__ keys_a, const int32_t* __restrict__ keys_b, int max_passes,
                  const int32_t* __restrict__ budget_row, const int32_t* __restrict__ seg_start,
                  const int32_t* __restrict__ seg_end, const float* __restrict__ carry,
                  const int32_t* __restrict__ carry_cnt, T* __restrict__ k_out, T* __restrict__ v_out,
                  int32_t* __restrict__ counts, int n, int cap, int n_chunks) {
  constexpr int E = D / 32;
  const int g = blockIdx.y, lane = threadIdx.x % 32;
  const int tensor = blockIdx.z;
  const int S = min(budget_row[0], cap);
  const int border = blockIdx.x * 8 + threadIdx.x / 32 + 1;       // between chunks border - 1 and border
  const int q = border * kSegChunk;
  if (S <= 0 || q >= n) return;
  const bool in_b = ((sort_passes_done(S, max_passes) - 1) & 1) != 0;
  const int32_t* kg = (in_b ? keys_b : keys_a) + (size_t)g * n;
  const int slot = min(max(kg[q - 1], 0), S - 1);
  if (min(max(kg[q], 0), S - 1) != slot) return;                  // no slot crosses this border
  const int start = seg_start[(size_t)g * n + slot], end = seg_end[(size_t)g * n + slot];
  const int c0 = start / kSegChunk, c1 = (end - 1) / kSegChunk;
  if (c0 != border - 1) return;                                   // an earlier border finishes this slot
  T* out_g = (tensor == 0 ? k_out : v_out) + (size_t)g * cap * D;
  float* base = const_cast<float*>(carry);
  float acc[E];
  const float* p = carry_ptr<D>(base, g, c0, 1, n_chunks) + tensor * D;
#pragma unroll
  for (int e = 0; e < E; ++e) acc[e] = p[lane * E + e];
  int members = carry_cnt[((size_t)g * n_chunks + c0) * 2 + 1];
  for (int cb = c0 + 1; cb <= c1; cb += 8) {
    float x[8][E];
    int m[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int c = min(cb + u, c1);
      const float* pc = carry_ptr<D>(base, g, c, 0, n_chunks) + tensor * D;
#pragma unroll
      for (int e = 0; e < E; ++e) x[u][e] = pc[lane * E + e];
      m[u] = carry_cnt[((size_t)g * n_chunks + c) * 2];
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (cb + u <= c1) {
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] += x[u][e];
        members += m[u];
      }
    }
  }
  store_row<T, E>(out_g + (size_t)slot * D, lane, acc, (float)members);
  if (tensor == 0 && lane == 0) counts[(size_t)g * cap + slot] = members;
}

// Without merging (merge_mode 1) the kept rows are copied: one warp per (slot, tensor).
// grid = (blocks, heads, 2).
template <typename T, int D>
__global__ void __launch_bounds__(256)
copy_kept_kernel(const T* __restrict__ k, const T* __restrict__ v, const int32_t* __restrict__ idx_conserved,
                 const int32_t* __restrict__ budget_row, T* __restrict__ k_out, T* __restrict__ v_out,
                 int32_t* __restrict__ counts, int n, int cap) {
  constexpr int E = D / 32;
  const int g = blockIdx.y, lane = threadIdx.x % 32;
  const int tensor = blockIdx.z;
  const T* x_g = (tensor == 0 ? k : v) + (size_t)g * n * D;
  T* out_g = (tensor == 0 ? k_out : v_out) + (size_t)g * cap * D;
  const int S = min(budget_row[0], cap);
  // the grid is sized on the host for the largest possible S: walk the slots with a stride
  for (int slot = blockIdx.x * 8 + threadIdx.x / 32; slot < S; slot += gridDim.x * 8) {
    const int own = min(max(idx_conserved[(size_t)g * cap + slot], 0), n - 1);
    float acc[E];
    load_row<T, E>(x_g + (size_t)own * D, lane, acc);
    store_row<T, E>(out_g + (size_t)slot * D, lane, acc, 1.f);
    if (tensor == 0 && lane == 0) counts[(size_t)g * cap + slot] = 1;
  }
}

}  // namespace meda
