// Eq. 8 with every prompt row as a query (no observation window): the accumulated score of key j
// is the column sum of the whole causal attention matrix,
//   A_s[g][j] = sum over the query heads h of KV head g and over the rows i >= j of softmax_j(q_i.k / sqrt(d)).
// bf16 / head_dim 128, two passes of the streaming UMMA pipeline over the causal half of the matrix:
//
//  PromptStatsPolicy  resident block = 256 query rows of one head, streamed tiles = the keys those rows
//                     can see; every epilogue thread owns one query row and keeps its online softmax
//                     normaliser (max, sum of exp2).  Two epilogue groups take alternate key tiles;
//                     prompt_ref_kernel merges their partials into one reference per row.
//  PromptSweepPolicy  resident block = 256 keys of one KV head, streamed tiles = the query rows of one
//                     query head from the block's first key on; every epilogue thread owns one key and
//                     sums exp2(t - ref[row]) over the rows that see it.  With ref = max + log2(sum)
//                     that exponential already is the softmax probability: one fused multiply-add,
//                     one exp2 and one add per logit.  The query heads of a KV head follow each other
//                     in the same block; the rows a key block streams are cut into a few runs, and two
//                     epilogue groups take alternate row tiles: prompt_sum_kernel adds those partial
//                     scores in a fixed order.
//
// Logits are kept in base-2 units: t = (q.k) * scale * log2(e).
#pragma once

#include "attn_sm100.cuh"

namespace meda {

constexpr float kPromptHidden = -1e30f;     // replaces a logit the causal mask hides: its exp2 is exactly 0
constexpr float kPromptNoRow = -1e30f;      // negated reference of a row past the end of the prompt: every exp2 is 0

// ---------------------------------------------------------------------------------------------
// Pass 1: normalisers of every prompt row
// ---------------------------------------------------------------------------------------------
struct PromptStatsPolicy {
  struct Params {
    float2* partial;             // [2][Hq][n_pad] (max, sum exp2) per epilogue group, base-2 units
    int n, n_pad, hq, group;
    int row_blocks;              // ceil(n / 256)
    float sc2;                   // scale * log2(e)
  };
  static constexpr int kABuffers = 2;
  static constexpr int kBStages = 3;
  static constexpr int kEpilogueGroups = 2;
  static constexpr uint32_t kExtraBytes = 0;
  static constexpr uint32_t kItemExtraBytes = 0;

  __device__ static bool active(const Params&) { return true; }
  // Longest items first: the last row block sees every key.
  __device__ static bool get_item(const Params& p, int it, StreamItem& o) {
    const int idx = blockIdx.x + it * gridDim.x;
    if (idx >= p.row_blocks * p.hq) return false;
    const int rb = p.row_blocks - 1 - idx / p.hq, h = idx % p.hq;
    o.a_row = rb * 256;
    o.a_head = h;
    o.b_row = 0;
    o.b_head = h / p.group;
    const int last_row = min(o.a_row + 255, p.n - 1);
    o.n_tiles = last_row / 128 + 1;                  // keys 0 .. last_row
    o.last_n = 128;
    o.m_tiles = (p.n - o.a_row > 128) ? 2 : 1;
    o.u0 = h;
    o.u1 = rb;
    return true;
  }

  struct Epilogue {
    int lane, row_in_block, group;
    float m, z;                  // running (max, sum) of this thread's query row
    __device__ void init(const Params&, unsigned char*, int ewarp, int lane_) {
      lane = lane_;
      group = ewarp / kUsEpilogueWarps;
      row_in_block = ((ewarp % kUsEpilogueWarps) / 4) * 128 + ((ewarp + 2) % 4) * 32 + lane_;
    }
    __device__ void item_begin(const Params&, const StreamItem&, const unsigned char*) {
      m = -INFINITY;
      z = 0.f;
    }
    // 32 consecutive keys starting at j0 against query row r (which sees keys j <= r).
    __device__ __forceinline__ void chunk(const Params& p, const uint32_t (&acc)[32], int j0, int r) {
      if (j0 + 31 <= r) {
        float t[12];
#pragma unroll
        for (int x = 0; x < 10; ++x)
          t[x] = sm100::fmax3(__uint_as_float(acc[3 * x]), __uint_as_float(acc[3 * x + 1]), __uint_as_float(acc[3 * x + 2]));
        t[10] = __uint_as_float(acc[30]);
        t[11] = __uint_as_float(acc[31]);
        const float u0 = sm100::fmax3(t[0], t[1], t[2]), u1 = sm100::fmax3(t[3], t[4], t[5]);
        const float u2 = sm100::fmax3(t[6], t[7], t[8]), u3 = sm100::fmax3(t[9], t[10], t[11]);
        const float cm = fmaxf(sm100::fmax3(u0, u1, u2), u3);
        const float m_new = fmaxf(m, cm * p.sc2);
        // four running sums as two packed pairs: the scaling and the additions take half the issue slots
        const uint64_t sc2x2 = f32x2(p.sc2, p.sc2), ref2 = f32x2(-m_new, -m_new);
        uint64_t a01 = f32x2(0.f, 0.f), a23 = a01;
#pragma unroll
        for (int x = 0; x < 32; x += 4) {
          float t0, t1, t2, t3;
          f32x2_split(fma_f32x2(sm100::pack_f32x2(acc[x + 0], acc[x + 1]), sc2x2, ref2), t0, t1);
          f32x2_split(fma_f32x2(sm100::pack_f32x2(acc[x + 2], acc[x + 3]), sc2x2, ref2), t2, t3);
          a01 = add_f32x2(a01, f32x2(fast_exp2(t0), fast_exp2(t1)));
          a23 = add_f32x2(a23, f32x2(fast_exp2(t2), fast_exp2(t3)));
        }
        float a0, a1, a2, a3;
        f32x2_split(a01, a0, a1);
        f32x2_split(a23, a2, a3);
        z = z * fast_exp2(m - m_new) + ((a0 + a1) + (a2 + a3));
        m = m_new;
      } else {
        // the chunk on the diagonal
#pragma unroll
        for (int x = 0; x < 32; ++x) {
          if (j0 + x <= r) {
            const float t = __uint_as_float(acc[x]) * p.sc2;
            if (t > m) { z = z * fast_exp2(m - t) + 1.f; m = t; }
            else z += fast_exp2(t - m);
          }
        }
      }
    }
    __device__ void tile(const Params& p, const StreamItem& it, int tile, uint32_t taddr) {
      const int r = it.a_row + row_in_block;            // this thread's query row
      const bool valid = r < p.n;
      const int warp_last = r - lane + 31;              // the warp's last row sees the most keys
      const int c0 = tile * 128;
      uint32_t acc[32];
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        const int j0 = c0 + 32 * c;
        if (j0 > warp_last) break;                      // hidden from every row of the warp
        sm100::tmem_ld_32x32_issue(taddr + 32u * c, acc);
        sm100::tmem_ld_wait();
        sm100::tmem_ld_pin(acc);
        if (valid && j0 <= r) chunk(p, acc, j0, r);
      }
    }
    __device__ void item_end(const Params& p, const StreamItem& it) {
      const int r = it.a_row + row_in_block;
      if (r >= p.n) return;
      p.partial[((size_t)group * p.hq + it.u0) * p.n_pad + r] = make_float2(m, z);
    }
  };
};

// ref[h][r] = -(max + log2(sum)) of row r over both partials (base-2 units, negated: the sweep adds it);
// rows past the end of the prompt (the padding up to n_pad) get a reference no logit reaches.
__global__ void __launch_bounds__(256)
prompt_ref_kernel(const float2* __restrict__ partial, float* __restrict__ ref, int hq, int n, int n_pad) {
  const size_t total = (size_t)hq * n_pad;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
    const int r = (int)(e % n_pad);
    float out = kPromptNoRow;
    if (r < n) {
      const float2 a = partial[e], b = partial[total + e];
      const float m = fmaxf(a.x, b.x);                  // finite: every row sees itself
      const float z = a.y * fast_exp2(a.x - m) + b.y * fast_exp2(b.x - m);
      out = -(m + log2f(z));
    }
    ref[e] = out;
  }
}

// ---------------------------------------------------------------------------------------------
// Pass 2: column sums
// ---------------------------------------------------------------------------------------------
// The rows a 256-key block streams (from its first key to the end of the prompt) are cut into up to
// `splits` contiguous runs of row tiles, so that short prompts still fill the GPU; a block with fewer
// row tiles than that has one run per tile.
__host__ __device__ inline int prompt_block_tiles(int n, int blk) { return (n - blk * 256 + 127) / 128; }
__host__ __device__ inline int prompt_block_splits(int n, int blk, int splits) {
  const int t = prompt_block_tiles(n, blk);
  return t < splits ? t : splits;
}

struct PromptSweepPolicy {
  struct Params {
    const float* ref;            // [Hq][n_pad], negated references
    float* partial;              // [splits * 2][Hkv][n]: one slot per (row run, epilogue group)
    int n, n_pad, hq, hkv, group;
    int n_blocks;                // ceil(n / 256)
    int splits;                  // row runs per key block (1..8)
    int full_blocks;             // key blocks with at least `splits` row tiles: blocks 0 .. full_blocks - 1
    float sc2;
  };
  static constexpr int kABuffers = 2;
  static constexpr int kBStages = 3;
  static constexpr int kEpilogueGroups = 2;
  static constexpr uint32_t kExtraBytes = 0;
  static constexpr uint32_t kItemExtraBytes = 0;

  __device__ static bool active(const Params&) { return true; }
  // A unit = (key block, KV head, row run), longest first (block 0 streams the most rows); the thread
  // block that takes a unit walks the query heads of its KV head back to back, one item each.
  __device__ static bool get_item(const Params& p, int it, StreamItem& o) {
    int u = blockIdx.x + (it / p.group) * gridDim.x;
    const int per_full = p.hkv * p.splits;
    int blk, runs;
    if (u < p.full_blocks * per_full) {
      blk = u / per_full;
      u -= blk * per_full;
      runs = p.splits;
    } else {
      u -= p.full_blocks * per_full;
      for (blk = p.full_blocks; blk < p.n_blocks; ++blk) {      // at most splits / 2 short blocks at the end
        runs = prompt_block_splits(p.n, blk, p.splits);
        if (u < p.hkv * runs) break;
        u -= p.hkv * runs;
      }
      if (blk >= p.n_blocks) return false;
    }
    const int g = u / runs, run = u % runs;
    const int tiles = prompt_block_tiles(p.n, blk);
    const int t_lo = run * tiles / runs, t_hi = (run + 1) * tiles / runs;     // runs <= tiles: never empty
    o.a_row = blk * 256;
    o.a_head = g;
    o.b_row = blk * 256 + t_lo * 128;                // earlier rows see none of these keys
    o.b_head = g * p.group + it % p.group;
    o.n_tiles = t_hi - t_lo;                         // rows past n read as zeros and carry the "no row" reference
    o.last_n = 128;
    o.m_tiles = (p.n - o.a_row > 128) ? 2 : 1;
    o.u0 = o.b_head;
    o.u1 = run;
    return true;
  }

  struct Epilogue {
    int lane, row_in_block, egroup;
    float score;                 // this thread's key, summed over the tiles and heads of the unit so far
    uint64_t s01, s23;           // partial sums inside one tile (packed pairs): small addends meet a small running sum
    __device__ void init(const Params&, unsigned char*, int ewarp, int lane_) {
      lane = lane_;
      egroup = ewarp / kUsEpilogueWarps;
      row_in_block = ((ewarp % kUsEpilogueWarps) / 4) * 128 + ((ewarp + 2) % 4) * 32 + lane_;
      score = 0.f;
    }
    __device__ void item_begin(const Params&, const StreamItem&, const unsigned char*) {}
    __device__ __forceinline__ void chunk(const Params& p, uint32_t (&acc)[32], const float4* __restrict__ ref4,
                                          int r0, int j) {
      if (r0 < j) {
        // rows before the key do not see it
#pragma unroll
        for (int x = 0; x < 32; ++x) if (r0 + x < j) acc[x] = __float_as_uint(kPromptHidden);
      }
      const uint64_t sc2x2 = f32x2(p.sc2, p.sc2);
#pragma unroll
      for (int x = 0; x < 32; x += 4) {
        // negated references of rows r0 + x .. r0 + x + 3, as two packed pairs
        const ulonglong2 c = __ldg(reinterpret_cast<const ulonglong2*>(ref4) + x / 4);
        float t0, t1, t2, t3;
        f32x2_split(fma_f32x2(sm100::pack_f32x2(acc[x + 0], acc[x + 1]), sc2x2, c.x), t0, t1);
        f32x2_split(fma_f32x2(sm100::pack_f32x2(acc[x + 2], acc[x + 3]), sc2x2, c.y), t2, t3);
        s01 = add_f32x2(s01, f32x2(fast_exp2(t0), fast_exp2(t1)));
        s23 = add_f32x2(s23, f32x2(fast_exp2(t2), fast_exp2(t3)));
      }
    }
    __device__ void tile(const Params& p, const StreamItem& it, int tile, uint32_t taddr) {
      const int j = it.a_row + row_in_block;            // this thread's key
      const bool valid = j < p.n;
      const int warp_first = j - lane;                  // the warp's first key is seen by the most rows
      const int r_tile = it.b_row + tile * 128;
      const float4* ref4 = reinterpret_cast<const float4*>(p.ref + (size_t)it.u0 * p.n_pad + r_tile);
      s01 = s23 = f32x2(0.f, 0.f);
      // one chunk in registers at a time (sixteen epilogue warps hide the load latency for each other, and
      // a block of this size has no registers for a second buffer)
      uint32_t acc[32];
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        if (r_tile + 32 * c + 31 < warp_first) continue;          // rows that see no key of the warp
        sm100::tmem_ld_32x32_issue(taddr + 32u * c, acc);
        sm100::tmem_ld_wait();
        sm100::tmem_ld_pin(acc);
        if (valid) chunk(p, acc, ref4 + 8 * c, r_tile + 32 * c, j);
      }
      float s0, s1, s2, s3;
      f32x2_split(s01, s0, s1);
      f32x2_split(s23, s2, s3);
      score += (s0 + s1) + (s2 + s3);
    }
    __device__ void item_end(const Params& p, const StreamItem& it) {
      if (it.u0 % p.group != p.group - 1) return;       // more heads of this KV head follow
      const int j = it.a_row + row_in_block;
      if (j < p.n) p.partial[((size_t)(it.u1 * 2 + egroup) * p.hkv + it.u0 / p.group) * p.n + j] = score;
      score = 0.f;
    }
  };
};

// scores[g][j] = the slots of key j's block added in slot order (row run by row run, epilogue group 0 then 1).
__global__ void __launch_bounds__(256)
prompt_sum_kernel(const float* __restrict__ partial, float* __restrict__ scores, int hkv, int n, int splits) {
  const size_t total = (size_t)hkv * n;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
    const int j = (int)(e % n);
    const int slots = 2 * prompt_block_splits(n, j / 256, splits);
    float acc = 0.f;
    for (int s = 0; s < slots; ++s) acc += partial[(size_t)s * total + e];
    scores[e] = acc;
  }
}

}  // namespace meda
