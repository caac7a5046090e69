// Phase A for bf16 / head_dim 128 on the tensor cores (Eq. 4-6 and Eq. 8 with the query rows
// restricted to the observation window).  Two policies of the streaming UMMA pipeline:
//
//  StatsPolicy  (sweep 1)  resident block = the window rows of one KV group (rows = (head, window
//               row)), streamed tiles = 128 keys each; every epilogue thread owns one query row and
//               keeps online softmax normalisers (max, sum of exp2) separately over visual and text
//               keys.  One exp2 per logit.
//  SweepPolicy  (sweep 2)  resident block = 256 keys of one KV head (rows = keys), streamed tiles =
//               the group's window rows, 128 columns each; every epilogue thread owns one key: it sums
//               the normalised probabilities of its key over all columns (the accumulated score,
//               Eq. 8) and keeps the head-averaged text-to-vision attention of its key for every
//               window row across the KV heads, from which the entropy partial follows (Eq. 5).
//               One exp2 per logit serves both the full and the visual-only softmax.
//
// Logits are kept in base-2 units: t = (q.k) * scale * log2(e).
#pragma once

#include "umma_stream.cuh"

namespace meda {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Packed fp32 pairs (sm_100): two fused multiply-adds / two additions per issue slot, each rounded exactly
// like the scalar instruction.  Operands are pairs of fp32 in 64-bit registers.
__device__ __forceinline__ uint64_t f32x2(float lo, float hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
}
__device__ __forceinline__ void f32x2_split(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// ---------------------------------------------------------------------------------------------
// Sweep 1: normalisers
// ---------------------------------------------------------------------------------------------
struct StatsPolicy {
  struct Params {
    const uint8_t* modality;     // padded to a multiple of 128 with the value 2 (= no key)
    float* partial;              // [chunks * 2][Hq][w][4]: one partial per (key chunk, epilogue group)
    int n, hq, group, w, cols;   // cols = group * w query rows per KV group
    int row_blocks;              // ceil(cols / 256)
    int chunks, tiles_per_chunk, tiles_total;
    float sc2;                   // scale * log2(e)
  };
  static constexpr int kABuffers = 1;
  static constexpr int kBStages = 4;
  static constexpr int kEpilogueGroups = 2;      // this sweep is bound by its epilogue: two tiles at a time
  static constexpr uint32_t kExtraBytes = kEpilogueGroups * kUsEpilogueWarps * 128;   // one modality slice per epilogue warp
  static constexpr uint32_t kItemExtraBytes = 0;

  __device__ static bool active(const Params&) { return true; }
  __device__ static bool get_item(const Params& p, int it, StreamItem& o) {
    const int idx = blockIdx.x + it * gridDim.x;
    const int per_group = p.row_blocks * p.chunks;
    const int n_groups = p.hq / p.group;
    if (idx >= per_group * n_groups) return false;
    const int g = idx / per_group, rb = (idx / p.chunks) % p.row_blocks, kc = idx % p.chunks;
    o.a_row = g * p.cols + rb * 256;
    o.a_head = 0;
    o.b_row = kc * p.tiles_per_chunk * 128;
    o.b_head = g;
    o.n_tiles = min(p.tiles_per_chunk, p.tiles_total - kc * p.tiles_per_chunk);
    o.last_n = 128;
    o.m_tiles = (p.cols - rb * 256 > 128) ? 2 : 1;
    o.u0 = g * 65536 + rb;        // group and row block
    o.u1 = kc;
    return o.n_tiles > 0;
  }

  struct Epilogue {
    uint8_t* mod_t;
    int lane, row_in_block, group;
    float mv, zv, mt, zt;        // running (max, sum) in base-2 logit units, visual and text keys
    __device__ void init(const Params&, unsigned char* extra, int ewarp, int lane_) {
      mod_t = extra + ewarp * 128;
      lane = lane_;
      group = ewarp / kUsEpilogueWarps;
      row_in_block = ((ewarp % kUsEpilogueWarps) / 4) * 128 + ((ewarp + 2) % 4) * 32 + lane_;
    }
    __device__ void item_begin(const Params&, const StreamItem&, const unsigned char*) {
      mv = mt = -INFINITY;
      zv = zt = 0.f;
    }
    __device__ __forceinline__ static void absorb(float& m, float& z, float t) {
      if (t > m) { z = z * fast_exp2(m - t) + 1.f; m = t; }
      else z += fast_exp2(t - m);
    }
    // 32 consecutive keys starting at j0 against this thread's query row.
    // uniform_text / uniform_visual: all 32 keys of the chunk are text / visual (the same for every row: the
    // caller derives them once per tile from two warp votes).
    __device__ __forceinline__ void chunk(const Params& p, const uint32_t (&r)[32], int chunk_idx, int j0,
                                          int last_visible, bool uniform_text, bool uniform_visual) {
      if ((uniform_text || uniform_visual) && j0 + 31 <= last_visible) {
        // one modality, all keys visible: chunk maximum first (three-input maxima), then one exp2 per key
        float t[12];
#pragma unroll
        for (int x = 0; x < 10; ++x)
          t[x] = sm100::fmax3(__uint_as_float(r[3 * x]), __uint_as_float(r[3 * x + 1]), __uint_as_float(r[3 * x + 2]));
        t[10] = __uint_as_float(r[30]);
        t[11] = __uint_as_float(r[31]);
        const float u0 = sm100::fmax3(t[0], t[1], t[2]), u1 = sm100::fmax3(t[3], t[4], t[5]);
        const float u2 = sm100::fmax3(t[6], t[7], t[8]), u3 = sm100::fmax3(t[9], t[10], t[11]);
        const float cm = fmaxf(sm100::fmax3(u0, u1, u2), u3);
        float& m = uniform_visual ? mv : mt;
        float& z = uniform_visual ? zv : zt;
        const float m_new = fmaxf(m, cm * p.sc2);
        // four running sums as two packed pairs: the scaling and the additions take half the issue slots
        const uint64_t sc2x2 = f32x2(p.sc2, p.sc2), ref2 = f32x2(-m_new, -m_new);
        uint64_t a01 = f32x2(0.f, 0.f), a23 = a01;
#pragma unroll
        for (int x = 0; x < 32; x += 4) {
          float t0, t1, t2, t3;
          f32x2_split(fma_f32x2(sm100::pack_f32x2(r[x + 0], r[x + 1]), sc2x2, ref2), t0, t1);
          f32x2_split(fma_f32x2(sm100::pack_f32x2(r[x + 2], r[x + 3]), sc2x2, ref2), t2, t3);
          a01 = add_f32x2(a01, f32x2(fast_exp2(t0), fast_exp2(t1)));
          a23 = add_f32x2(a23, f32x2(fast_exp2(t2), fast_exp2(t3)));
        }
        float a0, a1, a2, a3;
        f32x2_split(a01, a0, a1);
        f32x2_split(a23, a2, a3);
        z = z * fast_exp2(m - m_new) + ((a0 + a1) + (a2 + a3));
        m = m_new;
      } else {
#pragma unroll
        for (int x = 0; x < 32; ++x) {
          const int md = mod_t[chunk_idx * 32 + x];
          if (md < 2 && j0 + x <= last_visible) {
            if (md == MEDA_VISUAL) absorb(mv, zv, __uint_as_float(r[x]) * p.sc2);
            else absorb(mt, zt, __uint_as_float(r[x]) * p.sc2);
          }
        }
      }
    }
    __device__ void tile(const Params& p, const StreamItem& it, int tile, uint32_t taddr) {
      const int rb = it.u0 & 65535;
      const int r = rb * 256 + row_in_block;            // query row inside the KV group
      const bool valid = r < p.cols;
      const int i = r % p.w;
      const int last_visible = p.n - p.w + i;           // causal: keys j <= last_visible
      const int c0 = it.b_row + tile * 128;
      __syncwarp();
      const uint32_t mod4 = __ldg(reinterpret_cast<const uint32_t*>(p.modality + c0) + lane);   // keys 4 lane .. 4 lane + 3
      reinterpret_cast<uint32_t*>(mod_t)[lane] = mod4;
      __syncwarp();
      // which 32-key chunks hold one modality only: lanes 8 c .. 8 c + 7 cover chunk c
      const uint32_t text4 = __ballot_sync(0xffffffffu, mod4 == 0u);
      const uint32_t vis4 = __ballot_sync(0xffffffffu, mod4 == 0x01010101u);
      if (!__any_sync(0xffffffffu, valid)) return;
      // One chunk in registers at a time: with four epilogue warps per scheduler the load latency hides
      // behind the other warps, and a second buffer does not fit the 96 registers a 576-thread block
      // leaves (a kernel with a tensor-memory load in flight must not spill: the destination
      // registers could be saved before the load has landed).
      uint32_t acc[32];
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        sm100::tmem_ld_32x32_issue(taddr + 32u * c, acc);
        sm100::tmem_ld_wait();
        sm100::tmem_ld_pin(acc);
        if (valid)
          chunk(p, acc, c, c0 + 32 * c, last_visible, ((text4 >> (8 * c)) & 0xffu) == 0xffu,
                ((vis4 >> (8 * c)) & 0xffu) == 0xffu);
      }
    }
    __device__ void item_end(const Params& p, const StreamItem& it) {
      const int g = it.u0 >> 16, rb = it.u0 & 65535;
      const int r = rb * 256 + row_in_block;
      if (r >= p.cols) return;
      const int h = g * p.group + r / p.w, i = r % p.w;
      // all keys = visual and text together
      const float m_all = fmaxf(mv, mt);
      float z_all = 0.f;
      if (m_all > -INFINITY) z_all = zv * fast_exp2(mv - m_all) + zt * fast_exp2(mt - m_all);
      float4 out;
      out.x = m_all * kLn2;
      out.y = z_all;
      out.z = mv * kLn2;
      out.w = zv;
      reinterpret_cast<float4*>(p.partial)[((size_t)(it.u1 * kEpilogueGroups + group) * p.hq + h) * p.w + i] = out;
    }
  };
};

// ---------------------------------------------------------------------------------------------
// Per-column constants of sweep 2, from the normalisers (column = query head * w + window row).
//   vis[c]  = (m_vis * log2e + log2(z_vis * Hq),  Hq * z_vis * exp(m_vis - m_all) / z_all)   for visual keys
//   text[c] = (m_all * log2e,                     1 / z_all)                                 for text keys
// For a visual key one e = exp2(t - vis.x) is already the head-averaged visual-softmax probability
// p_vis / Hq, and e * vis.y is the full-softmax probability; for a text key exp2(t - text.x) * text.y
// is the full-softmax probability.  A row that sees no visual key gets (+huge, 0): e = 0.
// ---------------------------------------------------------------------------------------------
// Two layouts of the tables: (ref, ratio) per column, or, for the sweep that works on pairs of columns with
// packed arithmetic, four floats per pair of columns: (-ref, -ref', ratio, ratio').
__device__ __forceinline__ void store_sweep_coef(float2* table, size_t col, float2 c, bool paired) {
  if (!paired) {
    table[col] = c;
  } else {
    float* f = reinterpret_cast<float*>(table) + (col / 2) * 4 + (col & 1);
    f[0] = -c.x;
    f[2] = c.y;
  }
}

__global__ void sweep_coef_kernel(const float* __restrict__ row_stats, float2* __restrict__ vis,
                                  float2* __restrict__ text, int rows, float hq, bool paired) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= rows) return;
  const float4 s = reinterpret_cast<const float4*>(row_stats)[c];
  float2 a = make_float2(1e30f, 0.f);
  if (s.w > 0.f) {
    a.x = fmaf(s.z, kLog2e, log2f(s.w * hq));
    a.y = hq * s.w * expf(s.z - s.x) / s.y;
  }
  store_sweep_coef(vis, c, a, paired);
  store_sweep_coef(text, c, make_float2(s.x * kLog2e, 1.f / s.y), paired);
}

// ---------------------------------------------------------------------------------------------
// Sweep 2: scores and entropy.  W = window (32 or 64), MODE = entropy_mode.  The per-column constants
// of the item's KV group travel with the resident key block (bulk copies on the same barrier) and
// are read from shared memory, one broadcast load per logit.
// ---------------------------------------------------------------------------------------------
constexpr int kSweepMaxCols = 512;                     // query rows per KV group the tensor-core sweep accepts

template <int W, int MODE>
struct SweepPolicy {
  struct Params {
    const uint8_t* modality;     // padded as above
    const float2* vis;           // [Hq * w]
    const float2* text;          // [Hq * w]
    float* scores;               // [Hkv][n] or null
    float* ent_partial;          // [blocks * 8] or null
    int n, hkv, cols;            // cols = group * W columns per KV head (multiple of 32, <= kSweepMaxCols)
    int n_blocks;                // ceil(n / 256)
    float sc2;
    float ln_hq;                 // ln(n_q_heads): ln p = ln(p / Hq) + ln Hq in the mean of per-head entropies
  };
  static constexpr int kABuffers = 2;
  static constexpr int kBStages = 2;
  static constexpr int kEpilogueGroups = 1;
  static constexpr uint32_t kExtraBytes = 0;
  static constexpr uint32_t kTextOff = kSweepMaxCols * 8;
  static constexpr uint32_t kItemExtraBytes = kSweepMaxCols * (8 + 8);

  __device__ static bool active(const Params&) { return true; }
  // Each block takes whole 256-key blocks and walks all KV heads of a block back to back, so that
  // the head-averaged attention of its keys is complete inside one thread.
  __device__ static bool get_item(const Params& p, int it, StreamItem& o) {
    const int blk = blockIdx.x + (it / p.hkv) * gridDim.x;
    if (blk >= p.n_blocks) return false;
    const int g = it % p.hkv;
    o.a_row = blk * 256;
    o.a_head = g;
    o.b_row = g * p.cols;
    o.b_head = 0;
    o.n_tiles = (p.cols + 127) / 128;
    o.last_n = p.cols - (o.n_tiles - 1) * 128;      // cols is a multiple of 32
    o.m_tiles = (p.n - o.a_row > 128) ? 2 : 1;
    o.u0 = g;
    o.u1 = blk;
    return true;
  }
  __device__ static uint32_t item_extra_bytes(const Params& p, const StreamItem&) { return (uint32_t)p.cols * 16u; }
  __device__ static void item_extra_issue(const Params& p, const StreamItem& it, unsigned char* dst, uint64_t* bar) {
    sm100::bulk_load(dst, p.vis + it.b_row, (uint32_t)p.cols * 8u, bar);
    sm100::bulk_load(dst + kTextOff, p.text + it.b_row, (uint32_t)p.cols * 8u, bar);
  }

  struct Epilogue {
    int lane, ewarp, row_in_block;
    const float4* cvis;          // this item's constants in shared memory, two columns per 16 bytes
    const float4* ctext;
    float abar[W];               // head-averaged visual-softmax attention of this key, per window row
    float plogp;                 // MODE 1 accumulator
    float score;
    int md, first_row;           // this thread's key: modality, first window row that sees it
    bool valid, masked;
    __device__ void init(const Params&, unsigned char*, int ewarp_, int lane_) {
      lane = lane_;
      ewarp = ewarp_;
      row_in_block = (ewarp_ / 4) * 128 + ((ewarp_ + 2) % 4) * 32 + lane_;
#pragma unroll
      for (int x = 0; x < W; ++x) abar[x] = 0.f;
      plogp = 0.f;
    }
    __device__ void item_begin(const Params& p, const StreamItem& it, const unsigned char* item_extra) {
      score = 0.f;
      cvis = reinterpret_cast<const float4*>(item_extra);
      ctext = reinterpret_cast<const float4*>(item_extra + kTextOff);
      // what the tiles need to know about this thread's key, fetched once per item, off the tile path
      const int j = it.a_row + row_in_block;
      valid = j < p.n;
      md = p.modality[j];                                  // the padded map covers j up to the block end
      first_row = j - (p.n - W);                           // causal: window rows i >= first_row see key j
      masked = __any_sync(0xffffffffu, valid && first_row > 0);
    }

    // A visual key against 32 query columns (one head's window rows OFF .. OFF + 31), all of which see it.
    template <int OFF>
    __device__ __forceinline__ void chunk_visual(const Params& p, const uint32_t (&r)[32], const float4* c4) {
#pragma unroll
      for (int x = 0; x < 32; x += 2) {
        const float4 c = c4[x / 2];                        // (ref, ratio) of columns x and x + 1
        const float t0 = fmaf(__uint_as_float(r[x]), p.sc2, -c.x);
        const float t1 = fmaf(__uint_as_float(r[x + 1]), p.sc2, -c.z);
        const float e0 = fast_exp2(t0), e1 = fast_exp2(t1);
        score = fmaf(e0, c.y, score);
        score = fmaf(e1, c.w, score);
        if (MODE == 0) {
          abar[OFF + x] += e0;
          abar[OFF + x + 1] += e1;
        } else {
          plogp = fmaf(e0, fmaf(t0, kLn2, p.ln_hq), plogp);
          plogp = fmaf(e1, fmaf(t1, kLn2, p.ln_hq), plogp);
        }
      }
    }
    __device__ __forceinline__ void chunk_text(const Params& p, const uint32_t (&r)[32], const float4* c4) {
#pragma unroll
      for (int x = 0; x < 32; x += 2) {
        const float4 c = c4[x / 2];
        score = fmaf(fast_exp2(fmaf(__uint_as_float(r[x]), p.sc2, -c.x)), c.y, score);
        score = fmaf(fast_exp2(fmaf(__uint_as_float(r[x + 1]), p.sc2, -c.z)), c.w, score);
      }
    }
    // `masked`: some key of the warp lies inside the observation window (the last W of the sequence), so
    // window rows before first_row do not see it.  Those logits are replaced by a hugely negative
    // value, whose exp2 is exactly zero, and the ordinary routines run.  Only the last key block
    // gets here.
    __device__ __forceinline__ void chunk(const Params& p, uint32_t (&r)[32], int local) {
      if (masked) {
        const int row0 = local % W;
#pragma unroll
        for (int x = 0; x < 32; ++x) if (row0 + x < first_row) r[x] = __float_as_uint(-1e30f);
      }
      if (md == MEDA_VISUAL) {
        if (W == 32 || local % W == 0) chunk_visual<0>(p, r, cvis + local / 2);
        else chunk_visual<(W > 32 ? 32 : 0)>(p, r, cvis + local / 2);
      } else {
        chunk_text(p, r, ctext + local / 2);
      }
    }
    __device__ void tile(const Params& p, const StreamItem& it, int tile, uint32_t taddr) {
      const int n_chunks = (tile == it.n_tiles - 1 ? it.last_n : 128) / 32;
      const int local0 = tile * 128;                       // column inside the KV group: head * W + row
      if (W > 32) {
        // 64 running sums per thread leave no room for a second register buffer (nothing may spill
        // while a tensor-memory load is in flight): one chunk at a time
        uint32_t acc[32];
#pragma unroll 1
        for (int c = 0; c < n_chunks; ++c) {
          sm100::tmem_ld_32x32_issue(taddr + 32u * c, acc);
          sm100::tmem_ld_wait();
          sm100::tmem_ld_pin(acc);
          if (valid) chunk(p, acc, local0 + 32 * c);
        }
        return;
      }
      // two register buffers: the load of chunk c + 1 is in flight while chunk c is reduced
      uint32_t ra[32], rb[32];
      sm100::tmem_ld_32x32_issue(taddr, ra);
      sm100::tmem_ld_wait();
      sm100::tmem_ld_pin(ra);
      if (n_chunks > 1) sm100::tmem_ld_32x32_issue(taddr + 32u, rb);
      if (valid) chunk(p, ra, local0);
      if (n_chunks > 1) {
        sm100::tmem_ld_wait();
        sm100::tmem_ld_pin(rb);
        if (n_chunks > 2) sm100::tmem_ld_32x32_issue(taddr + 64u, ra);
        if (valid) chunk(p, rb, local0 + 32);
      }
      if (n_chunks > 2) {
        sm100::tmem_ld_wait();
        sm100::tmem_ld_pin(ra);
        if (n_chunks > 3) sm100::tmem_ld_32x32_issue(taddr + 96u, rb);
        if (valid) chunk(p, ra, local0 + 64);
      }
      if (n_chunks > 3) {
        sm100::tmem_ld_wait();
        sm100::tmem_ld_pin(rb);
        if (valid) chunk(p, rb, local0 + 96);
      }
    }
    __device__ void item_end(const Params& p, const StreamItem& it) {
      const int j = it.a_row + row_in_block;
      if (p.scores && j < p.n) p.scores[(size_t)it.u0 * p.n + j] = score;
      if (it.u0 == p.hkv - 1) {
        // all heads of this key block are in: entropy partial of this warp's 32 keys
        float acc = plogp;
        if (MODE == 0) {
#pragma unroll
          for (int x = 0; x < W; ++x) {
            const float a = abar[x];
            if (a > 0.f) acc = fmaf(a, __logf(a), acc);
            abar[x] = 0.f;
          }
        }
        plogp = 0.f;
        acc = warp_sum(acc);
        if (p.ent_partial && lane == 0) p.ent_partial[(size_t)it.u1 * kUsEpilogueWarps + ewarp] = acc;
      }
    }
  };
};

}  // namespace meda
