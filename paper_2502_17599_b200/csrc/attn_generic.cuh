// Phase A, dtype-generic CUDA-core kernels (the fp32 path, and the bring-up path for bf16):
// window logits, softmax normalisers, per-key accumulated scores (Eq. 8) and the cross-modal
// attention entropy (Eq. 4-6).  One tile = kGenericKeyTile keys staged in shared memory as fp32.
#pragma once

#include "meda_common.cuh"

namespace meda {

constexpr int kAttnThreads = 256;

struct AttnGenericSmem {
  // byte offsets inside dynamic shared memory
  int q_off, k_off, s_off, abar_off, misc_off, total;
};

__host__ __device__ inline AttnGenericSmem attn_generic_smem(int w, int d, bool with_abar) {
  AttnGenericSmem L;
  int off = 0;
  L.q_off = off;    off += w * d * 4;
  L.k_off = off;    off += kGenericKeyTile * (d + 1) * 4;
  L.s_off = off;    off += w * kGenericKeyTile * 4;
  L.abar_off = off; off += with_abar ? w * kGenericKeyTile * 4 : 0;
  L.misc_off = off; off += (kGenericKeyTile * 4 + 64) * 4;
  L.total = off;
  return L;
}

// Where the operands of a launch live when they are not the dense [heads][w] window and [heads][n] cache:
// a block of query rows inside a longer query tensor, a prefix of the key cache, scores added to what the
// array holds.  A zero stride means "dense" (w or n rows per head).
struct AttnView {
  int rows_from_pos0 = 0;        // 1: query row i sits at position pos0 + i (default: the last w tokens)
  int pos0 = 0;
  int64_t q_head_stride = 0;     // rows between consecutive heads of the query tensor
  int64_t k_head_stride = 0;     // rows between consecutive KV heads of the key cache
  int64_t score_stride = 0;      // floats between consecutive KV heads of the score array
  int accumulate = 0;            // 1: scores are added to the array's contents
};

// Stage one query head [w][d] and one key tile [tile][d] as fp32; rows past n are zero.
template <typename T>
__device__ __forceinline__ void stage_q(float* qs, const T* q_h, int w, int d) {
  for (int e = threadIdx.x; e < w * d; e += blockDim.x) qs[e] = to_f32<T>(q_h[e]);
}
template <typename T>
__device__ __forceinline__ void stage_k(float* ks, const T* k_g, int j0, int n, int d) {
  for (int e = threadIdx.x; e < kGenericKeyTile * d; e += blockDim.x) {
    int r = e / d, c = e - r * d;
    int j = j0 + r;
    ks[r * (d + 1) + c] = (j < n) ? to_f32<T>(k_g[(size_t)j * d + c]) : 0.f;
  }
}

// s[i][jl] = scale * q_i . k_jl for the staged tile; -inf where the key is past the end of the
// sequence or hidden from row i by the causal mask.
__device__ __forceinline__ void tile_logits(float* s, const float* qs, const float* ks, int w, int d,
                                            int j0, int n, float scale, const int32_t* __restrict__ q_pos = nullptr,
                                            int pos0 = -1) {
  if (pos0 < 0) pos0 = n - w;                             // default rows: the last w tokens
  const int jl = threadIdx.x % kGenericKeyTile;
  const int ig = threadIdx.x / kGenericKeyTile;           // 0..3
  constexpr int kRowStep = kAttnThreads / kGenericKeyTile;
  const int j = j0 + jl;
  const float* kr = ks + jl * (d + 1);
  for (int i = ig; i < w; i += kRowStep) {
    const float* qr = qs + i * d;
    float acc = 0.f;
#pragma unroll 8
    for (int t = 0; t < d; ++t) acc = fmaf(qr[t], kr[t], acc);
    bool visible = (j < n) && (j <= (q_pos ? q_pos[i] : pos0 + i));
    s[i * kGenericKeyTile + jl] = visible ? acc * scale : -INFINITY;
  }
}

// ---------------------------------------------------------------------------------------------
// Sweep 1: partial normalisers.  grid = (chunks, Hq); block (c, h) walks tiles c, c+chunks, ...
// partial[c][h][i] = (m_all, z_all, m_vis, z_vis) over the keys of those tiles.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kAttnThreads)
stats_partial_kernel(const T* __restrict__ q_win, const T* __restrict__ k, const uint8_t* __restrict__ modality,
                     float* __restrict__ partial, int hq, int group, int n, int w, int d, float scale,
                     const int32_t* __restrict__ q_pos = nullptr, int subset = MEDA_VISUAL, int subset_only = 0,
                     AttnView view = AttnView()) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const AttnGenericSmem L = attn_generic_smem(w, d, false);
  float* qs = reinterpret_cast<float*>(smem_raw + L.q_off);
  float* ks = reinterpret_cast<float*>(smem_raw + L.k_off);
  float* s = reinterpret_cast<float*>(smem_raw + L.s_off);

  const int h = blockIdx.y, g = h / group;
  const int chunks = gridDim.x;
  const int n_tiles = (n + kGenericKeyTile - 1) / kGenericKeyTile;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const T* k_g = k + (size_t)g * (view.k_head_stride ? view.k_head_stride : n) * d;
  const int pos0 = view.rows_from_pos0 ? view.pos0 : -1;

  stage_q<T>(qs, q_win + (size_t)h * (view.q_head_stride ? view.q_head_stride : w) * d, w, d);
  // running (m, z) of every window row, updated by lane 0 of the warp that owns the row
  __shared__ float rs[kMaxWindow][4];
  for (int i = threadIdx.x; i < w; i += blockDim.x) {
    rs[i][0] = -INFINITY; rs[i][1] = 0.f; rs[i][2] = -INFINITY; rs[i][3] = 0.f;
  }
  __syncthreads();

  for (int tile = blockIdx.x; tile < n_tiles; tile += chunks) {
    const int j0 = tile * kGenericKeyTile;
    if (subset_only) {
      // only the restricted normaliser is wanted: a tile without a key of the subset contributes nothing
      const int jj = j0 + (int)threadIdx.x;
      const int mine = (threadIdx.x < kGenericKeyTile && jj < n && modality[jj] == subset) ? 1 : 0;
      if (!__syncthreads_or(mine)) continue;
    }
    stage_k<T>(ks, k_g, j0, n, d);
    __syncthreads();
    tile_logits(s, qs, ks, w, d, j0, n, scale, q_pos, pos0);
    __syncthreads();
    for (int i = warp; i < w; i += kAttnThreads / 32) {
      float a0 = s[i * kGenericKeyTile + lane], a1 = s[i * kGenericKeyTile + lane + 32];
      bool v0 = (j0 + lane < n) && modality[min(j0 + lane, n - 1)] == subset;
      bool v1 = (j0 + lane + 32 < n) && modality[min(j0 + lane + 32, n - 1)] == subset;
      float b0 = v0 ? a0 : -INFINITY, b1 = v1 ? a1 : -INFINITY;
      float m_all = warp_max(fmaxf(a0, a1));
      float m_vis = warp_max(fmaxf(b0, b1));
      float z_all = 0.f, z_vis = 0.f;
      if (m_all > -INFINITY) z_all = warp_sum(expf(a0 - m_all) + expf(a1 - m_all));
      if (m_vis > -INFINITY) z_vis = warp_sum(expf(b0 - m_vis) + expf(b1 - m_vis));
      if (lane == 0) {
        float m = rs[i][0], z = rs[i][1];
        merge_mz(m, z, m_all, z_all);
        rs[i][0] = m; rs[i][1] = z;
        m = rs[i][2]; z = rs[i][3];
        merge_mz(m, z, m_vis, z_vis);
        rs[i][2] = m; rs[i][3] = z;
      }
    }
    __syncthreads();
  }
  float* out = partial + ((size_t)blockIdx.x * hq + h) * w * 4;
  for (int e = threadIdx.x; e < w * 4; e += blockDim.x) out[e] = rs[e / 4][e % 4];
}

// row_stats[row] = merge over the key chunks' partial normalisers, row = h * w + i.  One warp per row:
// lane l merges chunks l, l + 32, ... in order, then the lanes are merged pairwise in a fixed
// butterfly, so the result does not depend on scheduling.  grid = ceil(rows / 8), block = 256.
__global__ void __launch_bounds__(256)
stats_combine_kernel(const float* __restrict__ partial, float* __restrict__ row_stats, int chunks, int rows) {
  const int row = blockIdx.x * 8 + threadIdx.x / 32, lane = threadIdx.x % 32;
  if (row >= rows) return;
  float m = -INFINITY, z = 0.f, mv = -INFINITY, zv = 0.f;
  for (int c = lane; c < chunks; c += 32) {
    const float4 p = reinterpret_cast<const float4*>(partial)[(size_t)c * rows + row];
    merge_mz(m, z, p.x, p.y);
    merge_mz(mv, zv, p.z, p.w);
  }
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o), z2 = __shfl_xor_sync(0xffffffffu, z, o);
    const float mv2 = __shfl_xor_sync(0xffffffffu, mv, o), zv2 = __shfl_xor_sync(0xffffffffu, zv, o);
    // both partners must compute the same bits: merge in (lower lane, higher lane) order
    const bool low = (lane & o) == 0;
    float ma = low ? m : m2, za = low ? z : z2, mb = low ? m2 : m, zb = low ? z2 : z;
    merge_mz(ma, za, mb, zb);
    m = ma; z = za;
    float mva = low ? mv : mv2, zva = low ? zv : zv2, mvb = low ? mv2 : mv, zvb = low ? zv2 : zv;
    merge_mz(mva, zva, mvb, zvb);
    mv = mva; zv = zva;
  }
  if (lane == 0) reinterpret_cast<float4*>(row_stats)[row] = make_float4(m, z, mv, zv);
}

// ---------------------------------------------------------------------------------------------
// Sweep 2: scores and/or entropy.  grid = key tiles; each block walks all query heads so that the
// head-averaged visual attention of its keys (Sec. 3.2 defines A as the mean over the heads of the
// per-head attention) is complete inside the block.  ent_partial[tile] = sum over the tile's visual keys
// and all window rows of a log a (entropy_mode 0) or of the head mean of p log p (mode 1).
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kAttnThreads)
scores_entropy_kernel(const T* __restrict__ q_win, const T* __restrict__ k, const uint8_t* __restrict__ modality,
                      const float* __restrict__ row_stats, float* __restrict__ scores,
                      float* __restrict__ ent_partial, int hq, int group, int n, int w, int d, float scale,
                      int entropy_mode, int want_scores, int want_entropy,
                      const int32_t* __restrict__ q_pos = nullptr, int subset = MEDA_VISUAL,
                      AttnView view = AttnView()) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const AttnGenericSmem L = attn_generic_smem(w, d, true);
  float* qs = reinterpret_cast<float*>(smem_raw + L.q_off);
  float* ks = reinterpret_cast<float*>(smem_raw + L.k_off);
  float* s = reinterpret_cast<float*>(smem_raw + L.s_off);
  float* abar = reinterpret_cast<float*>(smem_raw + L.abar_off);
  float* colsum = reinterpret_cast<float*>(smem_raw + L.misc_off);   // [4][tile]
  float* red = colsum + 4 * kGenericKeyTile;                          // [64]

  const int j0 = blockIdx.x * kGenericKeyTile;
  const int jl = threadIdx.x % kGenericKeyTile;
  const int ig = threadIdx.x / kGenericKeyTile;
  constexpr int kRowStep = kAttnThreads / kGenericKeyTile;
  const int j = j0 + jl;
  const bool in_range = j < n;
  const bool visual = in_range && modality[in_range ? j : 0] == subset;      // "in the subset the entropy is taken over"
  const float inv_hq = 1.f / (float)hq;
  const int pos0 = view.rows_from_pos0 ? view.pos0 : -1;
  const size_t q_stride = (size_t)(view.q_head_stride ? view.q_head_stride : w) * d;
  const size_t k_stride = (size_t)(view.k_head_stride ? view.k_head_stride : n) * d;
  const size_t score_stride = view.score_stride ? (size_t)view.score_stride : (size_t)n;
  if (!want_scores && !__syncthreads_or(visual ? 1 : 0)) {
    // entropy only, and no key of this tile is in the subset: nothing to add
    if (threadIdx.x == 0) ent_partial[blockIdx.x] = 0.f;
    return;
  }

  for (int e = threadIdx.x; e < w * kGenericKeyTile; e += blockDim.x) abar[e] = 0.f;
  float plogp = 0.f;     // entropy_mode 1 accumulator
  float group_score = 0.f;

  for (int h = 0; h < hq; ++h) {
    const int g = h / group;
    __syncthreads();
    stage_q<T>(qs, q_win + (size_t)h * q_stride, w, d);
    if (h % group == 0) stage_k<T>(ks, k + (size_t)g * k_stride, j0, n, d);
    __syncthreads();
    tile_logits(s, qs, ks, w, d, j0, n, scale, q_pos, pos0);
    // each thread revisits only the logits it wrote itself: no barrier needed here
    float part = 0.f;
    for (int i = ig; i < w; i += kRowStep) {
      const float* rsp = row_stats + ((size_t)h * w + i) * 4;
      float sv = s[i * kGenericKeyTile + jl];
      if (sv > -INFINITY) {
        if (want_scores) part += expf(sv - rsp[0]) / rsp[1];
        if (visual && want_entropy) {
          float pv = expf(sv - rsp[2]) / rsp[3];
          if (entropy_mode == 0) abar[i * kGenericKeyTile + jl] += pv * inv_hq;
          else if (pv > 0.f) plogp += pv * logf(pv) * inv_hq;
        }
      }
    }
    if (want_scores) {
      colsum[ig * kGenericKeyTile + jl] = part;
      __syncthreads();
      if (ig == 0) {
        group_score += colsum[jl] + colsum[kGenericKeyTile + jl] + colsum[2 * kGenericKeyTile + jl] +
                       colsum[3 * kGenericKeyTile + jl];
        if (h % group == group - 1) {
          if (in_range) {
            float* out = scores + (size_t)g * score_stride + j;
            *out = view.accumulate ? *out + group_score : group_score;
          }
          group_score = 0.f;
        }
      }
    }
  }
  if (!want_entropy) return;
  float acc = plogp;
  if (entropy_mode == 0) {
    for (int i = ig; i < w; i += kRowStep) {
      float a = abar[i * kGenericKeyTile + jl];
      if (a > 0.f) acc += a * logf(a);
    }
  }
  acc = warp_sum(acc);
  __syncthreads();
  if (threadIdx.x % 32 == 0) red[threadIdx.x / 32] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int x = 0; x < kAttnThreads / 32; ++x) t += red[x];
    ent_partial[blockIdx.x] = t;
  }
}

// entropy[layer] = -(1 / rows) * sum of the partials in index order (fixed-shape reduction, so
// repeated runs give identical bits).  rows = window rows that see at least one visual key.
__global__ void entropy_finalize_kernel(const float* __restrict__ ent_partial, int n_partials,
                                        const float* __restrict__ row_stats, int w, float* __restrict__ entropy_out,
                                        int accumulate = 0) {
  __shared__ double red[256];
  // window rows that see a key of the subset (head 0's normaliser tells): one row per thread, w <= 128
  const int rows = __syncthreads_count((int)threadIdx.x < w && row_stats[threadIdx.x * 4 + 3] > 0.f);
  double acc = 0.0;
  for (int e = threadIdx.x; e < n_partials; e += blockDim.x) acc += (double)ent_partial[e];
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const float term = rows > 0 ? (float)(-red[0] / (double)rows) : 0.f;
    *entropy_out = accumulate ? *entropy_out + term : term;      // E_CM = (-E_TV) + (-E_VT), Eq. 6
  }
}

}  // namespace meda
