// C-ABI entry points of the MEDA compression pass (declared in include/meda.h): argument checks,
// context and scratch memory, and kernel launches.  Host code here only enqueues work.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <new>
#include <vector>

#include "allocate.cuh"
#include "attn_generic.cuh"
#include "attn_sm100.cuh"
#include "decode.cuh"
#include "meda_common.cuh"
#include "group_reduce.cuh"
#include "merge_generic.cuh"
#include "nearest_sm100.cuh"
#include "nearest_small_sm100.cuh"
#include "prompt_scores_sm100.cuh"
#include "select.cuh"
#include "window_stats_sm100.cuh"
#include "window_sweep_sm100.cuh"

using namespace meda;

namespace {

constexpr int kMaxDynSmem = 227 * 1024;

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

#define MEDA_CUDA_TRY(expr)                         \
  do {                                              \
    cudaError_t e__ = (expr);                       \
    if (e__ != cudaSuccess) return MEDA_ERR_CUDA;   \
  } while (0)

inline meda_status launch_status() { return cudaGetLastError() == cudaSuccess ? MEDA_OK : MEDA_ERR_CUDA; }

template <typename T>
meda_status carve(T** p, int64_t count, int64_t* total) {
  int64_t bytes = ((count * (int64_t)sizeof(T)) + 255) / 256 * 256;
  if (bytes == 0) bytes = 256;
  if (cudaMalloc(reinterpret_cast<void**>(p), (size_t)bytes) != cudaSuccess) return MEDA_ERR_CUDA;
  *total += bytes;
  return MEDA_OK;
}

void free_workspace(Workspace& ws) {
  cudaFree(ws.modality);
  cudaFree(ws.status);
  cudaFree(ws.stats_partial);
  cudaFree(ws.decode_partial);
  cudaFree(ws.row_stats_vis);
  cudaFree(ws.ent_partial);
  cudaFree(ws.inv_norm);
  cudaFree(ws.target);
  cudaFree(ws.idx_less);
  cudaFree(ws.kc);
  cudaFree(ws.coef_vis);
  cudaFree(ws.coef_text);
  cudaFree(ws.tile_class);
  cudaFree(ws.stats_counters);
  cudaFree(ws.sweep_counter);
  for (int i = 0; i < 2; ++i) { cudaFree(ws.sort_keys[i]); cudaFree(ws.sort_rows[i]); }
  cudaFree(ws.sort_table);
  cudaFree(ws.seg_start);
  cudaFree(ws.seg_end);
  cudaFree(ws.carry);
  cudaFree(ws.carry_cnt);
  ws = Workspace();
}

// grid.x of a kernel that walks up to `slots` conserved slots with a stride, `per_block` slots per block
// and step, replicated `copies` times in grid.y / grid.z: about sixteen blocks per SM in total.  The slot
// count is only known on the device, so the grid is sized for the worst case and must stay small.
int slot_blocks(const meda_ctx* ctx, int slots, int per_block, int copies) {
  const int needed = (slots + per_block - 1) / per_block;
  return std::max(1, std::min(needed, (ctx->sm_count * 16 + copies - 1) / copies));
}

int generic_tiles(int n) { return (n + kGenericKeyTile - 1) / kGenericKeyTile; }

// Raises a kernel's dynamic shared memory limit to the most the SM offers next to the kernel's
// static shared memory.  The limit belongs to the kernel, not to a context, so it is never set
// to one context's need: contexts of different shapes coexist.
template <typename K>
meda_status raise_dyn_smem(K kernel) {
  cudaFuncAttributes a;
  MEDA_CUDA_TRY(cudaFuncGetAttributes(&a, kernel));
  MEDA_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kMaxDynSmem - (int)a.sharedSizeBytes));
  return MEDA_OK;
}

template <typename T>
meda_status set_generic_attrs() {
  meda_status r = raise_dyn_smem(stats_partial_kernel<T>);
  if (r == MEDA_OK) r = raise_dyn_smem(scores_entropy_kernel<T>);
  if (r == MEDA_OK) r = raise_dyn_smem(nearest_generic_kernel<T>);
  return r;
}

// Brackets one kernel launch with profiling events (when enabled) and counts it.
struct LaunchScope {
  meda_ctx* ctx;
  cudaStream_t st;
  int slot = -1;
  LaunchScope(meda_ctx* c, int klass, cudaStream_t s) : ctx(c), st(s) {
    ++ctx->launches;
    Profiler& p = ctx->prof;
    if (p.enabled && p.used < Profiler::kPool) {
      slot = p.used++;
      p.klass[slot] = klass;
      cudaEventRecord(p.begin[slot], st);
    } else if (p.enabled) {
      ++p.dropped;
    }
  }
  ~LaunchScope() {
    if (slot >= 0) cudaEventRecord(ctx->prof.end[slot], st);
  }
};

void profiler_release(Profiler& p) {
  if (p.begin) {
    for (int i = 0; i < Profiler::kPool; ++i) {
      if (p.begin[i]) cudaEventDestroy(p.begin[i]);
      if (p.end[i]) cudaEventDestroy(p.end[i]);
    }
  }
  free(p.begin);
  free(p.end);
  free(p.klass);
  p = Profiler();
}

bool layer_ok(const meda_ctx* ctx, int32_t layer) { return ctx && layer >= 0 && layer < ctx->cfg.n_layers; }

// ---- TMA descriptors ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

void* resolve_encode_tiled() {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess)
    return nullptr;
  return fn;
}

// bf16 tensor [heads][rows][128] (row-major, dense) as a 3-D map with 64-column x box_rows boxes and
// the 128-byte swizzle the UMMA operand descriptors expect.  Out-of-range rows read as zeros.
bool make_rows_map(const meda_ctx* ctx, CUtensorMap* map, const void* base, int64_t rows, int64_t heads,
                   int64_t head_stride_rows, uint32_t box_rows) {
  cuuint64_t dims[3] = {(cuuint64_t)kFastDim, (cuuint64_t)rows, (cuuint64_t)heads};
  cuuint64_t strides[2] = {(cuuint64_t)kFastDim * 2, (cuuint64_t)head_stride_rows * kFastDim * 2};
  cuuint32_t box[3] = {64, box_rows, 1};
  cuuint32_t elem[3] = {1, 1, 1};
  CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
      map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, elem,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// ---- phase A launches ------------------------------------------------------------------------
template <typename T>
meda_status launch_stats(meda_ctx* ctx, const void* q_win, const void* k, float* row_stats, cudaStream_t st) {
  const meda_config& c = ctx->cfg;
  const float scale = 1.0f / sqrtf((float)c.head_dim);
  const int chunks = std::min(kStatsChunks, generic_tiles(c.n_tokens));
  const int smem = attn_generic_smem(c.window, c.head_dim, false).total;
  {
    LaunchScope scope(ctx, MEDA_K_STATS, st);
    stats_partial_kernel<T><<<dim3(chunks, c.n_q_heads), kAttnThreads, smem, st>>>(
        static_cast<const T*>(q_win), static_cast<const T*>(k), ctx->ws.modality, ctx->ws.stats_partial,
        c.n_q_heads, ctx->group, c.n_tokens, c.window, c.head_dim, scale);
  }
  {
    LaunchScope scope(ctx, MEDA_K_STATS_COMBINE, st);
    stats_combine_kernel<<<(c.n_q_heads * c.window + 7) / 8, 256, 0, st>>>(ctx->ws.stats_partial, row_stats, chunks,
                                                                               c.n_q_heads * c.window);
  }
  return launch_status();
}

template <typename T>
meda_status launch_sweep(meda_ctx* ctx, int32_t layer, const void* q_win, const void* k, const float* row_stats,
                         float* scores, float* entropy, cudaStream_t st) {
  const meda_config& c = ctx->cfg;
  const float scale = 1.0f / sqrtf((float)c.head_dim);
  const int tiles = generic_tiles(c.n_tokens);
  const int smem = attn_generic_smem(c.window, c.head_dim, true).total;
  {
    LaunchScope scope(ctx, MEDA_K_SWEEP, st);
    scores_entropy_kernel<T><<<tiles, kAttnThreads, smem, st>>>(
        static_cast<const T*>(q_win), static_cast<const T*>(k), ctx->ws.modality, row_stats, scores,
        ctx->ws.ent_partial, c.n_q_heads, ctx->group, c.n_tokens, c.window, c.head_dim, scale, c.entropy_mode,
        scores != nullptr, entropy != nullptr);
  }
  if (entropy) {
    LaunchScope scope(ctx, MEDA_K_ENTROPY_FINAL, st);
    entropy_finalize_kernel<<<1, 256, 0, st>>>(ctx->ws.ent_partial, tiles, row_stats, c.window, entropy + layer);
  }
  return launch_status();
}

// bf16, head_dim 128, window 32 or 64: both sweeps on the tensor cores.  The normaliser sweep also merges its
// partial results (the last warp to finish a set of rows does) and writes the per-column constants of the
// second sweep, so no other launch is needed in between.
meda_status launch_stats_fast(meda_ctx* ctx, const void* q_win, const void* k, float* row_stats, cudaStream_t st) {
  const meda_config& c = ctx->cfg;
  if (((reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(q_win)) & 15u) != 0) return MEDA_ERR_INVALID_ARG;
  CUtensorMap map_k;
  if (!make_rows_map(ctx, &map_k, k, c.n_tokens, c.n_kv_heads, c.n_tokens, 128)) return MEDA_ERR_CUDA;
  WinStatsParams prm;
  prm.q = static_cast<const __nv_bfloat16*>(q_win);
  prm.modality = ctx->ws.modality;
  prm.tile_class = ctx->ws.tile_class;
  prm.partial = ctx->ws.stats_partial;
  prm.row_stats = row_stats;
  prm.coef_vis = ctx->ws.coef_vis;
  prm.coef_text = ctx->ws.coef_text;
  prm.coef_paired = ctx->fast_sweep_grouped ? 1 : 0;
  prm.counters = ctx->ws.stats_counters;
  prm.n = c.n_tokens; prm.hq = c.n_q_heads; prm.group = ctx->group; prm.w = c.window;
  prm.cols = ctx->group * c.window;
  prm.row_blocks = (prm.cols + 255) / 256;
  prm.chunks = ctx->stats_chunks;
  prm.tiles_per_chunk = ctx->stats_tiles_per_chunk;
  prm.tiles_total = (c.n_tokens + 127) / 128;
  prm.sc2 = kLog2e / sqrtf((float)c.head_dim);
  const int items = c.n_kv_heads * prm.row_blocks * prm.chunks;
  {
    LaunchScope scope(ctx, MEDA_K_STATS, st);
    window_stats_kernel<<<std::min(items, ctx->sm_count), kWsThreads, WinStatsSmem::alloc, st>>>(map_k, prm, ctx->ws.status);
  }
  return launch_status();
}

template <int W, int MODE>
void launch_sweep_policy(meda_ctx* ctx, const CUtensorMap& map_k, const CUtensorMap& map_q, float* scores,
                         bool want_entropy, cudaStream_t st) {
  const meda_config& c = ctx->cfg;
  using Policy = SweepPolicy<W, MODE>;
  typename Policy::Params prm;
  prm.modality = ctx->ws.modality;
  prm.vis = ctx->ws.coef_vis;
  prm.text = ctx->ws.coef_text;
  prm.scores = scores;
  prm.ent_partial = want_entropy ? ctx->ws.ent_partial : nullptr;
  prm.n = c.n_tokens; prm.hkv = c.n_kv_heads; prm.cols = ctx->group * c.window;
  prm.n_blocks = (c.n_tokens + 255) / 256;
  prm.sc2 = kLog2e / sqrtf((float)c.head_dim);
  prm.ln_hq = logf((float)c.n_q_heads);
  umma_stream_kernel<Policy><<<std::min(prm.n_blocks, ctx->sm_count), us_threads<Policy>(), StreamShared<Policy>::alloc, st>>>(
      map_k, map_q, prm, ctx->ws.status);
}

template <int W, int MODE>
meda_status raise_sweep_smem() {
  return cudaFuncSetAttribute(umma_stream_kernel<SweepPolicy<W, MODE>>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)StreamShared<SweepPolicy<W, MODE>>::alloc) == cudaSuccess ? MEDA_OK : MEDA_ERR_CUDA;
}

// The scores + entropy sweep for KV groups of 129 .. 256 query rows (grouped-query attention): one launch that
// also finishes the entropy.
template <int W, int MODE>
void launch_window_sweep(meda_ctx* ctx, const CUtensorMap& map_k, const CUtensorMap& map_q, const float* row_stats,
                         float* scores, float* entropy_out, cudaStream_t st) {
  const meda_config& c = ctx->cfg;
  WinSweepParams prm;
  prm.modality = ctx->ws.modality;
  prm.vis = ctx->ws.coef_vis;
  prm.text = ctx->ws.coef_text;
  prm.row_stats = row_stats;
  prm.scores = scores;
  prm.ent_partial = entropy_out ? ctx->ws.ent_partial : nullptr;
  prm.entropy_out = entropy_out;
  prm.done_counter = ctx->ws.sweep_counter;
  prm.n = c.n_tokens; prm.hkv = c.n_kv_heads; prm.cols = ctx->group * c.window;
  prm.n_blocks = (c.n_tokens + 255) / 256;
  prm.a_stages = win_sweep_a_stages(prm.cols);
  prm.sc2 = kLog2e / sqrtf((float)c.head_dim);
  prm.ln_hq = logf((float)c.n_q_heads);
  const WinSweepSmem L(prm.cols, prm.a_stages);
  window_sweep_kernel<W, MODE><<<std::min(prm.n_blocks, ctx->sm_count), kSwThreads, L.alloc(), st>>>(map_k, map_q, prm,
                                                                                                    ctx->ws.status);
}

template <int W, int MODE>
meda_status raise_window_sweep_smem() {
  return cudaFuncSetAttribute(window_sweep_kernel<W, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem) ==
                 cudaSuccess ? MEDA_OK : MEDA_ERR_CUDA;
}

// `coef_ready`: the per-column constants were written by the normaliser sweep that ran just before on this
// stream; otherwise (row_stats handed in by the caller) they are derived from row_stats first.
meda_status launch_sweep_fast(meda_ctx* ctx, int32_t layer, const void* q_win, const void* k, const float* row_stats,
                              float* scores, float* entropy, bool coef_ready, cudaStream_t st) {
  const meda_config& c = ctx->cfg;
  if (((reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(q_win)) & 15u) != 0) return MEDA_ERR_INVALID_ARG;
  const int cols = ctx->group * c.window;
  const bool grouped = ctx->fast_sweep_grouped;     // the kernel for several query heads per KV head
  CUtensorMap map_q, map_k;
  if (!make_rows_map(ctx, &map_q, q_win, (int64_t)c.n_q_heads * c.window, 1, (int64_t)c.n_q_heads * c.window,
                     grouped ? (uint32_t)cols : 128u) ||
      !make_rows_map(ctx, &map_k, k, c.n_tokens, c.n_kv_heads, c.n_tokens, 128))
    return MEDA_ERR_CUDA;
  const int rows = c.n_q_heads * c.window;
  if (!coef_ready) {
    LaunchScope scope(ctx, MEDA_K_STATS_COMBINE, st);
    sweep_coef_kernel<<<(rows + 255) / 256, 256, 0, st>>>(row_stats, ctx->ws.coef_vis, ctx->ws.coef_text, rows,
                                                          (float)c.n_q_heads, grouped);
  }
  if (grouped) {
    LaunchScope scope(ctx, MEDA_K_SWEEP, st);
    float* e_out = entropy ? entropy + layer : nullptr;
    if (c.entropy_mode == 0) launch_window_sweep<32, 0>(ctx, map_k, map_q, row_stats, scores, e_out, st);
    else launch_window_sweep<32, 1>(ctx, map_k, map_q, row_stats, scores, e_out, st);
    return launch_status();
  }
  {
    LaunchScope scope(ctx, MEDA_K_SWEEP, st);
    const bool e = entropy != nullptr;
    if (c.window == 32 && c.entropy_mode == 0) launch_sweep_policy<32, 0>(ctx, map_k, map_q, scores, e, st);
    else if (c.window == 32) launch_sweep_policy<32, 1>(ctx, map_k, map_q, scores, e, st);
    else if (c.entropy_mode == 0) launch_sweep_policy<64, 0>(ctx, map_k, map_q, scores, e, st);
    else launch_sweep_policy<64, 1>(ctx, map_k, map_q, scores, e, st);
  }
  if (entropy) {
    LaunchScope scope(ctx, MEDA_K_ENTROPY_FINAL, st);
    entropy_finalize_kernel<<<1, 256, 0, st>>>(ctx->ws.ent_partial, ((c.n_tokens + 255) / 256) * kUsEpilogueWarps,
                                               row_stats, c.window, entropy + layer);
  }
  return launch_status();
}

// The E_VT term of Eq. 5-6 on the CUDA-core kernels, any dtype: visual query rows at given positions
// against the TEXT keys they see.  Adds -E_VT to entropy[layer].
template <typename T>
meda_status launch_evt(meda_ctx* ctx, int32_t layer, const void* q_vis, const int32_t* q_vis_pos, int32_t rows,
                       const void* k, float* entropy, cudaStream_t st) {
  const meda_config& c = ctx->cfg;
  const float scale = 1.0f / sqrtf((float)c.head_dim);
  const int tiles = generic_tiles(c.n_tokens);
  const int chunks = std::min(kStatsChunks, tiles);
  const int stats_smem = attn_generic_smem(rows, c.head_dim, false).total;
  const int sweep_smem = attn_generic_smem(rows, c.head_dim, true).total;
  if (sweep_smem > kMaxDynSmem - 4096) return MEDA_ERR_SHAPE;
  {
    LaunchScope scope(ctx, MEDA_K_STATS, st);
    stats_partial_kernel<T><<<dim3(chunks, c.n_q_heads), kAttnThreads, stats_smem, st>>>(
        static_cast<const T*>(q_vis), static_cast<const T*>(k), ctx->ws.modality, ctx->ws.stats_partial, c.n_q_heads,
        ctx->group, c.n_tokens, rows, c.head_dim, scale, q_vis_pos, MEDA_TEXT, 1);
  }
  {
    LaunchScope scope(ctx, MEDA_K_STATS_COMBINE, st);
    stats_combine_kernel<<<(c.n_q_heads * rows + 7) / 8, 256, 0, st>>>(ctx->ws.stats_partial, ctx->ws.row_stats_vis, chunks,
                                                                       c.n_q_heads * rows);
  }
  {
    LaunchScope scope(ctx, MEDA_K_SWEEP, st);
    scores_entropy_kernel<T><<<tiles, kAttnThreads, sweep_smem, st>>>(
        static_cast<const T*>(q_vis), static_cast<const T*>(k), ctx->ws.modality, ctx->ws.row_stats_vis, nullptr,
        ctx->ws.ent_partial, c.n_q_heads, ctx->group, c.n_tokens, rows, c.head_dim, scale, c.entropy_mode, 0, 1,
        q_vis_pos, MEDA_TEXT);
  }
  {
    LaunchScope scope(ctx, MEDA_K_ENTROPY_FINAL, st);
    entropy_finalize_kernel<<<1, 256, 0, st>>>(ctx->ws.ent_partial, tiles, ctx->ws.row_stats_vis, rows, entropy + layer, 1);
  }
  return launch_status();
}

// ---- Eq. 8 over every prompt row ---------------------------------------------------------------
// Rows per head of the per-row reference array: a multiple of 128 so that a streamed tile of query
// rows never reads past it.
int64_t prompt_n_pad(const meda_ctx* ctx) { return ((int64_t)ctx->cfg.n_tokens + 127) / 128 * 128; }

// Row runs per key block of the column-sum pass: enough (key block, KV head, run) units for about six per SM.
int prompt_splits(const meda_ctx* ctx) {
  const int64_t units = (int64_t)((ctx->cfg.n_tokens + 255) / 256) * ctx->cfg.n_kv_heads;
  return (int)std::max<int64_t>(1, std::min<int64_t>(8, (6 * (int64_t)ctx->sm_count + units - 1) / units));
}

// Per-row references, then one region that first holds the two partial normalisers of every row and later
// the partial scores of every key.
int64_t prompt_scratch_bytes(const meda_ctx* ctx) {
  if (!ctx->fast) return 0;                            // the CUDA-core path works inside the context's own scratch
  const int64_t n_pad = prompt_n_pad(ctx);
  const int64_t stats_part = 2 * (int64_t)sizeof(float2) * ctx->cfg.n_q_heads * n_pad;
  const int64_t score_part = 2 * (int64_t)sizeof(float) * prompt_splits(ctx) * ctx->cfg.n_kv_heads * n_pad;
  return (int64_t)sizeof(float) * ctx->cfg.n_q_heads * n_pad + std::max(stats_part, score_part);
}

// bf16, head_dim 128: two launches of the streaming tensor-core pipeline over the causal half of the matrix.
meda_status launch_prompt_fast(meda_ctx* ctx, const void* q_all, const void* k, float* scores, void* scratch,
                               cudaStream_t st) {
  const meda_config& c = ctx->cfg;
  if (((reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(q_all) | reinterpret_cast<uintptr_t>(scratch)) & 15u) != 0)
    return MEDA_ERR_INVALID_ARG;
  CUtensorMap map_q, map_k;
  if (!make_rows_map(ctx, &map_q, q_all, c.n_tokens, c.n_q_heads, c.n_tokens, 128) ||
      !make_rows_map(ctx, &map_k, k, c.n_tokens, c.n_kv_heads, c.n_tokens, 128))
    return MEDA_ERR_CUDA;
  const int n_pad = (int)prompt_n_pad(ctx);
  float* ref = static_cast<float*>(scratch);
  float2* partial = reinterpret_cast<float2*>(ref + (size_t)c.n_q_heads * n_pad);
  const float sc2 = kLog2e / sqrtf((float)c.head_dim);
  const int blocks256 = (c.n_tokens + 255) / 256;
  {
    PromptStatsPolicy::Params prm;
    prm.partial = partial;
    prm.n = c.n_tokens; prm.n_pad = n_pad; prm.hq = c.n_q_heads; prm.group = ctx->group;
    prm.row_blocks = blocks256;
    prm.sc2 = sc2;
    LaunchScope scope(ctx, MEDA_K_STATS, st);
    umma_stream_kernel<PromptStatsPolicy><<<(int)std::min<int64_t>((int64_t)blocks256 * c.n_q_heads, ctx->sm_count),
                                            us_threads<PromptStatsPolicy>(), StreamShared<PromptStatsPolicy>::alloc, st>>>(
        map_q, map_k, prm, ctx->ws.status);
  }
  {
    LaunchScope scope(ctx, MEDA_K_STATS_COMBINE, st);
    prompt_ref_kernel<<<4 * ctx->sm_count, 256, 0, st>>>(partial, ref, c.n_q_heads, c.n_tokens, n_pad);
  }
  const int splits = prompt_splits(ctx);
  float* score_part = reinterpret_cast<float*>(partial);     // the partial normalisers are spent once ref is written
  {
    PromptSweepPolicy::Params prm;
    prm.ref = ref;
    prm.partial = score_part;
    prm.n = c.n_tokens; prm.n_pad = n_pad; prm.hq = c.n_q_heads; prm.hkv = c.n_kv_heads; prm.group = ctx->group;
    prm.n_blocks = blocks256;
    prm.splits = splits;
    prm.full_blocks = 0;
    int64_t units = 0;
    for (int blk = 0; blk < blocks256; ++blk) {
      if (prompt_block_tiles(c.n_tokens, blk) >= splits) prm.full_blocks = blk + 1;
      units += (int64_t)c.n_kv_heads * prompt_block_splits(c.n_tokens, blk, splits);
    }
    prm.sc2 = sc2;
    LaunchScope scope(ctx, MEDA_K_SWEEP, st);
    umma_stream_kernel<PromptSweepPolicy><<<(int)std::min<int64_t>(units, ctx->sm_count), us_threads<PromptSweepPolicy>(),
                                            StreamShared<PromptSweepPolicy>::alloc, st>>>(map_k, map_q, prm, ctx->ws.status);
  }
  {
    LaunchScope scope(ctx, MEDA_K_STATS_COMBINE, st);
    prompt_sum_kernel<<<2 * ctx->sm_count, 256, 0, st>>>(score_part, scores, c.n_kv_heads, c.n_tokens, splits);
  }
  return launch_status();
}

// Any dtype and head dimension: the prompt rows in blocks of `window` rows through the CUDA-core kernels
// of the observation window; block b sees the keys up to its last row and adds its column sums.
template <typename T>
meda_status launch_prompt_generic(meda_ctx* ctx, const void* q_all, const void* k, float* scores, cudaStream_t st) {
  const meda_config& c = ctx->cfg;
  const float scale = 1.0f / sqrtf((float)c.head_dim);
  MEDA_CUDA_TRY(cudaMemsetAsync(scores, 0, sizeof(float) * (size_t)c.n_kv_heads * c.n_tokens, st));
  for (int p0 = 0; p0 < c.n_tokens; p0 += c.window) {
    const int rows = std::min(c.window, c.n_tokens - p0);
    const int n_seen = p0 + rows;
    const int tiles = generic_tiles(n_seen);
    const int chunks = std::min(kStatsChunks, tiles);
    AttnView view;
    view.rows_from_pos0 = 1;
    view.pos0 = p0;
    view.q_head_stride = c.n_tokens;
    view.k_head_stride = c.n_tokens;
    view.score_stride = c.n_tokens;
    view.accumulate = 1;
    const T* q_block = static_cast<const T*>(q_all) + (size_t)p0 * c.head_dim;
    {
      LaunchScope scope(ctx, MEDA_K_STATS, st);
      stats_partial_kernel<T><<<dim3(chunks, c.n_q_heads), kAttnThreads, attn_generic_smem(rows, c.head_dim, false).total, st>>>(
          q_block, static_cast<const T*>(k), ctx->ws.modality, ctx->ws.stats_partial, c.n_q_heads, ctx->group, n_seen,
          rows, c.head_dim, scale, nullptr, MEDA_VISUAL, 0, view);
    }
    {
      LaunchScope scope(ctx, MEDA_K_STATS_COMBINE, st);
      stats_combine_kernel<<<(c.n_q_heads * rows + 7) / 8, 256, 0, st>>>(ctx->ws.stats_partial, ctx->ws.row_stats_vis,
                                                                         chunks, c.n_q_heads * rows);
    }
    {
      LaunchScope scope(ctx, MEDA_K_SWEEP, st);
      scores_entropy_kernel<T><<<tiles, kAttnThreads, attn_generic_smem(rows, c.head_dim, true).total, st>>>(
          q_block, static_cast<const T*>(k), ctx->ws.modality, ctx->ws.row_stats_vis, scores, ctx->ws.ent_partial,
          c.n_q_heads, ctx->group, n_seen, rows, c.head_dim, scale, c.entropy_mode, 1, 0, nullptr, MEDA_VISUAL, view);
    }
  }
  return launch_status();
}

// ---- phase B launches ------------------------------------------------------------------------
// bf16, head_dim 128: gather + tcgen05 similarity/arg-max + remap to the less-important order.
meda_status launch_nearest_fast(meda_ctx* ctx, const void* k, const int32_t* budget_row, const int32_t* idx_conserved,
                                const int32_t* idx_less, int32_t* target, int32_t cap, cudaStream_t st) {
  const meda_config& c = ctx->cfg;
  const int n = c.n_tokens;
  if ((reinterpret_cast<uintptr_t>(k) & 15u) != 0) return MEDA_ERR_INVALID_ARG;
  CUtensorMap map_kc;
  if (!make_rows_map(ctx, &map_kc, ctx->ws.kc, ctx->kc_rows, c.n_kv_heads, ctx->kc_rows, kNtTileN)) return MEDA_ERR_CUDA;
  const int max_slots = std::min(cap, n);
  {
    LaunchScope scope(ctx, MEDA_K_PREP, st);
    gather_conserved_bf16_kernel<<<dim3(slot_blocks(ctx, max_slots, 8, c.n_kv_heads), c.n_kv_heads), 256, 0, st>>>(
        static_cast<const __nv_bfloat16*>(k), idx_conserved, budget_row, ctx->ws.kc, ctx->ws.inv_norm, n, cap,
        ctx->kc_rows, ctx->inv_stride);
  }
  {
    const int items = ((n + 255) / 256) * c.n_kv_heads;
    NearestParams prm{static_cast<const __nv_bfloat16*>(k), ctx->ws.inv_norm, budget_row, idx_less, target,
                      n, c.n_kv_heads, cap, ctx->inv_stride};
    LaunchScope scope(ctx, MEDA_K_NEAREST, st);
    nearest_kernel<<<std::min(items, ctx->sm_count), kNtThreads, NearestSmem::alloc, st>>>(map_kc, prm, ctx->ws.status);
  }
  // The budget stays on the device, so both kernels are enqueued and the layer's S decides on the device which
  // of them works: a layer with few slots streams the key cache in row order instead.
  CUtensorMap map_k, map_kc128;
  if (!make_rows_map(ctx, &map_k, k, n, c.n_kv_heads, n, 128) ||
      !make_rows_map(ctx, &map_kc128, ctx->ws.kc, ctx->kc_rows, c.n_kv_heads, ctx->kc_rows, 128))
    return MEDA_ERR_CUDA;
  {
    NearestSmallPolicy::Params prm{ctx->ws.inv_norm, budget_row, idx_conserved, target, n, c.n_kv_heads, cap,
                                   ctx->inv_stride, (n + 255) / 256};
    const int items = prm.row_blocks * c.n_kv_heads;
    LaunchScope scope(ctx, MEDA_K_NEAREST_SMALL, st);
    umma_stream_kernel<NearestSmallPolicy><<<std::min(items, ctx->sm_count), us_threads<NearestSmallPolicy>(),
                                             StreamShared<NearestSmallPolicy>::alloc, st>>>(map_k, map_kc128, prm,
                                                                                            ctx->ws.status);
  }
  return launch_status();
}

// Grouping sort + segmented average (Eq. 12) for any dtype / head_dim.
template <typename T, int D>
void launch_seg_kernels(meda_ctx* ctx, const void* k, const void* v, const int32_t* budget_row,
                        const int32_t* idx_conserved, void* k_out, void* v_out, int32_t* counts, int32_t cap,
                        int evict, cudaStream_t st) {
  const meda_config& c = ctx->cfg;
  const int n = c.n_tokens;
  const int max_slots = std::min(cap, n);
  if (!evict) {
    LaunchScope scope(ctx, MEDA_K_REDUCE, st);
    seg_reduce_kernel<T, D><<<dim3((ctx->seg_chunks + kSegWarps - 1) / kSegWarps, c.n_kv_heads, 2), kSegWarps * 32, 0, st>>>(
        static_cast<const T*>(k), static_cast<const T*>(v), ctx->ws.sort_keys[0], ctx->ws.sort_rows[0],
        ctx->ws.sort_keys[1], ctx->ws.sort_rows[1], ctx->sort_passes, budget_row,
        static_cast<T*>(k_out), static_cast<T*>(v_out), counts, ctx->ws.seg_start, ctx->ws.seg_end, ctx->ws.carry,
        ctx->ws.carry_cnt, n, cap, ctx->seg_chunks);
  }
  LaunchScope scope(ctx, MEDA_K_REDUCE, st);
  if (evict) {
    copy_kept_kernel<T, D><<<dim3(slot_blocks(ctx, max_slots, 8, 2 * c.n_kv_heads), c.n_kv_heads, 2), 256, 0, st>>>(
        static_cast<const T*>(k), static_cast<const T*>(v), idx_conserved, budget_row, static_cast<T*>(k_out),
        static_cast<T*>(v_out), counts, n, cap);
  } else {
    seg_border_kernel<T, D><<<dim3((ctx->seg_chunks + 7) / 8, c.n_kv_heads, 2), 256, 0, st>>>(
        ctx->ws.sort_keys[0], ctx->ws.sort_keys[1], ctx->sort_passes, budget_row, ctx->ws.seg_start, ctx->ws.seg_end,
        ctx->ws.carry, ctx->ws.carry_cnt, static_cast<T*>(k_out), static_cast<T*>(v_out), counts, n, cap,
        ctx->seg_chunks);
  }
}

template <typename T>
meda_status launch_group_reduce(meda_ctx* ctx, const void* k, const void* v, const int32_t* budget_row,
                                const int32_t* idx_conserved, const int32_t* idx_less, const int32_t* target,
                                void* k_out, void* v_out, int32_t* counts, int32_t cap, cudaStream_t st) {
  const meda_config& c = ctx->cfg;
  const int n = c.n_tokens;
  const int evict = c.merge_mode == 1;
  const int max_slots = std::min(cap, n);
  const int32_t* keys = target;
  const int32_t* rows = idx_less;
  if (!evict) {
    const dim3 grid(ctx->sort_chunks, c.n_kv_heads);
    for (int pass = 0; pass < ctx->sort_passes; ++pass) {
      int32_t* ko = ctx->ws.sort_keys[pass & 1];
      int32_t* ro = ctx->ws.sort_rows[pass & 1];
      const int shift = pass * kSortBits;
      {
        LaunchScope scope(ctx, MEDA_K_GROUP, st);
        sort_hist_kernel<<<grid, kSortWarps * 32, 0, st>>>(keys, budget_row, ctx->ws.sort_table, n, cap, shift,
                                                           ctx->sort_chunks);
      }
      {
        LaunchScope scope(ctx, MEDA_K_GROUP, st);
        sort_scatter_kernel<<<grid, kSortWarps * 32, 0, st>>>(keys, rows, idx_conserved, budget_row,
                                                              ctx->ws.sort_table, ko, ro, n, cap, shift,
                                                              ctx->sort_chunks);
      }
      keys = ko;
      rows = ro;
    }
  }
  switch (c.head_dim) {
    case 64: launch_seg_kernels<T, 64>(ctx, k, v, budget_row, idx_conserved, k_out, v_out, counts, cap, evict, st); break;
    case 128: launch_seg_kernels<T, 128>(ctx, k, v, budget_row, idx_conserved, k_out, v_out, counts, cap, evict, st); break;
    default: launch_seg_kernels<T, 256>(ctx, k, v, budget_row, idx_conserved, k_out, v_out, counts, cap, evict, st); break;
  }
  return launch_status();
}

template <typename T>
meda_status launch_merge(meda_ctx* ctx, const void* k, const void* v, const int32_t* budget_row,
                         const int32_t* idx_conserved, const int32_t* idx_less, void* k_out, void* v_out,
                         int32_t* counts, int32_t* target, int32_t cap, cudaStream_t st) {
  const meda_config& c = ctx->cfg;
  const int n = c.n_tokens, d = c.head_dim;
  const int max_slots = std::min(cap, n);
  const int evict = c.merge_mode == 1;
  if (!evict && ctx->fast) {
    meda_status r = launch_nearest_fast(ctx, k, budget_row, idx_conserved, idx_less, target, cap, st);
    if (r != MEDA_OK) return r;
  } else if (!evict) {
    {
      LaunchScope scope(ctx, MEDA_K_PREP, st);
      conserved_inv_norm_kernel<T><<<dim3((max_slots + 7) / 8, c.n_kv_heads), 256, 0, st>>>(
          static_cast<const T*>(k), idx_conserved, budget_row, ctx->ws.inv_norm, n, d, cap, ctx->inv_stride);
    }
    const int nn_smem = (kNnTile * (d + 1) + kNnTile * (kNnDk + 1)) * 4;
    LaunchScope scope(ctx, MEDA_K_NEAREST, st);
    nearest_generic_kernel<T><<<dim3((n + kNnTile - 1) / kNnTile, c.n_kv_heads), 256, nn_smem, st>>>(
        static_cast<const T*>(k), idx_conserved, idx_less, budget_row, ctx->ws.inv_norm, target, n, d, cap,
        ctx->inv_stride);
  }
  return launch_group_reduce<T>(ctx, k, v, budget_row, idx_conserved, idx_less, target, k_out, v_out, counts, cap, st);
}

}  // namespace

// ---- scratch and set-up of meda_row_stats_static -----------------------------------------------
// The partial normalisers of the entry point that must not allocate: [chunks][rows][4] floats at the
// largest size it accepts.  This name is only a device address inside device code; host code must
// ask the runtime for the address (static_stats_scratch below) and never pass the name to a kernel.
static __device__ __align__(256) float g_static_stats_partial[(size_t)MEDA_STATIC_STATS_CHUNKS *
                                                             MEDA_STATIC_STATS_MAX_ROWS * 4];
static_assert(MEDA_STATIC_STATS_CHUNKS == meda::kStatsChunks, "the static scratch is sized for the generic sweep");

namespace {

constexpr int kStaticMaxDevices = 64;
struct StaticStatsDevice {
  float* partial = nullptr;   // device address of g_static_stats_partial on this device
  bool ready = false;
};
StaticStatsDevice g_static_stats_devices[kStaticMaxDevices];
std::mutex g_static_stats_mutex;

// Once per device, with that device current: the array's device address and the kernels' shared
// memory limit.  Neither call allocates.  Returns the address through *partial.
meda_status static_stats_scratch(float** partial) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return MEDA_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_stats_mutex);
  StaticStatsDevice& d = g_static_stats_devices[dev];
  if (!d.ready) {
    float* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_stats_partial) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return MEDA_ERR_CUDA;
    }
    if (raise_dyn_smem(stats_partial_kernel<float>) != MEDA_OK || raise_dyn_smem(stats_partial_kernel<__nv_bfloat16>) != MEDA_OK)
      return MEDA_ERR_CUDA;
    d.partial = ptr;
    d.ready = true;
  }
  *partial = d.partial;
  return MEDA_OK;
}

// ---- decoding step over a layer's cache --------------------------------------------------------
template <typename T, int D, int G>
meda_status launch_decode_g(meda_ctx* ctx, const void* q, const void* k_c, const void* v_c, const int32_t* budget_row,
                            int rows, int cap, float* out, cudaStream_t st) {
  const meda_config& c = ctx->cfg;
  {
    LaunchScope scope(ctx, MEDA_K_DECODE, st);
    decode_partial_kernel<T, D, G><<<dim3(kDecSplits, c.n_kv_heads), kDecWarps * 32, 0, st>>>(
        static_cast<const T*>(q), static_cast<const T*>(k_c), static_cast<const T*>(v_c), budget_row, rows, cap,
        ctx->ws.decode_partial, 1.0f / sqrtf((float)D));
  }
  LaunchScope scope(ctx, MEDA_K_DECODE, st);
  decode_combine_kernel<D><<<c.n_q_heads, D, 0, st>>>(ctx->ws.decode_partial, budget_row, rows, cap, out);
  return launch_status();
}

template <typename T, int D>
meda_status launch_decode(meda_ctx* ctx, const void* q, const void* k_c, const void* v_c, const int32_t* budget_row,
                          int rows, int cap, float* out, cudaStream_t st) {
  switch (ctx->group) {
    case 1: return launch_decode_g<T, D, 1>(ctx, q, k_c, v_c, budget_row, rows, cap, out, st);
    case 2: return launch_decode_g<T, D, 2>(ctx, q, k_c, v_c, budget_row, rows, cap, out, st);
    case 3: return launch_decode_g<T, D, 3>(ctx, q, k_c, v_c, budget_row, rows, cap, out, st);
    case 4: return launch_decode_g<T, D, 4>(ctx, q, k_c, v_c, budget_row, rows, cap, out, st);
    case 7: return launch_decode_g<T, D, 7>(ctx, q, k_c, v_c, budget_row, rows, cap, out, st);
    case 8: return launch_decode_g<T, D, 8>(ctx, q, k_c, v_c, budget_row, rows, cap, out, st);
    default: return MEDA_ERR_UNSUPPORTED;
  }
}

}  // namespace

#pragma GCC visibility push(default)
extern "C" {

meda_status meda_decode_attention(meda_ctx* ctx, int32_t layer, const void* q, const void* k_cache, const void* v_cache,
                                  const int32_t* budgets, int32_t n_rows, int32_t capacity, float* out, void* stream) {
  if (!layer_ok(ctx, layer) || !q || !k_cache || !v_cache || !out) return MEDA_ERR_INVALID_ARG;
  if (capacity < 1 || (!budgets && (n_rows < 1 || n_rows > capacity))) return MEDA_ERR_INVALID_ARG;
  const meda_config& c = ctx->cfg;
  const int32_t* row = budgets ? budgets + (size_t)layer * 3 : nullptr;
  cudaStream_t st = as_stream(stream);
  if (c.head_dim == 64)
    return c.dtype == MEDA_F32 ? launch_decode<float, 64>(ctx, q, k_cache, v_cache, row, n_rows, capacity, out, st)
                               : launch_decode<__nv_bfloat16, 64>(ctx, q, k_cache, v_cache, row, n_rows, capacity, out, st);
  if (c.head_dim == 128)
    return c.dtype == MEDA_F32 ? launch_decode<float, 128>(ctx, q, k_cache, v_cache, row, n_rows, capacity, out, st)
                               : launch_decode<__nv_bfloat16, 128>(ctx, q, k_cache, v_cache, row, n_rows, capacity, out, st);
  return MEDA_ERR_UNSUPPORTED;
}

meda_status meda_row_stats_static(const void* q_win, const void* k, const uint8_t* modality, int32_t n_q_heads,
                                  int32_t n_kv_heads, int32_t head_dim, int32_t n_tokens, int32_t window,
                                  int32_t dtype, float* row_stats, void* stream) {
  if (!q_win || !k || !modality || !row_stats) return MEDA_ERR_INVALID_ARG;
  if (dtype != MEDA_BF16 && dtype != MEDA_F32) return MEDA_ERR_INVALID_ARG;
  if (n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads != 0 || n_tokens < 1 || window < 1 ||
      window > n_tokens || window > kMaxWindow)
    return MEDA_ERR_SHAPE;
  if (head_dim != 64 && head_dim != 128 && head_dim != 256) return MEDA_ERR_SHAPE;
  if ((int64_t)n_q_heads * window > MEDA_STATIC_STATS_MAX_ROWS) return MEDA_ERR_SHAPE;   // beyond the fixed scratch
  const int smem = attn_generic_smem(window, head_dim, false).total;
  if (smem > kMaxDynSmem - 4096) return MEDA_ERR_SHAPE;   // leaves room for the kernel's static shared memory

  float* partial = nullptr;
  meda_status r = static_stats_scratch(&partial);
  if (r != MEDA_OK) return r;

  cudaStream_t st = as_stream(stream);
  const int chunks = std::min(kStatsChunks, generic_tiles(n_tokens));
  const int group = n_q_heads / n_kv_heads;
  const float scale = 1.0f / sqrtf((float)head_dim);
  // Every (chunk, head) block writes its whole slice of `partial` before the second kernel reads
  // it, so what an earlier call left there is never seen.
  if (dtype == MEDA_F32)
    stats_partial_kernel<float><<<dim3(chunks, n_q_heads), kAttnThreads, smem, st>>>(
        static_cast<const float*>(q_win), static_cast<const float*>(k), modality, partial, n_q_heads, group, n_tokens,
        window, head_dim, scale);
  else
    stats_partial_kernel<__nv_bfloat16><<<dim3(chunks, n_q_heads), kAttnThreads, smem, st>>>(
        static_cast<const __nv_bfloat16*>(q_win), static_cast<const __nv_bfloat16*>(k), modality, partial, n_q_heads,
        group, n_tokens, window, head_dim, scale);
  stats_combine_kernel<<<(n_q_heads * window + 7) / 8, 256, 0, st>>>(partial, row_stats, chunks, n_q_heads * window);
  return launch_status();
}

const char* meda_status_string(meda_status status) {
  switch (status) {
    case MEDA_OK: return "ok";
    case MEDA_ERR_INVALID_ARG: return "invalid argument";
    case MEDA_ERR_SHAPE: return "unsupported or inconsistent shape";
    case MEDA_ERR_BUDGET_INFEASIBLE: return "budget infeasible";
    case MEDA_ERR_WORKSPACE: return "output capacity too small";
    case MEDA_ERR_CUDA: return "CUDA runtime error";
    case MEDA_ERR_UNSUPPORTED: return "not implemented";
    case MEDA_ERR_TIMEOUT: return "bounded device wait ran out";
  }
  return "unknown status";
}

meda_status meda_create(const meda_config* config, const meda_span* spans_host, int32_t n_spans, meda_ctx** out) {
  if (out) *out = nullptr;
  if (!config || !spans_host || !out || n_spans <= 0) return MEDA_ERR_INVALID_ARG;
  const meda_config& c = *config;
  if (c.dtype != MEDA_BF16 && c.dtype != MEDA_F32) return MEDA_ERR_INVALID_ARG;
  if (c.entropy_mode < 0 || c.entropy_mode > 1 || c.alloc_mode < 0 || c.alloc_mode > 1 || c.merge_mode < 0 ||
      c.merge_mode > 1)
    return MEDA_ERR_INVALID_ARG;
  if (c.n_layers < 1 || c.n_layers > kMaxLayers || c.n_q_heads < 1 || c.n_kv_heads < 1 ||
      c.n_q_heads % c.n_kv_heads != 0 || c.n_tokens < 1 || c.window < 1 || c.window > c.n_tokens ||
      c.window > kMaxWindow)
    return MEDA_ERR_SHAPE;
  if (c.head_dim != 64 && c.head_dim != 128 && c.head_dim != 256) return MEDA_ERR_SHAPE;
  // byte offsets of a row inside one head's cache are 32-bit in the segmented average, token indices int32 everywhere
  if ((int64_t)c.n_tokens * c.head_dim * (c.dtype == MEDA_F32 ? 4 : 2) >= (int64_t(1) << 32) ||
      (int64_t)c.n_tokens * c.n_kv_heads >= (int64_t(1) << 31))
    return MEDA_ERR_SHAPE;
  if (c.beta_recent < 0 || c.beta_important < 0 || c.beta_recent + c.beta_important <= 0) return MEDA_ERR_INVALID_ARG;
  if (c.min_budget < 1 || c.min_budget > c.n_tokens) return MEDA_ERR_BUDGET_INFEASIBLE;
  if (c.global_budget < (int64_t)c.n_layers * c.min_budget || c.global_budget > (int64_t)c.n_layers * c.n_tokens)
    return MEDA_ERR_BUDGET_INFEASIBLE;
  if (attn_generic_smem(c.window, c.head_dim, true).total > kMaxDynSmem) return MEDA_ERR_SHAPE;

  // modality map from the span table: sorted, disjoint, covering [0, n)
  std::vector<uint8_t> modality((size_t)c.n_tokens);
  int32_t pos = 0, n_visual = 0;
  for (int32_t s = 0; s < n_spans; ++s) {
    const meda_span& sp = spans_host[s];
    if (sp.begin != pos || sp.end <= sp.begin || sp.end > c.n_tokens) return MEDA_ERR_INVALID_ARG;
    if (sp.modality != MEDA_TEXT && sp.modality != MEDA_VISUAL) return MEDA_ERR_INVALID_ARG;
    for (int32_t j = sp.begin; j < sp.end; ++j) modality[(size_t)j] = (uint8_t)sp.modality;
    if (sp.modality == MEDA_VISUAL) n_visual += sp.end - sp.begin;
    pos = sp.end;
  }
  if (pos != c.n_tokens) return MEDA_ERR_INVALID_ARG;

  meda_ctx* ctx = new (std::nothrow) meda_ctx();
  if (!ctx) return MEDA_ERR_CUDA;
  ctx->cfg = c;
  ctx->group = c.n_q_heads / c.n_kv_heads;
  ctx->n_visual = n_visual;
  if (cudaGetDevice(&ctx->device) != cudaSuccess ||
      cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device) != cudaSuccess) {
    delete ctx;
    return MEDA_ERR_CUDA;
  }
  ctx->fast = c.dtype == MEDA_BF16 && c.head_dim == kFastDim;
  ctx->fast_attn = ctx->fast && (c.window == 32 || c.window == 64) && ctx->group * c.window <= kSweepMaxCols;
  const int cols_per_group = ctx->group * c.window;
  // (window 32 only: with 64 rows the kernel's per-thread state does not fit its registers)
  ctx->fast_sweep_grouped = ctx->fast_attn && c.window == 32 && cols_per_group > 128 && cols_per_group <= kSwMaxCols;
  ctx->ent_slots = std::max(generic_tiles(c.n_tokens), ((c.n_tokens + 127) / 128) * kSwEpilogueWarps);
  {
    // Key chunks of the tensor-core normaliser sweep.  An item = (KV head, row block, key chunk); the grid is
    // one block per SM, so a launch takes ceil(items / SMs) waves of (tiles per chunk + about 1.5 tiles of
    // per-item overhead: resident block reload, pipeline refill).  Take the chunk count with the cheapest
    // estimate, at most four waves.
    const int tiles = (c.n_tokens + 127) / 128;
    const int row_blocks = (ctx->group * c.window + 255) / 256;
    const int per_chunk_items = std::max(1, c.n_kv_heads * row_blocks);
    int want = 1;
    double best = 1e300;
    for (int cand = 1; cand <= tiles && cand <= kWsMaxChunks && cand * per_chunk_items <= 4 * ctx->sm_count; ++cand) {
      const int tpc = (tiles + cand - 1) / cand;
      const int chunks = (tiles + tpc - 1) / tpc;
      const int waves = (chunks * per_chunk_items + ctx->sm_count - 1) / ctx->sm_count;
      const double cost = waves * (tpc + 1.5);
      if (cost < best) { best = cost; want = cand; }
    }
    ctx->stats_tiles_per_chunk = (tiles + want - 1) / want;
    ctx->stats_chunks = (tiles + ctx->stats_tiles_per_chunk - 1) / ctx->stats_tiles_per_chunk;
  }

  Workspace& ws = ctx->ws;
  const int64_t n = c.n_tokens, hkv = c.n_kv_heads;
  meda_status st = MEDA_OK;
  const int64_t mod_bytes = (n + 255) / 256 * 256 + 128;
  if (st == MEDA_OK) st = carve(&ws.modality, mod_bytes, &ws.bytes);
  if (st == MEDA_OK && cudaMemset(ws.modality, 2, (size_t)mod_bytes) != cudaSuccess) st = MEDA_ERR_CUDA;
  if (st == MEDA_OK) st = carve(&ws.status, 1, &ws.bytes);
  // the partial normalisers also serve the visual query window of meda_layer_entropy (up to kMaxWindow rows)
  if (st == MEDA_OK)
    st = carve(&ws.stats_partial,
               std::max((int64_t)std::max(kStatsChunks, (ctx->stats_chunks + 7) / 8 * 8) * c.n_q_heads * c.window * 4,
                        (int64_t)kStatsChunks * c.n_q_heads * kMaxWindow * 4), &ws.bytes);
  if (st == MEDA_OK) st = carve(&ws.row_stats_vis, (int64_t)c.n_q_heads * kMaxWindow * 4, &ws.bytes);
  if (ctx->fast_attn) {
    if (st == MEDA_OK) st = carve(&ws.coef_vis, (int64_t)c.n_q_heads * c.window, &ws.bytes);
    if (st == MEDA_OK) st = carve(&ws.coef_text, (int64_t)c.n_q_heads * c.window, &ws.bytes);
    if (st == MEDA_OK && cudaFuncSetAttribute(window_stats_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)WinStatsSmem::alloc) != cudaSuccess) st = MEDA_ERR_CUDA;
    // one class byte per 32-key chunk (0 all text, 1 all visual, 2 mixed or past the end), four per 128-key tile
    const int64_t n_tiles128 = (n + 127) / 128;
    std::vector<uint32_t> tile_class((size_t)n_tiles128, 0u);
    for (int64_t ch = 0; ch < n_tiles128 * 4; ++ch) {
      uint32_t cls = 2u;
      if (ch * 32 + 32 <= n) {
        int vis = 0;
        for (int x = 0; x < 32; ++x) vis += modality[(size_t)(ch * 32 + x)] == MEDA_VISUAL;
        cls = vis == 32 ? 1u : (vis == 0 ? 0u : 2u);
      }
      tile_class[(size_t)(ch / 4)] |= cls << (8 * (ch % 4));
    }
    if (st == MEDA_OK) st = carve(&ws.tile_class, n_tiles128, &ws.bytes);
    if (st == MEDA_OK && cudaMemcpy(ws.tile_class, tile_class.data(), (size_t)n_tiles128 * 4, cudaMemcpyHostToDevice) != cudaSuccess)
      st = MEDA_ERR_CUDA;
    ctx->stats_counter_count = (int)(hkv * ((ctx->group * c.window + 255) / 256) * kWsEpilogueWarps);
    if (st == MEDA_OK) st = carve(&ws.stats_counters, ctx->stats_counter_count, &ws.bytes);
    if (st == MEDA_OK && cudaMemset(ws.stats_counters, 0, (size_t)ctx->stats_counter_count * 4) != cudaSuccess) st = MEDA_ERR_CUDA;
    if (st == MEDA_OK) st = raise_sweep_smem<32, 0>();
    if (st == MEDA_OK) st = raise_sweep_smem<32, 1>();
    if (st == MEDA_OK) st = raise_sweep_smem<64, 0>();
    if (st == MEDA_OK) st = raise_sweep_smem<64, 1>();
    if (st == MEDA_OK) st = raise_window_sweep_smem<32, 0>();
    if (st == MEDA_OK) st = raise_window_sweep_smem<32, 1>();
    if (st == MEDA_OK) st = carve(&ws.sweep_counter, 1, &ws.bytes);
    if (st == MEDA_OK && cudaMemset(ws.sweep_counter, 0, 4) != cudaSuccess) st = MEDA_ERR_CUDA;
  }
  if (st == MEDA_OK) st = carve(&ws.ent_partial, ctx->ent_slots, &ws.bytes);
  if (st == MEDA_OK) st = carve(&ws.decode_partial, (int64_t)c.n_q_heads * kDecSplits * (c.head_dim + 2), &ws.bytes);
  ctx->sort_chunks = (int)((n + kSortBlockItems - 1) / kSortBlockItems + 7) / 8 * 8;   // padded: the scatter reads whole vectors
  ctx->seg_chunks = (int)((n + kSegChunk - 1) / kSegChunk);
  ctx->sort_passes = n <= kSortBins ? 1 : (n <= (int64_t)kSortBins * kSortBins ? 2 : 3);
  for (int i = 0; i < 2; ++i) {
    if (st == MEDA_OK) st = carve(&ws.sort_keys[i], hkv * n, &ws.bytes);
    if (st == MEDA_OK) st = carve(&ws.sort_rows[i], hkv * n, &ws.bytes);
  }
  if (st == MEDA_OK) st = carve(&ws.sort_table, hkv * kSortBins * ctx->sort_chunks, &ws.bytes);
  if (st == MEDA_OK) st = carve(&ws.seg_start, hkv * n, &ws.bytes);
  if (st == MEDA_OK) st = carve(&ws.seg_end, hkv * n, &ws.bytes);
  if (st == MEDA_OK) st = carve(&ws.carry, hkv * ctx->seg_chunks * 2 * 2 * c.head_dim, &ws.bytes);
  if (st == MEDA_OK) st = carve(&ws.carry_cnt, hkv * ctx->seg_chunks * 2, &ws.bytes);
  ctx->kc_rows = (int)((n + 127) / 128 * 128);
  ctx->inv_stride = ctx->kc_rows + 128;
  if (st == MEDA_OK) st = carve(&ws.inv_norm, hkv * ctx->inv_stride, &ws.bytes);
  if (ctx->fast) {
    if (st == MEDA_OK) st = carve(&ws.kc, hkv * ctx->kc_rows * kFastDim, &ws.bytes);
    if (st == MEDA_OK && cudaMemset(ws.kc, 0, (size_t)(hkv * ctx->kc_rows * kFastDim * 2)) != cudaSuccess) st = MEDA_ERR_CUDA;
    if (st == MEDA_OK && cudaMemset(ws.inv_norm, 0, (size_t)(hkv * ctx->inv_stride * 4)) != cudaSuccess) st = MEDA_ERR_CUDA;
    if (st == MEDA_OK) {
      ctx->encode_tiled = resolve_encode_tiled();
      if (!ctx->encode_tiled) st = MEDA_ERR_CUDA;
    }
    if (st == MEDA_OK && cudaFuncSetAttribute(nearest_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)NearestSmem::alloc) != cudaSuccess)
      st = MEDA_ERR_CUDA;
    if (st == MEDA_OK && cudaFuncSetAttribute(umma_stream_kernel<NearestSmallPolicy>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)StreamShared<NearestSmallPolicy>::alloc) != cudaSuccess)
      st = MEDA_ERR_CUDA;
    if (st == MEDA_OK && cudaFuncSetAttribute(umma_stream_kernel<PromptStatsPolicy>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)StreamShared<PromptStatsPolicy>::alloc) != cudaSuccess)
      st = MEDA_ERR_CUDA;
    if (st == MEDA_OK && cudaFuncSetAttribute(umma_stream_kernel<PromptSweepPolicy>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)StreamShared<PromptSweepPolicy>::alloc) != cudaSuccess)
      st = MEDA_ERR_CUDA;
  }
  if (st == MEDA_OK) st = carve(&ws.target, hkv * n, &ws.bytes);
  if (st == MEDA_OK) st = carve(&ws.idx_less, hkv * n, &ws.bytes);
  if (st == MEDA_OK && cudaMemcpy(ws.modality, modality.data(), (size_t)n, cudaMemcpyHostToDevice) != cudaSuccess)
    st = MEDA_ERR_CUDA;
  if (st == MEDA_OK && cudaMemset(ws.status, 0, sizeof(int)) != cudaSuccess) st = MEDA_ERR_CUDA;
  if (st == MEDA_OK) {
    // The limit is a property of the kernel, not of the context: always raise it to the ceiling so
    // that contexts of different shapes can coexist.
    st = c.dtype == MEDA_F32 ? set_generic_attrs<float>() : set_generic_attrs<__nv_bfloat16>();
  }
  // selection: one cluster per KV head while a head's keys fit the cluster's shared memory
  ctx->select_cluster = select_cluster_size(c.n_tokens, c.n_kv_heads, ctx->sm_count, kMaxDynSmem);
  if (st == MEDA_OK && ctx->select_cluster == 8) st = raise_dyn_smem(select_topk_cluster_kernel<8>);
  if (st == MEDA_OK && ctx->select_cluster == 4) st = raise_dyn_smem(select_topk_cluster_kernel<4>);
  if (st == MEDA_OK && ctx->select_cluster == 2) st = raise_dyn_smem(select_topk_cluster_kernel<2>);
  if (st == MEDA_OK && ctx->select_cluster == 1) st = raise_dyn_smem(select_topk_cluster_kernel<1>);
  if (st != MEDA_OK) {
    free_workspace(ws);
    delete ctx;
    cudaGetLastError();
    return st;
  }
  *out = ctx;
  return MEDA_OK;
}

void meda_destroy(meda_ctx* ctx) {
  if (!ctx) return;
  profiler_release(ctx->prof);
  free_workspace(ctx->ws);
  delete ctx;
}

int64_t meda_workspace_bytes(const meda_ctx* ctx) { return ctx ? ctx->ws.bytes : 0; }

int64_t meda_launch_count(const meda_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* meda_kernel_class_name(int32_t kernel_class) {
  static const char* const names[MEDA_K_CLASSES] = {"stats", "stats_combine", "sweep", "entropy_final", "allocate",
                                                    "select", "prep", "nearest", "nearest_small", "group", "reduce",
                                                    "decode"};
  return kernel_class >= 0 && kernel_class < MEDA_K_CLASSES ? names[kernel_class] : nullptr;
}

meda_status meda_profile_enable(meda_ctx* ctx, int32_t enable) {
  if (!ctx) return MEDA_ERR_INVALID_ARG;
  Profiler& p = ctx->prof;
  if (!enable) {
    p.enabled = false;
    return MEDA_OK;
  }
  if (!p.begin) {
    p.begin = static_cast<cudaEvent_t*>(calloc(Profiler::kPool, sizeof(cudaEvent_t)));
    p.end = static_cast<cudaEvent_t*>(calloc(Profiler::kPool, sizeof(cudaEvent_t)));
    p.klass = static_cast<int*>(calloc(Profiler::kPool, sizeof(int)));
    if (!p.begin || !p.end || !p.klass) { profiler_release(p); return MEDA_ERR_CUDA; }
    for (int i = 0; i < Profiler::kPool; ++i) {
      if (cudaEventCreate(&p.begin[i]) != cudaSuccess || cudaEventCreate(&p.end[i]) != cudaSuccess) {
        profiler_release(p);
        return MEDA_ERR_CUDA;
      }
    }
  }
  p.used = 0;
  p.dropped = 0;
  p.enabled = true;
  return MEDA_OK;
}

int64_t meda_profile_dropped(const meda_ctx* ctx) { return ctx ? ctx->prof.dropped : 0; }

meda_status meda_profile_read(meda_ctx* ctx, float* ms_out, int32_t* launches_out) {
  if (!ctx) return MEDA_ERR_INVALID_ARG;
  Profiler& p = ctx->prof;
  float ms[MEDA_K_CLASSES] = {0};
  int32_t cnt[MEDA_K_CLASSES] = {0};
  for (int i = 0; i < p.used; ++i) {
    MEDA_CUDA_TRY(cudaEventSynchronize(p.end[i]));
    float t = 0.f;
    MEDA_CUDA_TRY(cudaEventElapsedTime(&t, p.begin[i], p.end[i]));
    ms[p.klass[i]] += t;
    cnt[p.klass[i]] += 1;
  }
  p.used = 0;
  p.dropped = 0;
  if (ms_out) memcpy(ms_out, ms, sizeof(ms));
  if (launches_out) memcpy(launches_out, cnt, sizeof(cnt));
  return MEDA_OK;
}

meda_status meda_poll_status(meda_ctx* ctx, void* stream) {
  if (!ctx) return MEDA_ERR_INVALID_ARG;
  int code = 0;
  MEDA_CUDA_TRY(cudaStreamSynchronize(as_stream(stream)));
  MEDA_CUDA_TRY(cudaMemcpy(&code, ctx->ws.status, sizeof(int), cudaMemcpyDeviceToHost));
  if (code != 0) {
    MEDA_CUDA_TRY(cudaMemset(ctx->ws.status, 0, sizeof(int)));
    // a kernel that gave up may have left its completion counters mid-count
    if (ctx->ws.stats_counters)
      MEDA_CUDA_TRY(cudaMemset(ctx->ws.stats_counters, 0, (size_t)ctx->stats_counter_count * sizeof(unsigned int)));
    if (ctx->ws.sweep_counter) MEDA_CUDA_TRY(cudaMemset(ctx->ws.sweep_counter, 0, sizeof(unsigned int)));
  }
  return (meda_status)code;
}

meda_status meda_selftest_wait_timeout(meda_ctx* ctx, int64_t wait_cycles, void* stream) {
  if (!ctx || wait_cycles < 1 || wait_cycles > 2000000000ll) return MEDA_ERR_INVALID_ARG;
  wait_timeout_selftest_kernel<<<1, 64, 0, as_stream(stream)>>>((long long)wait_cycles, ctx->ws.status);
  return launch_status();
}

meda_status meda_window_scores(meda_ctx* ctx, int32_t layer, const void* q_win, const void* k, float* row_stats,
                               float* scores, float* entropy, void* stream) {
  if (!layer_ok(ctx, layer) || !q_win || !k || !row_stats || !scores) return MEDA_ERR_INVALID_ARG;
  cudaStream_t st = as_stream(stream);
  meda_status r;
  if (ctx->fast_attn) {
    r = launch_stats_fast(ctx, q_win, k, row_stats, st);
    if (r == MEDA_OK) r = launch_sweep_fast(ctx, layer, q_win, k, row_stats, scores, entropy, true, st);
  } else if (ctx->cfg.dtype == MEDA_F32) {
    r = launch_stats<float>(ctx, q_win, k, row_stats, st);
    if (r == MEDA_OK) r = launch_sweep<float>(ctx, layer, q_win, k, row_stats, scores, entropy, st);
  } else {
    r = launch_stats<__nv_bfloat16>(ctx, q_win, k, row_stats, st);
    if (r == MEDA_OK) r = launch_sweep<__nv_bfloat16>(ctx, layer, q_win, k, row_stats, scores, entropy, st);
  }
  return r;
}

meda_status meda_window_scores_from_stats(meda_ctx* ctx, int32_t layer, const void* q_win, const void* k,
                                          const float* row_stats, float* scores, float* entropy, void* stream) {
  if (!layer_ok(ctx, layer) || !q_win || !k || !row_stats || !scores) return MEDA_ERR_INVALID_ARG;
  cudaStream_t st = as_stream(stream);
  if (ctx->fast_attn) return launch_sweep_fast(ctx, layer, q_win, k, row_stats, scores, entropy, false, st);
  if (ctx->cfg.dtype == MEDA_F32) return launch_sweep<float>(ctx, layer, q_win, k, row_stats, scores, entropy, st);
  return launch_sweep<__nv_bfloat16>(ctx, layer, q_win, k, row_stats, scores, entropy, st);
}

int64_t meda_prompt_scores_scratch_bytes(const meda_ctx* ctx) { return ctx ? prompt_scratch_bytes(ctx) : 0; }

meda_status meda_prompt_scores(meda_ctx* ctx, const void* q_all, const void* k, float* scores, void* scratch,
                               int64_t scratch_bytes, void* stream) {
  if (!ctx || !q_all || !k || !scores) return MEDA_ERR_INVALID_ARG;
  const int64_t need = prompt_scratch_bytes(ctx);
  if (need > 0 && (!scratch || scratch_bytes < need)) return MEDA_ERR_WORKSPACE;
  cudaStream_t st = as_stream(stream);
  if (ctx->fast) return launch_prompt_fast(ctx, q_all, k, scores, scratch, st);
  return ctx->cfg.dtype == MEDA_F32 ? launch_prompt_generic<float>(ctx, q_all, k, scores, st)
                                    : launch_prompt_generic<__nv_bfloat16>(ctx, q_all, k, scores, st);
}

meda_status meda_layer_entropy(meda_ctx* ctx, int32_t layer, const void* q_win, const void* k, const float* row_stats,
                               const void* q_vis, const int32_t* q_vis_pos, int32_t n_vis_rows, float* entropy,
                               void* stream) {
  if (!layer_ok(ctx, layer) || !k || !entropy) return MEDA_ERR_INVALID_ARG;
  const bool with_vis = q_vis || q_vis_pos || n_vis_rows != 0;
  if (with_vis && (!q_vis || !q_vis_pos || n_vis_rows < 1)) return MEDA_ERR_INVALID_ARG;
  if (with_vis && n_vis_rows > kMaxWindow) return MEDA_ERR_SHAPE;
  if (!q_win && !with_vis) return MEDA_ERR_INVALID_ARG;          // nothing to compute
  if (q_win && !row_stats) return MEDA_ERR_INVALID_ARG;
  cudaStream_t st = as_stream(stream);
  meda_status r = MEDA_OK;
  if (q_win) {
    if (ctx->fast_attn) r = launch_sweep_fast(ctx, layer, q_win, k, row_stats, nullptr, entropy, false, st);
    else if (ctx->cfg.dtype == MEDA_F32) r = launch_sweep<float>(ctx, layer, q_win, k, row_stats, nullptr, entropy, st);
    else r = launch_sweep<__nv_bfloat16>(ctx, layer, q_win, k, row_stats, nullptr, entropy, st);
  }
  if (r == MEDA_OK && with_vis)
    r = ctx->cfg.dtype == MEDA_F32 ? launch_evt<float>(ctx, layer, q_vis, q_vis_pos, n_vis_rows, k, entropy, st)
                                   : launch_evt<__nv_bfloat16>(ctx, layer, q_vis, q_vis_pos, n_vis_rows, k, entropy, st);
  return r;
}

meda_status meda_allocate_budgets(meda_ctx* ctx, const float* entropy, int32_t* budgets, void* stream) {
  if (!ctx || !entropy || !budgets) return MEDA_ERR_INVALID_ARG;
  const meda_config& c = ctx->cfg;
  LaunchScope scope(ctx, MEDA_K_ALLOCATE, as_stream(stream));
  allocate_budgets_kernel<<<1, 32, 0, as_stream(stream)>>>(entropy, budgets, c.n_layers, (long long)c.global_budget,
                                                           c.min_budget, c.n_tokens, c.beta_recent, c.beta_important,
                                                           c.alloc_mode, ctx->ws.status);
  return launch_status();
}

meda_status meda_select_topk(meda_ctx* ctx, int32_t layer, const float* scores, const int32_t* budgets,
                             int32_t* idx_conserved, int32_t* idx_less, int32_t out_capacity, void* stream) {
  if (!layer_ok(ctx, layer) || !scores || !budgets || !idx_conserved || !idx_less) return MEDA_ERR_INVALID_ARG;
  if (out_capacity < 1) return MEDA_ERR_WORKSPACE;
  const meda_config& c = ctx->cfg;
  LaunchScope scope(ctx, MEDA_K_SELECT, as_stream(stream));
  if (ctx->select_cluster) {
    const int cs = ctx->select_cluster;
    const int smem = select_cluster_smem(c.n_tokens, cs).total;
    const int32_t* row = budgets + (size_t)layer * 3;
#define MEDA_LAUNCH_SELECT(C)                                                                                  \
  select_topk_cluster_kernel<C><<<C * c.n_kv_heads, kSelThreads, smem, as_stream(stream)>>>(                    \
      scores, ctx->ws.modality, row, idx_conserved, idx_less, c.n_tokens, out_capacity, ctx->ws.status)
    if (cs == 8) MEDA_LAUNCH_SELECT(8);
    else if (cs == 4) MEDA_LAUNCH_SELECT(4);
    else if (cs == 2) MEDA_LAUNCH_SELECT(2);
    else MEDA_LAUNCH_SELECT(1);
#undef MEDA_LAUNCH_SELECT
  } else
    select_topk_kernel<<<c.n_kv_heads, kSelThreads, 0, as_stream(stream)>>>(
        scores, ctx->ws.modality, budgets + (size_t)layer * 3, idx_conserved, idx_less, c.n_tokens, out_capacity,
        ctx->ws.status);
  return launch_status();
}

meda_status meda_merge_kv(meda_ctx* ctx, int32_t layer, const void* k, const void* v, const int32_t* budgets,
                          const int32_t* idx_conserved, const int32_t* idx_less, void* k_out, void* v_out,
                          int32_t* counts, int32_t* target, int32_t out_capacity, void* stream) {
  if (!layer_ok(ctx, layer) || !k || !v || !budgets || !idx_conserved || !idx_less || !k_out || !v_out || !counts)
    return MEDA_ERR_INVALID_ARG;
  if (out_capacity < 1) return MEDA_ERR_WORKSPACE;
  int32_t* tgt = target ? target : ctx->ws.target;
  const int32_t* row = budgets + (size_t)layer * 3;
  if (ctx->cfg.dtype == MEDA_F32)
    return launch_merge<float>(ctx, k, v, row, idx_conserved, idx_less, k_out, v_out, counts, tgt, out_capacity,
                               as_stream(stream));
  return launch_merge<__nv_bfloat16>(ctx, k, v, row, idx_conserved, idx_less, k_out, v_out, counts, tgt, out_capacity,
                                     as_stream(stream));
}

meda_status meda_compress_layer(meda_ctx* ctx, int32_t layer, const void* k, const void* v, const float* scores,
                                const int32_t* budgets, void* k_out, void* v_out, int32_t* counts,
                                int32_t* idx_conserved, int32_t out_capacity, void* stream) {
  if (!layer_ok(ctx, layer) || !k || !v || !scores || !budgets || !k_out || !v_out || !counts || !idx_conserved)
    return MEDA_ERR_INVALID_ARG;
  meda_status r = meda_select_topk(ctx, layer, scores, budgets, idx_conserved, ctx->ws.idx_less, out_capacity, stream);
  if (r != MEDA_OK) return r;
  return meda_merge_kv(ctx, layer, k, v, budgets, idx_conserved, ctx->ws.idx_less, k_out, v_out, counts, nullptr,
                       out_capacity, stream);
}

}  // extern "C"
#pragma GCC visibility pop
