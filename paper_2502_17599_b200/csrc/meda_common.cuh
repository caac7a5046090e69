// Shared declarations of the CUDA implementation: context layout, device status word, small
// device helpers.  Nothing here is used by (or shared with) the CPU oracle.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/meda.h"

namespace meda {

constexpr int kMaxWindow = 128;
constexpr int kMaxLayers = 1024;
constexpr int kStatsChunks = 32;      // key chunks of the generic normaliser sweep
constexpr int kGenericKeyTile = 64;   // keys per tile in the generic phase-A kernels
constexpr float kCosEps = 1e-8f;      // lower clamp of a key norm (Eq. 11 is silent on zero norms)

struct Workspace {
  uint8_t* modality = nullptr;        // [n padded to a multiple of 256, + 128] 0 = text, 1 = visual, 2 = padding
  float2* coef_vis = nullptr;         // [Hq * w] per-column constants of the tensor-core scores sweep
  float2* coef_text = nullptr;        // [Hq * w]
  uint32_t* tile_class = nullptr;     // [ceil(n / 128)] one class byte per 32-key chunk: 0 text, 1 visual, 2 mixed / padding
  unsigned int* sweep_counter = nullptr;    // blocks of the grouped scores sweep that have finished, zero between launches
  unsigned int* stats_counters = nullptr;   // completion counters of the normaliser sweep's row sets, zero between launches
  int* status = nullptr;              // device status word (first error wins)
  float* stats_partial = nullptr;     // [chunks][Hq][w][4]
  float* row_stats_vis = nullptr;     // [Hq][<= kMaxWindow][4] normalisers of the visual query window (E_VT)
  float* ent_partial = nullptr;       // [ent_slots]
  float* decode_partial = nullptr;    // [Hq][splits][d + 2] partial softmax states of the decoding step
  float* inv_norm = nullptr;          // [Hkv][inv_stride]  1 / max(|k_c|, eps) per conserved slot
  __nv_bfloat16* kc = nullptr;        // [Hkv][kc_rows][128] gathered conserved keys (bf16, head_dim 128 only)
  int32_t* sort_keys[2] = {nullptr, nullptr};   // [Hkv][n] ping-pong: target slot of each sorted entry
  int32_t* sort_rows[2] = {nullptr, nullptr};   // [Hkv][n] ping-pong: token row of each sorted entry
  int32_t* sort_table = nullptr;      // [Hkv][bins][sort blocks] digit counts, then offsets
  int32_t* seg_start = nullptr;       // [Hkv][n] first sorted position of each slot's members
  int32_t* seg_end = nullptr;         // [Hkv][n] one past the last
  float* carry = nullptr;             // [Hkv][seg_chunks][2][2 * d] partial sums of slots that cross chunk borders
  int32_t* carry_cnt = nullptr;       // [Hkv][seg_chunks][2]
  int32_t* target = nullptr;          // [Hkv][n]  used when the caller passes no target array
  int32_t* idx_less = nullptr;        // [Hkv][n]  used by meda_compress_layer
  int64_t bytes = 0;
};

}  // namespace meda

namespace meda {
// Optional per-launch timing: pairs of events recorded around kernel launches.
struct Profiler {
  static constexpr int kPool = 16384;
  bool enabled = false;
  cudaEvent_t* begin = nullptr;   // [kPool]
  cudaEvent_t* end = nullptr;     // [kPool]
  int* klass = nullptr;           // [kPool]
  int used = 0;
  int64_t dropped = 0;            // launches since the last read that found the pool full and went untimed
};
}  // namespace meda

struct meda_ctx {
  meda_config cfg;
  meda::Profiler prof;
  int64_t launches = 0;
  int device = 0;
  int sm_count = 0;
  int group = 1;          // query heads per KV head
  int n_visual = 0;
  int ent_slots = 0;      // entries of ent_partial written by one entropy sweep
  int inv_stride = 0;     // floats per head in ws.inv_norm (padded so 128-wide slices can be read whole)
  int kc_rows = 0;        // rows per head in ws.kc
  int sort_chunks = 0;    // blocks per head in the grouping sort (columns of its digit table)
  int seg_chunks = 0;     // warp-chunks per head in the segmented average
  int sort_passes = 1;    // 9-bit digit passes needed to order slots < n_tokens
  bool fast = false;      // bf16 with head_dim 128: tensor-core kernels are used
  bool fast_attn = false; // ... and window 32 or 64: phase A runs on the tensor cores too
  bool fast_sweep_grouped = false;   // ... and 129 .. 256 query rows per KV head: the grouped scores sweep
  int select_cluster = 0;        // blocks per thread-block cluster (one cluster per KV head) of the selection; 0: single-block kernel
  int stats_chunks = 0;   // key chunks of the tensor-core normaliser sweep
  int stats_tiles_per_chunk = 0;
  int stats_counter_count = 0;
  void* encode_tiled = nullptr;   // cuTensorMapEncodeTiled, resolved through the runtime
  meda::Workspace ws;
};

namespace meda {

template <typename T>
__device__ __forceinline__ float to_f32(T x);
template <>
__device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__device__ __forceinline__ T from_f32(float x);
template <>
__device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// First error wins; later ones are dropped.
__device__ __forceinline__ void set_status(int* status, int code) { atomicCAS(status, 0, code); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// (m, z) <- merge of two online-softmax states; an empty state is (-inf, 0).
__device__ __forceinline__ void merge_mz(float& m, float& z, float m2, float z2) {
  float mn = fmaxf(m, m2);
  if (mn == -INFINITY) { m = mn; z = 0.f; return; }
  z = z * __expf(m - mn) + z2 * __expf(m2 - mn);
  m = mn;
}

}  // namespace meda
