// Shared device helpers and the internal handle layouts of the SSD verify library.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "ssd.h"

namespace ssd {

constexpr int R_MAX = 16;      // most query rows per stream in one forward (gamma + 1 <= 16)
constexpr int ATTN_CHUNK = 64; // keys per split of the generic verify-attention kernel

typedef __nv_bfloat16 bf16;

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<bf16>(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

// Eight consecutive elements (16-byte aligned for bf16, 32-byte for fp32) as floats.
__device__ __forceinline__ void load8(const float* p, float (&o)[8]) {
  float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
  o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w; o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
}
__device__ __forceinline__ void unpack8(uint4 v, float (&o)[8]) {
  // a bf16 is the upper half of an fp32
  o[0] = __uint_as_float(v.x << 16); o[1] = __uint_as_float(v.x & 0xFFFF0000u);
  o[2] = __uint_as_float(v.y << 16); o[3] = __uint_as_float(v.y & 0xFFFF0000u);
  o[4] = __uint_as_float(v.z << 16); o[5] = __uint_as_float(v.z & 0xFFFF0000u);
  o[6] = __uint_as_float(v.w << 16); o[7] = __uint_as_float(v.w & 0xFFFF0000u);
}
__device__ __forceinline__ void load8(const bf16* p, float (&o)[8]) {
  unpack8(*reinterpret_cast<const uint4*>(p), o);
}
// Streaming (read-once) variant for weights: bypass L1 allocation.
__device__ __forceinline__ void load8_stream(const bf16* p, float (&o)[8]) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  unpack8(v, o);
}
__device__ __forceinline__ void load8_stream(const float* p, float (&o)[8]) { load8(p, o); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Which rows a forward pass covers: streams b0..b0+nb-1, R rows each; row m = bi*R + r sits at
// position len[b0+bi] + r of its stream.
struct RowMap {
  int b0, nb, R;
};

struct LayerW {
  const void *norm1, *w_qkv, *b_qkv, *w_o, *norm2, *w_gu, *w_d;
};

}  // namespace ssd

// Device-side view of the weights packed for the persistent small-batch kernel (fast.h).
struct ssd_fast_model {
  bool enabled = false;
  const uint8_t* wstream = nullptr;
  const uint64_t* stream_off = nullptr;
  const uint8_t* chunks = nullptr;
  const int32_t *chunk_cnt = nullptr, *unit_cnt = nullptr, *unit_off = nullptr, *unit_tile = nullptr;
  const float *bias_qkv = nullptr, *gains = nullptr;
  int n_cta = 0, max_units = 0, down_split = 1, o_split = 1, max_stage_k = 0;
  const int32_t* layer_map = nullptr;  // device: layer -> layer of the packed streams (null: identity)
  int n_src_layers = 0;                // layers in the packed streams
};

// Device-side view of the weights packed for the tensor-core projections of batched forwards (tc.h).
struct ssd_tc_layer {
  const uint8_t *w_qkv, *w_o, *w_gu, *w_d;
};
struct ssd_tc_model {
  bool enabled = false;
  std::vector<ssd_tc_layer> layers;
  const uint8_t* head = nullptr;
  int n_sm = 148;  // SMs of the device the model was created on: sizes the K splits
};

struct ssd_model {
  ssd_model_config cfg;
  int el;  // bytes per weight element
  char* arena;
  const void* embed;
  std::vector<ssd::LayerW> layers;
  const void *norm_f, *head;
  const double* inv_freq;  // [head_dim / 2]
  ssd_fast_model fast;
  ssd_tc_model tc;
};

struct ssd_streams {
  ssd_model_config cfg;  // shape the cache was laid out for
  int el;
  int B, cap, max_gamma, max_rows, nsplit_max;
  char* kv;
  size_t kv_layer_elems;  // elements per layer: B * 2 * Hkv * cap * hd
  char* ws;
  size_t ws_bytes;
  // regions of the workspace
  int32_t *len, *pending, *status, *counters, *row_ids, *accept_flags;
  float *h, *qkv, *qrot, *rope_cs, *part, *logits, *row_stats, *xn, *attn_out, *act;
  // staging for the host-buffer entry point
  int32_t *st_tokens, *st_k, *st_y;
  float *st_probs, *st_uni;
  // persistent small-batch kernel: fixed-point residual stream, attention partials and counters,
  // grid-barrier words
  long long* hfix;
  uint32_t *xa, *xb, *xd, *xq;  // projection / attention inputs in tensor-core operand layout
  long long *ssq_a, *ssq_b;
  uint32_t *flags, *epoch_base;
  float* attn_part;    // persistent kernel, key-split attention: per-CTA partials
  uint32_t* attn_cnt;  // and the per-slice arrival counters
  int key_split;       // 1: forwards on these streams use the key-split variant
  // paged cache (ssd_streams_create_paged): pool kv[layer][page][2][Hkv][64][hd], block tables and
  // the free stack in the workspace; cap = max_pages * 64
  int paged, n_pages, max_pages;
  int32_t *page_table, *pages_used, *free_stack, *free_top;
  // batched tensor-core forward: packed operands (inputs of QKV / gate-up / head, of O, of down)
  // and the partial sums of the K-split projections
  uint8_t *tc_xa, *tc_xattn, *tc_xact;
  float* tc_part;
  // host-buffer entry: side stream for the upload of the draft rows, and its two events
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_free = nullptr, ev_probs = nullptr;
  char* h_stage = nullptr;  // pinned host staging of that entry: [tokens | uniforms] then [k | y]
  size_t h_stage_in = 0;
  int split_act;     // persistent kernel: activations as bf16 hi + lo pairs (1) or plain bf16 (0)
  int path;          // 0: pick the persistent kernel when the forward fits it, 1: generic kernels only
  int attn_kernel;   // batched path: 0 by key range per CTA, 1 warp-level kernel, 2 tcgen05 kernel
  long long* trace;  // optional phase-boundary clock trace of the persistent kernel (null: off)
  int trace_cap;
};
