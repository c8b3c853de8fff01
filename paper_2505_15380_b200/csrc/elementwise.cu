// Small memory-bound pieces of the verify forward: id gather, embedding lookup, RMSNorm, the
// rotary table, and the QKV post-processing that rotates q/k and appends K/V to the cache
// (the decoder is the Qwen2.5-style Transformer of Sec. 3.1).
#include <atomic>

#include "kernels.h"

namespace ssd {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }
uint64_t launch_count() { return g_launches.load(std::memory_order_relaxed); }

// Row ids of a verify step: row 0 of stream b is its pending token, rows 1..gamma the draft.
__global__ void gather_verify_ids_kernel(const int32_t* __restrict__ pending,
                                         const int32_t* __restrict__ draft, int gamma, int B,
                                         int32_t* __restrict__ row_ids) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  int R = gamma + 1;
  if (i >= B * R) return;
  int b = i / R, r = i % R;
  row_ids[i] = r == 0 ? pending[b] : draft[b * gamma + r - 1];
}

void launch_gather_verify_ids(const int32_t* pending, const int32_t* draft_tokens, int gamma,
                              int B, int32_t* row_ids, cudaStream_t st) {
  int n = B * (gamma + 1);
  gather_verify_ids_kernel<<<(n + 127) / 128, 128, 0, st>>>(pending, draft_tokens, gamma, B,
                                                            row_ids);
  count_launch();
}

template <typename T>
__global__ void embed_kernel(const T* __restrict__ table, int vocab_in, int d,
                             const int32_t* __restrict__ row_ids, float* __restrict__ h,
                             int32_t* status) {
  int m = blockIdx.x;
  int id = row_ids[m];
  if (id < 0 || id >= vocab_in) {
    if (threadIdx.x == 0) atomicOr(status, SSD_STATUS_BAD_TOKEN);
    id = min(max(id, 0), vocab_in - 1);
  }
  const T* src = table + (size_t)id * d;
  for (int j = threadIdx.x; j < d; j += blockDim.x) h[(size_t)m * d + j] = to_f32<T>(src[j]);
}

void launch_embed(int dtype, const void* table, int vocab_in, int d, const int32_t* row_ids, int M,
                  float* h, int32_t* status, cudaStream_t st) {
  if (dtype == 0)
    embed_kernel<float><<<M, 128, 0, st>>>((const float*)table, vocab_in, d, row_ids, h, status);
  else
    embed_kernel<bf16><<<M, 128, 0, st>>>((const bf16*)table, vocab_in, d, row_ids, h, status);
  count_launch();
}

// cos/sin of position * inv_freq for every row of the forward, in double then rounded once.
__global__ void rope_table_kernel(const int32_t* __restrict__ len, RowMap rm,
                                  const double* __restrict__ inv_freq, int half,
                                  float* __restrict__ cs) {
  int m = blockIdx.x;
  int bi = m / rm.R, r = m % rm.R;
  double pos = (double)(len[rm.b0 + bi] + r);
  for (int j = threadIdx.x; j < half; j += blockDim.x) {
    double s, c;
    sincos(pos * inv_freq[j], &s, &c);
    cs[((size_t)m * half + j) * 2 + 0] = (float)c;
    cs[((size_t)m * half + j) * 2 + 1] = (float)s;
  }
}

void launch_rope_table(const int32_t* len, RowMap rm, const double* inv_freq, int half, float* cs,
                       cudaStream_t st) {
  rope_table_kernel<<<rm.nb * rm.R, 64, 0, st>>>(len, rm, inv_freq, half, cs);
  count_launch();
}

template <typename T>
__global__ void rmsnorm_kernel(const float* __restrict__ h, const T* __restrict__ gain,
                               float* __restrict__ out, int d, float eps) {
  __shared__ float red[32];
  int m = blockIdx.x;
  const float* x = h + (size_t)m * d;
  float ss = 0.f;
  for (int j = threadIdx.x; j < d; j += blockDim.x) ss += x[j] * x[j];
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x < 32) {
    float v = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
    v = warp_sum(v);
    if (threadIdx.x == 0) red[0] = rsqrtf(v / (float)d + eps);
  }
  __syncthreads();
  float inv = red[0];
  for (int j = threadIdx.x; j < d; j += blockDim.x)
    out[(size_t)m * d + j] = x[j] * inv * to_f32<T>(gain[j]);
}

void launch_rmsnorm(int dtype, const float* h, const void* gain, float* out, int M, int d, float eps,
                    cudaStream_t st) {
  if (dtype == 0)
    rmsnorm_kernel<float><<<M, 256, 0, st>>>(h, (const float*)gain, out, d, eps);
  else
    rmsnorm_kernel<bf16><<<M, 256, 0, st>>>(h, (const bf16*)gain, out, d, eps);
  count_launch();
}

// qkv [M, (Hq + 2 Hkv) * hd] fp32 (bias already added) ->
//   qrot [M, Hq * hd] fp32, rotated and pre-scaled by 1/sqrt(hd);
//   K (rotated) and V appended to the cache at slot len + r, in the cache's storage type.
template <typename T>
__global__ void qkv_post_kernel(const float* __restrict__ qkv, const float* __restrict__ cs,
                                float* __restrict__ qrot, T* __restrict__ kv_layer,
                                const int32_t* __restrict__ len, RowMap rm, int cap, int Hq,
                                int Hkv, int hd, float scale, int32_t* status) {
  int m = blockIdx.x;
  int bi = m / rm.R, r = m % rm.R, b = rm.b0 + bi;
  int pos = len[b] + r;
  int half = hd >> 1;
  int ld = (Hq + 2 * Hkv) * hd;
  const float* row = qkv + (size_t)m * ld;
  const float* c = cs + (size_t)m * half * 2;
  for (int i = threadIdx.x; i < Hq * half; i += blockDim.x) {
    int hh = i / half, j = i % half;
    float x1 = row[hh * hd + j], x2 = row[hh * hd + j + half];
    float co = c[2 * j], si = c[2 * j + 1];
    qrot[(size_t)m * Hq * hd + hh * hd + j] = (x1 * co - x2 * si) * scale;
    qrot[(size_t)m * Hq * hd + hh * hd + j + half] = (x2 * co + x1 * si) * scale;
  }
  if (pos < 0 || pos >= cap) {  // never write outside the stream's slice of the cache
    if (threadIdx.x == 0) atomicOr(status, SSD_STATUS_KV_OVERFLOW);
    return;
  }
  const float* krow = row + Hq * hd;
  const float* vrow = krow + Hkv * hd;
  for (int i = threadIdx.x; i < Hkv * half; i += blockDim.x) {
    int g = i / half, j = i % half;
    float x1 = krow[g * hd + j], x2 = krow[g * hd + j + half];
    float co = c[2 * j], si = c[2 * j + 1];
    T* kdst = kv_layer + (((size_t)b * 2 + 0) * Hkv + g) * (size_t)cap * hd + (size_t)pos * hd;
    kdst[j] = from_f32<T>(x1 * co - x2 * si);
    kdst[j + half] = from_f32<T>(x2 * co + x1 * si);
  }
  for (int i = threadIdx.x; i < Hkv * hd; i += blockDim.x) {
    int g = i / hd, j = i % hd;
    T* vdst = kv_layer + (((size_t)b * 2 + 1) * Hkv + g) * (size_t)cap * hd + (size_t)pos * hd;
    vdst[j] = from_f32<T>(vrow[g * hd + j]);
  }
}

void launch_qkv_post(int dtype, const float* qkv, const float* cs, float* qrot, void* kv_layer,
                     const int32_t* len, RowMap rm, int cap, int Hq, int Hkv, int hd,
                     int32_t* status, cudaStream_t st) {
  float scale = 1.0f / sqrtf((float)hd);
  int M = rm.nb * rm.R;
  if (dtype == 0)
    qkv_post_kernel<float><<<M, 128, 0, st>>>(qkv, cs, qrot, (float*)kv_layer, len, rm, cap, Hq,
                                              Hkv, hd, scale, status);
  else
    qkv_post_kernel<bf16><<<M, 128, 0, st>>>(qkv, cs, qrot, (bf16*)kv_layer, len, rm, cap, Hq, Hkv,
                                             hd, scale, status);
  count_launch();
}

// Prefill bookkeeping: len[b] += add; optionally pending[b] = ids[pending_index].
__global__ void advance_len_kernel(int32_t* len, int32_t* pending, int b, int add,
                                   const int32_t* ids, int pending_index) {
  len[b] += add;
  if (pending_index >= 0) pending[b] = ids[pending_index];
}

void launch_advance_len(int32_t* len, int32_t* pending, int b, int add, const int32_t* ids,
                        int pending_index, cudaStream_t st) {
  advance_len_kernel<<<1, 1, 0, st>>>(len, pending, b, add, ids, pending_index);
  count_launch();
}

// O(1) rollback from device arrays: len[b] = src_len[b] (clamped to the capacity).
__global__ void kv_restore_kernel(int32_t* len, int32_t* pending, const int32_t* src_len,
                                  const int32_t* src_pending, int B, int cap) {
  int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  len[b] = min(max(src_len[b], 0), cap);
  pending[b] = src_pending[b];
}

void launch_kv_restore(int32_t* len, int32_t* pending, const int32_t* src_len,
                       const int32_t* src_pending, int B, int cap, cudaStream_t st) {
  kv_restore_kernel<<<(B + 127) / 128, 128, 0, st>>>(len, pending, src_len, src_pending, B, cap);
  count_launch();
}

// Draft bookkeeping: every stream's committed length grows by `add`.
__global__ void advance_all_kernel(int32_t* len, int B, int add, int cap, int32_t* status) {
  int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  int nl = len[b] + add;
  if (nl > cap) {
    atomicOr(status, SSD_STATUS_KV_OVERFLOW);
    nl = cap;
  }
  len[b] = nl;
}

void launch_advance_all(int32_t* len, int B, int add, int cap, int32_t* status, cudaStream_t st) {
  advance_all_kernel<<<(B + 127) / 128, 128, 0, st>>>(len, B, add, cap, status);
  count_launch();
}

}  // namespace ssd
