// Generic verify attention (Eq. 4: the gamma+1 new rows of a stream attend to the cached prefix
// and, causally, to each other), grouped-query, any storage type, split over the key axis.
//
// Grid (split, kv head, stream).  A CTA stages its chunk of ATTN_CHUNK keys/values (fp32) and all
// G*R query rows of the kv head in shared memory; each warp then walks its rows with an online
// softmax (lane = key for the scores, lane = channel for the weighted sum) and writes an
// un-normalised partial (acc[hd], running max, running sum) per (row, head, split).  A second
// kernel merges the partials of a row by log-sum-exp weights.
#include <math_constants.h>

#include "kernels.h"

namespace ssd {

constexpr int ATTN_WARPS = 4;

template <typename T, int HD>
__global__ void __launch_bounds__(ATTN_WARPS * 32)
attn_split_kernel(const float* __restrict__ qrot, const T* __restrict__ kv_layer,
                  const int32_t* __restrict__ len, RowMap rm, int cap, int Hq, int Hkv,
                  float* __restrict__ part, int nsplit_max) {
  constexpr int NI = HD / 32;
  constexpr int KP = HD + 1;  // padded key row: lane = key reads are conflict-free
  extern __shared__ __align__(16) float smem[];
  const int s = blockIdx.x, g = blockIdx.y, bi = blockIdx.z, b = rm.b0 + bi;
  const int R = rm.R, G = Hq / Hkv, NQ = G * R;
  const int L = len[b];
  const int total = min(L + R, cap);
  const int k_begin = s * ATTN_CHUNK;
  if (k_begin >= total) return;
  const int k_end = min(k_begin + ATTN_CHUNK, total);
  const int nk = k_end - k_begin;
  float* Ks = smem;                      // [ATTN_CHUNK][KP]
  float* Vs = Ks + ATTN_CHUNK * KP;      // [ATTN_CHUNK][HD]
  float* Qs = Vs + ATTN_CHUNK * HD;      // [NQ][HD]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const T* kbase = kv_layer + (((size_t)b * 2 + 0) * Hkv + g) * (size_t)cap * HD + (size_t)k_begin * HD;
  const T* vbase = kv_layer + (((size_t)b * 2 + 1) * Hkv + g) * (size_t)cap * HD + (size_t)k_begin * HD;
  for (int i = tid; i < nk * (HD / 8); i += blockDim.x) {
    int key = i / (HD / 8), c = i % (HD / 8);
    float kx[8], vx[8];
    load8(kbase + (size_t)key * HD + c * 8, kx);
    load8(vbase + (size_t)key * HD + c * 8, vx);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      Ks[key * KP + c * 8 + e] = kx[e];
      Vs[key * HD + c * 8 + e] = vx[e];
    }
  }
  for (int i = tid; i < NQ * HD; i += blockDim.x) {
    int row = i / HD, d = i % HD;       // row = r * G + hl
    int r = row / G, hl = row % G;
    Qs[i] = qrot[((size_t)(bi * R + r) * Hq + g * G + hl) * HD + d];
  }
  __syncthreads();
  for (int row = warp; row < NQ; row += ATTN_WARPS) {
    const int r = row / G, hl = row % G;
    const int last_visible = L + r;      // row r sees keys 0..len+r
    float m_run = -CUDART_INF_F, l_run = 0.f, acc[NI];
#pragma unroll
    for (int i = 0; i < NI; ++i) acc[i] = 0.f;
    const float* q = Qs + row * HD;
    for (int t0 = 0; t0 < nk; t0 += 32) {
      const int kl = t0 + lane;
      const bool valid = kl < nk && (k_begin + kl) <= last_visible;
      float sc = 0.f;
      if (valid) {
        const float* kr = Ks + kl * KP;
#pragma unroll 8
        for (int d = 0; d < HD; ++d) sc = fmaf(q[d], kr[d], sc);
      }
      float tmax = warp_max(valid ? sc : -CUDART_INF_F);
      if (tmax == -CUDART_INF_F) continue;  // nothing visible in this tile (uniform per warp)
      float m_new = fmaxf(m_run, tmax);
      float p = valid ? expf(sc - m_new) : 0.f;
      float corr = expf(m_run - m_new);     // m_run = -inf gives 0
      l_run = l_run * corr + warp_sum(p);
#pragma unroll
      for (int i = 0; i < NI; ++i) acc[i] *= corr;
      const int lim = min(32, nk - t0);
      for (int kk = 0; kk < lim; ++kk) {
        float pk = __shfl_sync(0xffffffffu, p, kk);
        const float* vr = Vs + (t0 + kk) * HD;
#pragma unroll
        for (int i = 0; i < NI; ++i) acc[i] = fmaf(pk, vr[lane + 32 * i], acc[i]);
      }
      m_run = m_new;
    }
    const int m = bi * R + r, h = g * G + hl;
    float* dst = part + (((size_t)m * Hq + h) * nsplit_max + s) * (HD + 2);
#pragma unroll
    for (int i = 0; i < NI; ++i) dst[lane + 32 * i] = acc[i];
    if (lane == 0) {
      dst[HD] = m_run;
      dst[HD + 1] = l_run;
    }
  }
}

template <typename T, int HD>
__global__ void attn_merge_kernel(const float* __restrict__ part, const int32_t* __restrict__ len,
                                  RowMap rm, int cap, int Hq, int nsplit_max, float* __restrict__ out) {
  const int h = blockIdx.x, m = blockIdx.y;
  const int bi = m / rm.R, b = rm.b0 + bi;
  const int total = min(len[b] + rm.R, cap);
  const int ns = (total + ATTN_CHUNK - 1) / ATTN_CHUNK;
  const float* src = part + ((size_t)m * Hq + h) * nsplit_max * (HD + 2);
  float m_tot = -CUDART_INF_F;
  for (int s = 0; s < ns; ++s) m_tot = fmaxf(m_tot, src[s * (HD + 2) + HD]);
  float denom = 0.f;
  for (int s = 0; s < ns; ++s) {
    float ms = src[s * (HD + 2) + HD];
    if (ms != -CUDART_INF_F) denom += expf(ms - m_tot) * src[s * (HD + 2) + HD + 1];
  }
  for (int d = threadIdx.x; d < HD; d += blockDim.x) {
    float o = 0.f;
    for (int s = 0; s < ns; ++s) {
      float ms = src[s * (HD + 2) + HD];
      if (ms != -CUDART_INF_F) o += expf(ms - m_tot) * src[s * (HD + 2) + d];
    }
    out[((size_t)m * Hq + h) * HD + d] = o / denom;
  }
}

template <typename T, int HD>
static cudaError_t launch_t(const float* qrot, const void* kv_layer, const int32_t* len, RowMap rm,
                            int cap, int Hq, int Hkv, float* part, int nsplit_max, float* out,
                            cudaStream_t st) {
  const int NQ = (Hq / Hkv) * rm.R;
  size_t smem = sizeof(float) * ((size_t)ATTN_CHUNK * (HD + 1) + (size_t)ATTN_CHUNK * HD + (size_t)NQ * HD);
  auto kern = attn_split_kernel<T, HD>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  dim3 grid(nsplit_max, Hkv, rm.nb);
  kern<<<grid, ATTN_WARPS * 32, smem, st>>>(qrot, (const T*)kv_layer, len, rm, cap, Hq, Hkv, part,
                                            nsplit_max);
  count_launch();
  dim3 mg(Hq, rm.nb * rm.R);
  attn_merge_kernel<T, HD><<<mg, HD < 64 ? 32 : 64, 0, st>>>(part, len, rm, cap, Hq, nsplit_max,
                                                             out);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_attention_simt(int dtype, const float* qrot, const void* kv_layer,
                                  const int32_t* len, RowMap rm, int cap, int Hq, int Hkv, int hd,
                                  float* part, int nsplit_max, float* out, cudaStream_t st) {
#define SSD_ATTN_CASE(T)                                                                          \
  switch (hd) {                                                                                   \
    case 32: return launch_t<T, 32>(qrot, kv_layer, len, rm, cap, Hq, Hkv, part, nsplit_max, out, st);  \
    case 64: return launch_t<T, 64>(qrot, kv_layer, len, rm, cap, Hq, Hkv, part, nsplit_max, out, st);  \
    case 128: return launch_t<T, 128>(qrot, kv_layer, len, rm, cap, Hq, Hkv, part, nsplit_max, out, st); \
  }
  if (dtype == 0) {
    SSD_ATTN_CASE(float)
  } else {
    SSD_ATTN_CASE(bf16)
  }
#undef SSD_ATTN_CASE
  return cudaErrorInvalidValue;
}

}  // namespace ssd
