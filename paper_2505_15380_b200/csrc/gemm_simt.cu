// Generic weight-streaming projection kernel (any shape; fp32 or bf16 weights; fp32 activations
// and accumulation): C[M,N] = A[M,K] * W[N,K]^T.  One warp owns two adjacent weight rows (output
// columns) and streams them once with 16-byte loads while MT activation rows sit in shared memory
// (staged K_CHUNK columns at a time); the K dimension is split over the lanes and reduced with
// shuffles.  The projections of the verify forward (Sec. 3.1 decoder) are skinny
// (M = B * (gamma+1) rows), so the weights dominate the bytes.
#include "kernels.h"

namespace ssd {

constexpr int GEMM_MT = 8;        // activation rows per CTA pass
constexpr int GEMM_WARPS = 8;     // warps per CTA, two columns each
constexpr int GEMM_KC = 2048;     // activation columns staged per pass (8 * 2048 * 4 B = 64 KB)

template <typename T, int EPI, int KS>
__global__ void __launch_bounds__(GEMM_WARPS * 32)
gemm_simt_kernel(const float* __restrict__ A, int lda, const T* __restrict__ W,
                 const T* __restrict__ bias, float* __restrict__ C, int ldc, int M, int N, int K) {
  // KS warps share one pair of columns, each taking every KS-th 256-element slice of K; the
  // CTA covers NG = GEMM_WARPS / KS column pairs.
  constexpr int NG = GEMM_WARPS / KS;
  extern __shared__ __align__(16) float As[];  // [GEMM_MT][kc]
  __shared__ float red[GEMM_WARPS][GEMM_MT][2];
  const int m0 = blockIdx.y * GEMM_MT;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int grp = warp / KS, ks = warp % KS;
  const int n0 = (blockIdx.x * NG + grp) * 2;
  const bool active = n0 < N;
  const bool has1 = n0 + 1 < N;
  const T* w0 = W + (size_t)(active ? n0 : 0) * K;
  const T* w1 = W + (size_t)(has1 ? n0 + 1 : (active ? n0 : 0)) * K;
  const int kc_max = K < GEMM_KC ? K : GEMM_KC;
  float acc0[GEMM_MT], acc1[GEMM_MT];
#pragma unroll
  for (int r = 0; r < GEMM_MT; ++r) acc0[r] = acc1[r] = 0.f;
  for (int k0 = 0; k0 < K; k0 += GEMM_KC) {
    const int kc = min(GEMM_KC, K - k0);  // multiple of 8
    __syncthreads();
    for (int i = tid; i < GEMM_MT * (kc >> 2); i += blockDim.x) {
      int r = i / (kc >> 2), c = i % (kc >> 2);
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (m0 + r < M) v = *reinterpret_cast<const float4*>(A + (size_t)(m0 + r) * lda + k0 + c * 4);
      *reinterpret_cast<float4*>(As + (size_t)r * kc_max + c * 4) = v;
    }
    __syncthreads();
    if (active) {
      const int nch = kc >> 3;
      for (int c = lane + 32 * ks; c < nch; c += 64 * KS) {
        // two 16-byte chunks per column in flight before any arithmetic
        const int c2 = c + 32 * KS;
        const bool two = c2 < nch;
        float a[8], x0[8], x1[8], y0[8], y1[8];
        load8_stream(w0 + k0 + c * 8, x0);
        load8_stream(w1 + k0 + c * 8, x1);
        load8_stream(w0 + k0 + (two ? c2 : c) * 8, y0);
        load8_stream(w1 + k0 + (two ? c2 : c) * 8, y1);
#pragma unroll
        for (int r = 0; r < GEMM_MT; ++r) {
          load8(As + (size_t)r * kc_max + c * 8, a);
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            acc0[r] = fmaf(a[e], x0[e], acc0[r]);
            acc1[r] = fmaf(a[e], x1[e], acc1[r]);
          }
        }
        if (two) {
#pragma unroll
          for (int r = 0; r < GEMM_MT; ++r) {
            load8(As + (size_t)r * kc_max + c2 * 8, a);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              acc0[r] = fmaf(a[e], y0[e], acc0[r]);
              acc1[r] = fmaf(a[e], y1[e], acc1[r]);
            }
          }
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < GEMM_MT; ++r) {
    acc0[r] = warp_sum(acc0[r]);
    acc1[r] = warp_sum(acc1[r]);
  }
  if (KS > 1) {
    if (lane == 0) {
#pragma unroll
      for (int r = 0; r < GEMM_MT; ++r) {
        red[warp][r][0] = acc0[r];
        red[warp][r][1] = acc1[r];
      }
    }
    __syncthreads();
    if (ks == 0 && lane == 0) {
#pragma unroll
      for (int r = 0; r < GEMM_MT; ++r) {
        float s0 = 0.f, s1 = 0.f;
        for (int j = 0; j < KS; ++j) {  // fixed order: bit-reproducible
          s0 += red[warp + j][r][0];
          s1 += red[warp + j][r][1];
        }
        acc0[r] = s0;
        acc1[r] = s1;
      }
    }
  }
  if (!active || ks != 0 || lane != 0) return;
#pragma unroll
  for (int r = 0; r < GEMM_MT; ++r) {
    int m = m0 + r;
    if (m >= M) break;
    if (EPI == EPI_STORE_F32) {
      C[(size_t)m * ldc + n0] = acc0[r] + (bias ? to_f32<T>(bias[n0]) : 0.f);
      if (has1) C[(size_t)m * ldc + n0 + 1] = acc1[r] + (bias ? to_f32<T>(bias[n0 + 1]) : 0.f);
    } else if (EPI == EPI_RESIDUAL) {
      C[(size_t)m * ldc + n0] += acc0[r];
      if (has1) C[(size_t)m * ldc + n0 + 1] += acc1[r];
    } else {  // EPI_SWIGLU: row 2j = gate_j, row 2j+1 = up_j
      float g = acc0[r], u = acc1[r];
      C[(size_t)m * ldc + (n0 >> 1)] = g / (1.f + expf(-g)) * u;
    }
  }
}

template <typename T, int EPI, int KS>
static cudaError_t launch_ks(const float* A, int lda, const void* W, const void* bias, float* C,
                             int ldc, int M, int N, int K, cudaStream_t st) {
  size_t smem = (size_t)GEMM_MT * (K < GEMM_KC ? K : GEMM_KC) * sizeof(float);
  auto kern = gemm_simt_kernel<T, EPI, KS>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  constexpr int cols = (GEMM_WARPS / KS) * 2;
  dim3 grid((N + cols - 1) / cols, (M + GEMM_MT - 1) / GEMM_MT);
  kern<<<grid, GEMM_WARPS * 32, smem, st>>>(A, lda, (const T*)W, (const T*)bias, C, ldc, M, N, K);
  count_launch();
  return cudaGetLastError();
}

template <typename T, int EPI>
static cudaError_t launch_t(const float* A, int lda, const void* W, const void* bias, float* C,
                            int ldc, int M, int N, int K, cudaStream_t st) {
  if ((K & 7) || (lda & 3) || (EPI == EPI_SWIGLU && (N & 1))) return cudaErrorInvalidValue;
  // split K over more warps when there are too few columns to fill the GPU
  const int row_tiles = (M + GEMM_MT - 1) / GEMM_MT;
  int ks = 1;
  // (each CTA stages the activations once, so more CTAs also means more L2 reads: stop at one wave)
  while (ks < 8 && (long)((N + 16 / ks - 1) / (16 / ks)) * row_tiles < 148) ks *= 2;
  switch (ks) {
    case 1: return launch_ks<T, EPI, 1>(A, lda, W, bias, C, ldc, M, N, K, st);
    case 2: return launch_ks<T, EPI, 2>(A, lda, W, bias, C, ldc, M, N, K, st);
    case 4: return launch_ks<T, EPI, 4>(A, lda, W, bias, C, ldc, M, N, K, st);
    default: return launch_ks<T, EPI, 8>(A, lda, W, bias, C, ldc, M, N, K, st);
  }
}

cudaError_t launch_gemm_simt(int dtype, int epi, const float* A, int lda, const void* W,
                             const void* bias, float* C, int ldc, int M, int N, int K,
                             cudaStream_t st) {
#define SSD_GEMM_CASE(T)                                                                  \
  switch (epi) {                                                                          \
    case EPI_STORE_F32: return launch_t<T, EPI_STORE_F32>(A, lda, W, bias, C, ldc, M, N, K, st); \
    case EPI_RESIDUAL: return launch_t<T, EPI_RESIDUAL>(A, lda, W, bias, C, ldc, M, N, K, st);   \
    case EPI_SWIGLU: return launch_t<T, EPI_SWIGLU>(A, lda, W, bias, C, ldc, M, N, K, st);       \
  }
  if (dtype == 0) {
    SSD_GEMM_CASE(float)
  } else {
    SSD_GEMM_CASE(bf16)
  }
#undef SSD_GEMM_CASE
  return cudaErrorInvalidValue;
}

}  // namespace ssd
