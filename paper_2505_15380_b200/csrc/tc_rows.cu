// Row-wise kernels of the batched verify forward (Eq. 4's decoder pass for more than 16 rows):
// what sits between the tensor-core projections.  Each consumes a projection's partial sums
// (one slab per K slice, added here in a fixed order, so results are bit-reproducible) and
// produces the next projection's input already packed as a tensor-core operand (tc.h).
#include "kernels.h"
#include "tc.h"

namespace ssd {

namespace {

// Columns (k, k + 1), k even, of one token of a packed operand (chunks of Mc rows: tc.h); `row`
// points at the token's row term (tc_act_row_off): bf16 leading parts and remainders.
__device__ __forceinline__ void store_pair(uint8_t* row, int Mc, int k, float x0, float x1) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
  const __nv_bfloat162 l = __floats2bfloat162_rn(x0 - __low2float(h), x1 - __high2float(h));
  const size_t off = tc_act_col_off(Mc, k);
  *reinterpret_cast<__nv_bfloat162*>(row + off) = h;
  *reinterpret_cast<__nv_bfloat162*>(row + off + (size_t)Mc * 16) = l;
}

// Sum over the K slices of a projection's partial sums for two adjacent columns, in slice order
// (bit-reproducible).  The loads of up to 24 slices are in flight together: the kernels that call
// this are one dependent round trip to L2 after another, so every slice waited for separately is
// a microsecond (measured: rounds of eight cost 1.5 us more on 21 slices).  With many rows the
// kernels are built with eight in flight instead, which keeps them at four CTAs per SM: 448 rows
// then still run as one wave.
template <int NF>
__device__ __forceinline__ float2 sum_slices(float2 v, const float* __restrict__ p, size_t slice_stride, int nsplit) {
  for (int s = 0; s < nsplit; s += NF) {
    float2 t[NF];
#pragma unroll
    for (int i = 0; i < NF; ++i)
      t[i] = s + i < nsplit ? __ldcg(reinterpret_cast<const float2*>(p + (size_t)(s + i) * slice_stride))
                            : make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < NF; ++i) {
      if (s + i < nsplit) {
        v.x += t[i].x;
        v.y += t[i].y;
      }
    }
  }
  return v;
}

constexpr int TC_ROWS_DEEP = 256;  // up to this many rows (CTAs) the deep variant still is one wave

// One CTA per row.  h[m, :] += sum_s part[s][m][:]; out = h / rms(h) * gain, packed.
template <int NF, int MINB>
__global__ void __launch_bounds__(256, MINB)
tc_norm_pack_kernel(float* __restrict__ h, const float* __restrict__ part, int nsplit, int ld_part, int Mpad,
                    int Mc, int d, const bf16* __restrict__ gain, float eps, uint8_t* __restrict__ apack) {
  extern __shared__ float row[];
  __shared__ float red[8];
  const int m = blockIdx.x, tid = threadIdx.x;
  tc_pdl_trigger();
  tc_pdl_wait();
  float ss = 0.f;
  for (int j = tid * 2; j < d; j += 512) {
    float2 v = *reinterpret_cast<const float2*>(h + (size_t)m * d + j);
    if (nsplit > 0) {
      v = sum_slices<NF>(v, part + (size_t)m * ld_part + j, (size_t)Mpad * ld_part, nsplit);
      *reinterpret_cast<float2*>(h + (size_t)m * d + j) = v;
    }
    row[j] = v.x;
    row[j + 1] = v.y;
    ss += v.x * v.x + v.y * v.y;
  }
  ss = warp_sum(ss);
  if ((tid & 31) == 0) red[tid >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  const float inv = rsqrtf(tot / (float)d + eps);
  uint8_t* arow = apack + tc_act_row_off(Mc, (d + 15) >> 4, m);
  for (int j = tid * 2; j < d; j += 512) {
    const float2 g = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(gain + j));
    store_pair(arow, Mc, j, row[j] * inv * g.x, row[j + 1] * inv * g.y);
  }
}

__global__ void tc_pack_rows_kernel(const float* __restrict__ x, int K, int Mc, uint8_t* __restrict__ apack) {
  const int m = blockIdx.x;
  uint8_t* arow = apack + tc_act_row_off(Mc, (K + 15) >> 4, m);
  for (int j = threadIdx.x * 2; j < K; j += blockDim.x * 2)
    store_pair(arow, Mc, j, x[(size_t)m * K + j], x[(size_t)m * K + j + 1]);
}

// One CTA per row: q/k/v = sum of the K slices + bias; rotate q and k by the row's position
// (rotate-half pairs (j, j + hd/2)); q scaled by 1/sqrt(hd) to qrot; K (rotated) and V to the
// cache at slot len + r.
template <int NF, int MINB>
__global__ void __launch_bounds__(256, MINB)
tc_qkv_post_kernel(const float* __restrict__ part, int nsplit, int ld_part, int Mpad,
                   const bf16* __restrict__ bias, const float* __restrict__ cs, float* __restrict__ qrot,
                   bf16* __restrict__ kv_layer, const int32_t* __restrict__ len, RowMap rm, int cap, int Hq,
                   int Hkv, int hd, float scale, const int32_t* __restrict__ page_table, int max_pages,
                   int32_t* status) {
  extern __shared__ float row[];  // [(Hq + 2 Hkv) * hd]
  const int m = blockIdx.x, tid = threadIdx.x;
  tc_pdl_trigger();
  tc_pdl_wait();
  const int bi = m / rm.R, r = m % rm.R, b = rm.b0 + bi;
  const int pos = len[b] + r, half = hd >> 1, nq = (Hq + 2 * Hkv) * hd;
  for (int j = tid * 2; j < nq; j += 512) {
    float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(bias + j));
    v = sum_slices<NF>(v, part + (size_t)m * ld_part + j, (size_t)Mpad * ld_part, nsplit);
    row[j] = v.x;
    row[j + 1] = v.y;
  }
  __syncthreads();
  const float* c = cs + (size_t)m * half * 2;
  for (int i = tid; i < Hq * half; i += 256) {
    const int hh = i / half, j = i % half;
    const float x1 = row[hh * hd + j], x2 = row[hh * hd + j + half], co = c[2 * j], si = c[2 * j + 1];
    qrot[(size_t)m * Hq * hd + hh * hd + j] = (x1 * co - x2 * si) * scale;
    qrot[(size_t)m * Hq * hd + hh * hd + j + half] = (x2 * co + x1 * si) * scale;
  }
  if (pos < 0 || pos >= cap) {  // never write outside the stream's slice of the cache
    if (tid == 0) atomicOr(status, SSD_STATUS_KV_OVERFLOW);
    return;
  }
  const float* krow = row + Hq * hd;
  const float* vrow = krow + Hkv * hd;
  // where this row's K and V live: the stream's slice of a contiguous cache, or its page
  size_t owner = (size_t)b, rows_per = (size_t)cap, slot = (size_t)pos;
  if (page_table) {
    const int pg = page_table[(size_t)b * max_pages + pos / TC_PAGE_TOKENS];
    if (pg < 0) {  // no page was granted (pool exhausted): flagged by the page kernel
      return;
    }
    owner = (size_t)pg;
    rows_per = TC_PAGE_TOKENS;
    slot = (size_t)(pos % TC_PAGE_TOKENS);
  }
  for (int i = tid; i < Hkv * half; i += 256) {
    const int g = i / half, j = i % half;
    const float x1 = krow[g * hd + j], x2 = krow[g * hd + j + half], co = c[2 * j], si = c[2 * j + 1];
    bf16* kdst = kv_layer + ((owner * 2 + 0) * Hkv + g) * rows_per * hd + slot * hd;
    kdst[j] = __float2bfloat16_rn(x1 * co - x2 * si);
    kdst[j + half] = __float2bfloat16_rn(x2 * co + x1 * si);
  }
  for (int i = tid; i < Hkv * hd; i += 256) {
    const int g = i / hd, j = i % hd;
    bf16* vdst = kv_layer + ((owner * 2 + 1) * Hkv + g) * rows_per * hd + slot * hd;
    vdst[j] = __float2bfloat16_rn(vrow[g * hd + j]);
  }
}

}  // namespace

void launch_tc_norm_pack(float* h, const float* part, int nsplit, int ld_part, int M, int d,
                         const bf16* gain, float eps, uint8_t* apack, cudaStream_t st) {
  if (M <= TC_ROWS_DEEP)
    tc_launch_pdl(tc_norm_pack_kernel<24, 1>, dim3(M), dim3(256), (size_t)d * 4, st, h, part, part ? nsplit : 0,
                  ld_part, tc_round16(M), tc_chunks(M).rows, d, gain, eps, apack);
  else
    tc_launch_pdl(tc_norm_pack_kernel<8, 4>, dim3(M), dim3(256), (size_t)d * 4, st, h, part, part ? nsplit : 0,
                  ld_part, tc_round16(M), tc_chunks(M).rows, d, gain, eps, apack);
  count_launch();
}

void launch_tc_pack_rows(const float* x, int M, int K, uint8_t* apack, cudaStream_t st) {
  tc_pack_rows_kernel<<<M, 128, 0, st>>>(x, K, tc_chunks(M).rows, apack);
  count_launch();
}

void launch_tc_qkv_post(const float* part, int nsplit, int ld_part, int Mpad, const bf16* bias,
                        const float* cs, float* qrot, bf16* kv_layer, const int32_t* len, RowMap rm,
                        int cap, int Hq, int Hkv, int hd, const int32_t* page_table, int max_pages,
                        int32_t* status, cudaStream_t st) {
  const int M = rm.nb * rm.R;
  const size_t smem = (size_t)(Hq + 2 * Hkv) * hd * 4;
  if (M <= TC_ROWS_DEEP)
    tc_launch_pdl(tc_qkv_post_kernel<24, 1>, dim3(M), dim3(256), smem, st, part, nsplit, ld_part, Mpad, bias, cs, qrot,
                  kv_layer, len, rm, cap, Hq, Hkv, hd, 1.0f / sqrtf((float)hd), page_table, max_pages, status);
  else
    tc_launch_pdl(tc_qkv_post_kernel<8, 4>, dim3(M), dim3(256), smem, st, part, nsplit, ld_part, Mpad, bias, cs, qrot,
                  kv_layer, len, rm, cap, Hq, Hkv, hd, 1.0f / sqrtf((float)hd), page_table, max_pages, status);
  count_launch();
}

namespace {

__global__ void page_ensure_kernel(const int32_t* __restrict__ len, RowMap rm, int32_t* page_table,
                                   int32_t* pages_used, const int32_t* __restrict__ free_stack, int32_t* free_top,
                                   int max_pages, int32_t* status) {
  const int bi = blockIdx.x * blockDim.x + threadIdx.x;
  if (bi >= rm.nb) return;
  const int b = rm.b0 + bi;
  int need = (len[b] + rm.R + TC_PAGE_TOKENS - 1) / TC_PAGE_TOKENS;
  if (need > max_pages) {  // rows beyond the block table are not written (flagged as an overflow)
    atomicOr(status, SSD_STATUS_KV_OVERFLOW);
    need = max_pages;
  }
  int used = pages_used[b];
  while (used < need) {
    const int idx = atomicSub(free_top, 1) - 1;  // pops from different streams race only on this counter
    if (idx < 0) {
      atomicAdd(free_top, 1);
      atomicOr(status, SSD_STATUS_KV_OVERFLOW);  // the pool is exhausted: the rows of this page are dropped
      break;
    }
    page_table[(size_t)b * max_pages + used] = free_stack[idx];
    ++used;
  }
  pages_used[b] = used;
}

__global__ void page_release_kernel(const int32_t* __restrict__ len, int B, int32_t* page_table, int32_t* pages_used,
                                    int32_t* free_stack, int32_t* free_top, int max_pages) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int keep = (max(len[b], 0) + TC_PAGE_TOKENS - 1) / TC_PAGE_TOKENS;
  int used = pages_used[b];
  while (used > keep) {
    --used;
    const int idx = atomicAdd(free_top, 1);
    free_stack[idx] = page_table[(size_t)b * max_pages + used];
    page_table[(size_t)b * max_pages + used] = -1;
  }
  pages_used[b] = used;
}

}  // namespace

void launch_page_ensure(const int32_t* len, RowMap rm, int32_t* page_table, int32_t* pages_used,
                        int32_t* free_stack, int32_t* free_top, int max_pages, int32_t* status,
                        cudaStream_t st) {
  page_ensure_kernel<<<(rm.nb + 127) / 128, 128, 0, st>>>(len, rm, page_table, pages_used, free_stack, free_top,
                                                         max_pages, status);
  count_launch();
}

void launch_page_release(const int32_t* len, int B, int32_t* page_table, int32_t* pages_used,
                         int32_t* free_stack, int32_t* free_top, int max_pages, cudaStream_t st) {
  page_release_kernel<<<(B + 127) / 128, 128, 0, st>>>(len, B, page_table, pages_used, free_stack, free_top,
                                                      max_pages);
  count_launch();
}

}  // namespace ssd
