// Batched verify attention (Eq. 4: the gamma + 1 new rows of every stream attend to the stream's
// cached prefix and, causally, to each other; grouped-query) on the warp-level tensor-core
// instruction, for forwards of more than 16 rows.
//
// Grid (key split, kv head x row group, stream).  The G * R query rows that share a kv head (G
// query heads per kv head, R rows per stream) are cut into groups of 64: one CTA of four warps,
// 16 rows per warp, so the keys and values of the head are read once for all of them.  A CTA
// walks its key range in tiles of 64 keys: K and V (bf16, as cached) arrive in shared memory by
// 16-byte async copies into padded rows, double buffered; per tile a warp computes
// S = q K^T with q as a two-term bf16 split (leading part + remainder, so the scores are exact to
// ~2^-17), masks (row r of a stream sees keys 0 .. len + r), updates the running max / sum of
// its rows in registers and accumulates O += P V with P taken straight from the score registers
// (split the same way) and V through transposing matrix loads.  The un-normalised partial
// (O, max, sum) of each (row, head, split) goes to global memory; a second kernel merges the
// splits of a row by their log-sum-exp weights, in a fixed order, and writes the result as the
// packed tensor-core operand of the O projection (tc.h).
#include <math_constants.h>

#include "kernels.h"
#include "tc.h"

namespace ssd {

namespace {

constexpr int TA_WARPS = 4;
// The softmax weights P enter the second contraction as bf16 leading part + remainder.  Rounding
// them to bf16 instead (one instruction fewer in four) was measured: the logits of the 24- and
// 28-layer models then differ from the float64 oracle by 2.0e-2 and 1.4e-2, against 1e-4 with the
// split - too close to the 3e-2 bound to be the default.
constexpr bool TA_SPLIT_P = true;
constexpr int TA_TILE = 64;  // keys per tile
static_assert(TA_TILE == TC_PAGE_TOKENS, "a key tile of the batched attention is one page of a paged cache");

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void split2(float x, float y, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  const __nv_bfloat162 l = __floats2bfloat162_rn(x - __low2float(h), y - __high2float(h));
  hi = *reinterpret_cast<const uint32_t*>(&h);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}

template <int HD>
__global__ void __launch_bounds__(TA_WARPS * 32)
tc_attn_kernel(const float* __restrict__ qrot, const bf16* __restrict__ kv_layer, const int32_t* __restrict__ len,
               RowMap rm, int cap, int Hq, int Hkv, int n_rowgroups, float* __restrict__ part, int nsplit,
               int keys_per_split, const int32_t* __restrict__ page_table, int max_pages) {
  constexpr int ROWB = HD * 2 + 16;   // padded K / V row: conflict-free matrix loads
  constexpr int KSTEPS = HD / 16;
  constexpr int DT = HD / 8;
  constexpr int CH = HD / 8;          // 16-byte chunks per row
  constexpr int TILE_BYTES = TA_TILE * ROWB;
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* kv_s = smem;                                   // [2 stages][K tile | V tile]
  uint4* q_s = reinterpret_cast<uint4*>(smem + 4 * TILE_BYTES);  // [warp][kstep][lane][hi 4 words | lo 4 words]

  const int sp = blockIdx.x, gk = blockIdx.y / n_rowgroups, rg = blockIdx.y % n_rowgroups, bi = blockIdx.z;
  const int b = rm.b0 + bi, R = rm.R, G = Hq / Hkv, NQ = G * R;
  tc_pdl_trigger();
  tc_pdl_wait();
  const int L = len[b], total = min(L + R, cap);
  const int k_begin = sp * keys_per_split;
  if (k_begin >= total) return;
  const int k_end = min(k_begin + keys_per_split, total);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const bf16* kbase = kv_layer + (((size_t)b * 2 + 0) * Hkv + gk) * (size_t)cap * HD;
  const bf16* vbase = kv_layer + (((size_t)b * 2 + 1) * Hkv + gk) * (size_t)cap * HD;

  auto stage_tile = [&](int stage, int key0) {
    uint8_t* ks = kv_s + (size_t)stage * 2 * TILE_BYTES;
    const bf16 *kt = kbase, *vt = vbase;
    int first = 0;  // key index of the tile's base pointers
    if (page_table) {
      // a tile is one page: key splits start at multiples of the page size, which is the tile size
      const int pg = max(page_table[(size_t)b * max_pages + key0 / TC_PAGE_TOKENS], 0);
      kt = kv_layer + (((size_t)pg * 2 + 0) * Hkv + gk) * (size_t)TC_PAGE_TOKENS * HD;
      vt = kv_layer + (((size_t)pg * 2 + 1) * Hkv + gk) * (size_t)TC_PAGE_TOKENS * HD;
      first = key0;
    }
    for (int i = tid; i < TA_TILE * CH; i += TA_WARPS * 32) {
      const int key = i / CH, c = i % CH;
      // keys past the range repeat the last valid one: finite data, masked out below
      const size_t src = (size_t)(min(key0 + key, k_end - 1) - first) * HD + c * 8;
      cp_async16(smem_u32(ks + key * ROWB + c * 16), kt + src);
      cp_async16(smem_u32(ks + TILE_BYTES + key * ROWB + c * 16), vt + src);
    }
    cp_async_commit();
  };
  stage_tile(0, k_begin);

  // this warp's 16 rows: row i = hl * R + r of the kv head's G * R rows
  const int i0 = rg * (TA_WARPS * 16) + warp * 16 + g, i1 = i0 + 8;
  const bool warp_active = rg * (TA_WARPS * 16) + warp * 16 < NQ;
  const bool ok0 = i0 < NQ, ok1 = i1 < NQ;
  const int r0 = ok0 ? i0 % R : 0, r1 = ok1 ? i1 % R : 0;
  const int h0 = gk * G + (ok0 ? i0 / R : 0), h1 = gk * G + (ok1 ? i1 / R : 0);
  const int m0 = bi * R + r0, m1 = bi * R + r1;
  {  // q as A fragments (bf16 leading part + remainder), each lane its own
    const float* q0 = qrot + ((size_t)m0 * Hq + h0) * HD;
    const float* q1 = qrot + ((size_t)m1 * Hq + h1) * HD;
#pragma unroll
    for (int s = 0; s < KSTEPS; ++s) {
      float2 a0 = make_float2(0.f, 0.f), a1 = a0, a2 = a0, a3 = a0;
      if (ok0) {
        a0 = *reinterpret_cast<const float2*>(q0 + s * 16 + 2 * t);
        a2 = *reinterpret_cast<const float2*>(q0 + s * 16 + 8 + 2 * t);
      }
      if (ok1) {
        a1 = *reinterpret_cast<const float2*>(q1 + s * 16 + 2 * t);
        a3 = *reinterpret_cast<const float2*>(q1 + s * 16 + 8 + 2 * t);
      }
      uint4 hi, lo;
      split2(a0.x, a0.y, hi.x, lo.x);
      split2(a1.x, a1.y, hi.y, lo.y);
      split2(a2.x, a2.y, hi.z, lo.z);
      split2(a3.x, a3.y, hi.w, lo.w);
      uint4* dst = q_s + ((size_t)(warp * KSTEPS + s) * 32 + lane) * 2;
      dst[0] = hi;
      dst[1] = lo;
    }
  }
  __syncwarp();

  float m_run[2] = {-CUDART_INF_F, -CUDART_INF_F}, l_run[2] = {0.f, 0.f};
  float o[DT][4];
#pragma unroll
  for (int dt = 0; dt < DT; ++dt) o[dt][0] = o[dt][1] = o[dt][2] = o[dt][3] = 0.f;
  const int lim0 = L + r0, lim1 = L + r1;  // last visible key of the two rows

  const int n_tiles = (k_end - k_begin + TA_TILE - 1) / TA_TILE;
  for (int it = 0; it < n_tiles; ++it) {
    const int key0 = k_begin + it * TA_TILE;
    // One barrier per tile: it makes this tile's copies (all threads') visible, and it says that
    // every warp is done with the previous tile, whose buffer the next tile's copies may now
    // overwrite while this one is being used.
    cp_async_wait<0>();
    __syncthreads();
    if (it + 1 < n_tiles) stage_tile((it + 1) & 1, key0 + TA_TILE);
    if (warp_active) {
      const uint8_t* ks = kv_s + (size_t)(it & 1) * 2 * TILE_BYTES;
      const uint32_t k_addr = smem_u32(ks) + ((lane >> 4) * 8 + (lane & 7)) * ROWB + ((lane >> 3) & 1) * 16;
      const uint32_t v_addr = smem_u32(ks + TILE_BYTES) + (((lane >> 3) & 1) * 8 + (lane & 7)) * ROWB + (lane >> 4) * 16;
      float sc[TA_TILE / 8][4];
#pragma unroll
      for (int nt = 0; nt < TA_TILE / 8; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
      for (int s = 0; s < KSTEPS; ++s) {
        const uint4* qa = q_s + ((size_t)(warp * KSTEPS + s) * 32 + lane) * 2;
        const uint4 hi = qa[0], lo = qa[1];
        const uint32_t ahi[4] = {hi.x, hi.y, hi.z, hi.w}, alo[4] = {lo.x, lo.y, lo.z, lo.w};
#pragma unroll
        for (int nt = 0; nt < TA_TILE / 8; nt += 2) {
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4(k_addr + nt * 8 * ROWB + s * 32, b0, b1, b2, b3);
          mma_bf16(sc[nt], ahi, b0, b1);  // alternate the accumulators: no instruction waits for the one before
          mma_bf16(sc[nt + 1], ahi, b2, b3);
          mma_bf16(sc[nt], alo, b0, b1);
          mma_bf16(sc[nt + 1], alo, b2, b3);
        }
      }
      // mask, running max and sum (the sum stays per thread until the end).  Only the last
      // tile of a row's keys needs the mask: a tile that every row of the warp sees whole skips
      // it (rows that do not exist hold zeros; their results are never written).
      const int last_key = key0 + TA_TILE - 1;
      const bool whole = __all_sync(0xffffffffu, last_key < k_end && (!ok0 || last_key <= lim0) &&
                                                     (!ok1 || last_key <= lim1));
      float mt[2] = {-CUDART_INF_F, -CUDART_INF_F};
      if (!whole) {
#pragma unroll
        for (int nt = 0; nt < TA_TILE / 8; ++nt) {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int key = key0 + nt * 8 + 2 * t + e;
            if (!(ok0 && key < k_end && key <= lim0)) sc[nt][e] = -CUDART_INF_F;
            if (!(ok1 && key < k_end && key <= lim1)) sc[nt][2 + e] = -CUDART_INF_F;
          }
        }
      }
#pragma unroll
      for (int nt = 0; nt < TA_TILE / 8; ++nt) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          mt[0] = fmaxf(mt[0], sc[nt][e]);
          mt[1] = fmaxf(mt[1], sc[nt][2 + e]);
        }
      }
      float corr[2], mn[2];
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        mt[hh] = fmaxf(mt[hh], __shfl_xor_sync(0xffffffffu, mt[hh], 1));
        mt[hh] = fmaxf(mt[hh], __shfl_xor_sync(0xffffffffu, mt[hh], 2));
        mn[hh] = fmaxf(m_run[hh], mt[hh]);
        corr[hh] = mn[hh] == -CUDART_INF_F ? 1.f : __expf(m_run[hh] - mn[hh]);
        m_run[hh] = mn[hh];
        l_run[hh] *= corr[hh];
      }
#pragma unroll
      for (int dt = 0; dt < DT; ++dt) {
        o[dt][0] *= corr[0];
        o[dt][1] *= corr[0];
        o[dt][2] *= corr[1];
        o[dt][3] *= corr[1];
      }
      if (whole) {
#pragma unroll
        for (int nt = 0; nt < TA_TILE / 8; ++nt) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float p = __expf(sc[nt][e] - mn[e >> 1]);
            sc[nt][e] = p;
            l_run[e >> 1] += p;
          }
        }
      } else {
#pragma unroll
        for (int nt = 0; nt < TA_TILE / 8; ++nt) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float mm = mn[e >> 1];
            const float p = sc[nt][e] == -CUDART_INF_F ? 0.f : __expf(sc[nt][e] - mm);
            sc[nt][e] = p;
            l_run[e >> 1] += p;
          }
        }
      }
#pragma unroll
      for (int kk = 0; kk < TA_TILE / 16; ++kk) {
        uint32_t phi[4], plo[4];
        split2(sc[2 * kk][0], sc[2 * kk][1], phi[0], plo[0]);
        split2(sc[2 * kk][2], sc[2 * kk][3], phi[1], plo[1]);
        split2(sc[2 * kk + 1][0], sc[2 * kk + 1][1], phi[2], plo[2]);
        split2(sc[2 * kk + 1][2], sc[2 * kk + 1][3], phi[3], plo[3]);
#pragma unroll
        for (int dt = 0; dt < DT; dt += 2) {
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4_trans(v_addr + kk * 16 * ROWB + dt * 16, b0, b1, b2, b3);
          mma_bf16(o[dt], phi, b0, b1);
          mma_bf16(o[dt + 1], phi, b2, b3);
          if (TA_SPLIT_P) mma_bf16(o[dt], plo, b0, b1);
          if (TA_SPLIT_P) mma_bf16(o[dt + 1], plo, b2, b3);
        }
      }
    }
  }
  if (!warp_active) return;
#pragma unroll
  for (int hh = 0; hh < 2; ++hh) {
    l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 1);
    l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 2);
  }
  if (ok0) {
    float* dst = part + (((size_t)m0 * Hq + h0) * nsplit + sp) * (HD + 2);
#pragma unroll
    for (int dt = 0; dt < DT; ++dt) *reinterpret_cast<float2*>(dst + dt * 8 + 2 * t) = make_float2(o[dt][0], o[dt][1]);
    if (t == 0) {
      dst[HD] = m_run[0];
      dst[HD + 1] = l_run[0];
    }
  }
  if (ok1) {
    float* dst = part + (((size_t)m1 * Hq + h1) * nsplit + sp) * (HD + 2);
#pragma unroll
    for (int dt = 0; dt < DT; ++dt) *reinterpret_cast<float2*>(dst + dt * 8 + 2 * t) = make_float2(o[dt][2], o[dt][3]);
    if (t == 0) {
      dst[HD] = m_run[1];
      dst[HD + 1] = l_run[1];
    }
  }
}

// Grid (query head, row).  Merges the key splits of one (row, head) and writes the normalised
// output as columns h * HD .. of the packed operand.
template <int HD>
__global__ void tc_attn_merge_kernel(const float* __restrict__ part, const int32_t* __restrict__ len, RowMap rm,
                                     int cap, int Hq, int nsplit, int keys_per_split,
                                     uint8_t* __restrict__ apack, int Mc) {
  const int h = blockIdx.x, m = blockIdx.y;
  const int bi = m / rm.R, b = rm.b0 + bi;
  tc_pdl_trigger();
  tc_pdl_wait();
  const int total = min(len[b] + rm.R, cap);
  const int ns = (total + keys_per_split - 1) / keys_per_split;
  const float* src = part + ((size_t)m * Hq + h) * nsplit * (HD + 2);
  __shared__ float s_m[128], s_w[128];  // running max and sum of each split, then its weight
  for (int s = threadIdx.x; s < ns; s += blockDim.x) {
    s_m[s] = __ldcg(src + s * (HD + 2) + HD);
    s_w[s] = __ldcg(src + s * (HD + 2) + HD + 1);
  }
  __syncthreads();
  float m_tot = -CUDART_INF_F;
  for (int s = 0; s < ns; ++s) m_tot = fmaxf(m_tot, s_m[s]);
  float denom = 0.f;
  for (int s = 0; s < ns; ++s) {  // fixed order
    const float e = s_m[s] == -CUDART_INF_F ? 0.f : __expf(s_m[s] - m_tot);
    denom = fmaf(e, s_w[s], denom);
  }
  __syncthreads();
  for (int s = threadIdx.x; s < ns; s += blockDim.x) s_w[s] = s_m[s] == -CUDART_INF_F ? 0.f : __expf(s_m[s] - m_tot);
  __syncthreads();
  const float inv = 1.f / denom;
  uint8_t* arow = apack + tc_act_row_off(Mc, (Hq * HD + 15) >> 4, m);
  for (int d = threadIdx.x * 2; d < HD; d += blockDim.x * 2) {
    float o0 = 0.f, o1 = 0.f;
#pragma unroll 4
    for (int s = 0; s < ns; ++s) {  // fixed order
      const float2 v = __ldcg(reinterpret_cast<const float2*>(src + s * (HD + 2) + d));
      o0 = fmaf(s_w[s], v.x, o0);
      o1 = fmaf(s_w[s], v.y, o1);
    }
    o0 *= inv;
    o1 *= inv;
    const int k = h * HD + d;
    const __nv_bfloat162 hi = __floats2bfloat162_rn(o0, o1);
    const __nv_bfloat162 lo = __floats2bfloat162_rn(o0 - __low2float(hi), o1 - __high2float(hi));
    uint8_t* e = arow + tc_act_col_off(Mc, k);
    *reinterpret_cast<__nv_bfloat162*>(e) = hi;
    *reinterpret_cast<__nv_bfloat162*>(e + (size_t)Mc * 16) = lo;
  }
}

template <int HD>
cudaError_t launch_t(const float* qrot, const bf16* kv_layer, const int32_t* len, RowMap rm, int cap, int Hq,
                     int Hkv, float* part, int nsplit, int keys_per_split, uint8_t* apack_out, int Mpad,
                     const int32_t* page_table, int max_pages, int which_kernel, int32_t* status, cudaStream_t st) {
  const int NQ = (Hq / Hkv) * rm.R, n_rowgroups = (NQ + TA_WARPS * 16 - 1) / (TA_WARPS * 16);
  const size_t smem = (size_t)4 * TA_TILE * (HD * 2 + 16) + (size_t)TA_WARPS * (HD / 16) * 32 * 32;
  cudaError_t e;
  const bool t5 = HD >= 64 && (which_kernel == 2 || (which_kernel == 0 && keys_per_split >= TC_ATTN5_MIN_KEYS));
  if (t5) {  // tcgen05 contractions
    e = launch_tc_attention5(qrot, kv_layer, len, rm, cap, Hq, Hkv, HD, part, nsplit, keys_per_split, page_table,
                             max_pages, status, st);
    if (e != cudaSuccess) return e;
  } else {
    auto kern = tc_attn_kernel<HD>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = tc_launch_pdl(kern, dim3(nsplit, Hkv * n_rowgroups, rm.nb), dim3(TA_WARPS * 32), smem, st, qrot, kv_layer, len,
                      rm, cap, Hq, Hkv, n_rowgroups, part, nsplit, keys_per_split, page_table, max_pages);
    if (e != cudaSuccess) return e;
    count_launch();
  }
  e = tc_launch_pdl(tc_attn_merge_kernel<HD>, dim3(Hq, rm.nb * rm.R), dim3(HD / 2 < 32 ? 32 : HD / 2), 0, st,
                    (const float*)part, len, rm, cap, Hq, nsplit, keys_per_split, apack_out,
                    tc_chunks(rm.nb * rm.R).rows);
  if (e != cudaSuccess) return e;
  count_launch();
  return cudaGetLastError();
}

}  // namespace

int tc_attention_ctas_per_sm(int) { return 2; }

cudaError_t launch_tc_attention(const float* qrot, const bf16* kv_layer, const int32_t* len, RowMap rm,
                                int cap, int Hq, int Hkv, int hd, float* part, int nsplit,
                                int keys_per_split, uint8_t* apack_out, int Mpad,
                                const int32_t* page_table, int max_pages, int which_kernel, int32_t* status,
                                cudaStream_t st) {
  if (page_table && keys_per_split % TC_PAGE_TOKENS) return cudaErrorInvalidValue;
  switch (hd) {
    case 32: return launch_t<32>(qrot, kv_layer, len, rm, cap, Hq, Hkv, part, nsplit, keys_per_split, apack_out, Mpad, page_table, max_pages, which_kernel, status, st);
    case 64: return launch_t<64>(qrot, kv_layer, len, rm, cap, Hq, Hkv, part, nsplit, keys_per_split, apack_out, Mpad, page_table, max_pages, which_kernel, status, st);
    case 128: return launch_t<128>(qrot, kv_layer, len, rm, cap, Hq, Hkv, part, nsplit, keys_per_split, apack_out, Mpad, page_table, max_pages, which_kernel, status, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace ssd
