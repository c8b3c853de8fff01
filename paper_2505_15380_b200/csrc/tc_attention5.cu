// Batched verify attention (Eq. 4: the gamma + 1 new rows of every stream attend to the stream's
// cached prefix and, causally, to each other; grouped-query) on tcgen05 tensor cores, for head
// sizes 64 and 128 and forwards of more than 16 rows.
//
// Grid (key split, kv head x row group, stream), one CTA = up to 64 of the G * R query rows that
// share a kv head, over one range of keys, in tiles of 64 keys; two CTAs fit an SM, so that the
// row work of one overlaps the instructions of the other.  Both contractions are
// tcgen05.mma 128 x N x 16 with the accumulators in tensor memory:
//
//   S[row, key] = sum_d q[row, d] k[key, d]     A = q, rows 0..63 the bf16 leading parts, rows
//                                               64..127 the remainders of the same rows (one
//                                               instruction multiplies both; the two halves of S
//                                               are added by the row threads); B = the K tile
//   O[row, d]  += sum_key p[row, key] v[key, d] A = p, split and stacked the same way; B = the V
//                                               tile transposed (keys contiguous)
//
// Operands sit in shared memory in the canonical K-major layout without swizzle (tc.h): byte
// (k / 8) * rows * 16 + row * 16 + (k % 8) * 2.  A copy warp brings K by 16-byte async copies
// straight into that layout and V row by row; the row threads transpose V with transposing
// matrix loads.  Threads 0..127 own one tensor-memory lane each (lane r: leading parts of row r,
// lane r + 64: its remainders).  The two threads of a row split the tile's columns, pass each
// other the half of S they do not keep through shared memory (in the place of the raw V tile),
// apply mask, running max and sum, and write p as the next operand; when a running max grows,
// every thread rescales its lane of O in tensor memory.  Warp 4 issues the instructions: the O
// contraction of tile t and the S contraction of tile t + 1 alternately (instructions that
// follow one another into the same accumulator wait for each other, measured ~280 against ~165
// cycles); a first commit tells the row threads that O is up to date while S is still being
// computed, so that they transpose the next V tile meanwhile.
//
// The un-normalised partial (O, max, sum) of each (row, head, split) goes to global memory in the
// format of the warp-level kernel (tc_attention.cu), whose merge kernel finishes the job.
// Every wait is bounded; when one runs out the CTA raises SSD_STATUS_TIMEOUT, waits (bounded) for
// what it has in flight, frees its tensor memory and returns.
#include <math_constants.h>

#include "kernels.h"
#include "tc.h"

namespace ssd {

namespace {

constexpr int T5_TILE = 64;            // keys per tile: small enough for two CTAs per SM, whose phases then overlap
constexpr int T5_THREADS = 192;        // 4 row warps, the issuing warp, the copy warp
constexpr unsigned long long T5_WAIT_CYCLES = 2000000000ull;  // ~1 s

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort) {
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 15u) == 0u) {
      if (*abort) return false;
      if ((unsigned long long)(clock64() - t0) > T5_WAIT_CYCLES) {
        *abort = 1;
        return false;
      }
    }
  }
  return true;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort) {
  return mbar_try_wait(bar, parity) || mbar_wait_slow(bar, parity, abort);
}
// K-major operand without swizzle: start address, byte distance between core matrices along K
// (leading) and along the rows (stride), in units of 16 bytes; bit 46: descriptor format.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lead_bytes, uint32_t stride_bytes) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lead_bytes >> 4) << 16) |
         ((uint64_t)(stride_bytes >> 4) << 32) | (1ull << 46);
}
// kind::f16: fp32 accumulator, bf16 A and B, both K-major, M = 128.
__device__ __forceinline__ uint32_t umma_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void t5_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void t5_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
        "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
        "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
        "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
// Barrier among the 128 row threads only (the issuing warp does not take part).
__device__ __forceinline__ void row_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

struct T5Shared {
  unsigned long long mma_done;  // completes when the instructions of one issue round have finished
  unsigned long long o_done;    // completes earlier in the round: when its O += p V part has finished
  unsigned long long k_full, v_full;  // the copy warp's K / V tile has landed
  unsigned long long v_free;    // the row threads are done with the raw V tile and the exchange area
  uint32_t tmem_base;
  int abort;
  float mx[128];                // this tile's maximum over each row thread's half of the columns
};

template <int HD>
struct T5Lay {
  static constexpr int CH = HD / 8;                     // 16-byte chunks per K / V row
  static constexpr int Q_BYTES = CH * 2048;             // [d / 8][128 rows][16 B]
  static constexpr int K_BYTES = CH * T5_TILE * 16;     // [d / 8][keys of a tile][16 B]
  static constexpr int VROW = HD * 2 + 16;              // padded raw V row
  static constexpr int SX_STRIDE = T5_TILE + 4;         // floats per row of the exchange area
  static constexpr int VRAW_BYTES = (T5_TILE * VROW > 64 * SX_STRIDE * 4) ? T5_TILE * VROW : 64 * SX_STRIDE * 4;
  static constexpr int VT_BYTES = (T5_TILE / 8) * HD * 16;  // [key / 8][HD rows][16 B]
  static constexpr int P_BYTES = (T5_TILE / 8) * 2048;      // [key / 8][128 rows][16 B]
  static constexpr int OFF_Q = 0, OFF_K = OFF_Q + Q_BYTES, OFF_VRAW = OFF_K + K_BYTES,
                       OFF_VT = OFF_VRAW + VRAW_BYTES, OFF_P = OFF_VT + VT_BYTES, OFF_S = OFF_P + P_BYTES;
  static constexpr int TOTAL = OFF_S + (int)sizeof(T5Shared) + 64;
  static constexpr int TMEM_COLS = HD + T5_TILE <= 128 ? 128 : (HD + T5_TILE <= 256 ? 256 : 512);
  static constexpr int OX_STRIDE = HD + 4;              // floats per row of the final exchange (over the dead V / p areas)
  static_assert(64 * OX_STRIDE * 4 <= VRAW_BYTES + VT_BYTES + P_BYTES, "final exchange area");
};

// exp(x) for a row's scores; four partial sums keep the additions independent.
struct T5Sum {
  float a, b, c, d;
};

template <int HD>
__global__ void __launch_bounds__(T5_THREADS, 2)
tc_attn5_kernel(const float* __restrict__ qrot, const bf16* __restrict__ kv_layer, const int32_t* __restrict__ len,
                RowMap rm, int cap, int Hq, int Hkv, int n_rowgroups, float* __restrict__ part, int nsplit,
                int keys_per_split, const int32_t* __restrict__ page_table, int max_pages, int32_t* status) {
  using Lay = T5Lay<HD>;
  constexpr int CH = Lay::CH;
  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* Qs = smem + Lay::OFF_Q;
  uint8_t* Ks = smem + Lay::OFF_K;
  uint8_t* Vraw = smem + Lay::OFF_VRAW;
  float* Sx = reinterpret_cast<float*>(Vraw);  // the raw V tile is dead while the scores are exchanged
  uint8_t* Vt = smem + Lay::OFF_VT;
  uint8_t* Ps = smem + Lay::OFF_P;
  T5Shared& S = *reinterpret_cast<T5Shared*>(smem + Lay::OFF_S);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sp = blockIdx.x, gk = blockIdx.y / n_rowgroups, rg = blockIdx.y % n_rowgroups, bi = blockIdx.z;
  const int b = rm.b0 + bi, R = rm.R, G = Hq / Hkv, NQ = G * R;
  tc_pdl_trigger();
  tc_pdl_wait();
  const int L = len[b], total = min(L + R, cap);
  const int k_begin = sp * keys_per_split;
  if (k_begin >= total) return;  // uniform: nothing has been set up yet
  const int k_end = min(k_begin + keys_per_split, total);
  const int n_tiles = (k_end - k_begin + T5_TILE - 1) / T5_TILE;

  if (tid == 0) {
    mbar_init(smem_u32(&S.mma_done), 1);
    mbar_init(smem_u32(&S.o_done), 1);
    mbar_init(smem_u32(&S.k_full), 32);
    mbar_init(smem_u32(&S.v_full), 32);
    mbar_init(smem_u32(&S.v_free), 1);
    S.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&S.tmem_base)), "r"((uint32_t)Lay::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  t5_fence_before();
  __syncthreads();
  t5_fence_after();
  const uint32_t tmem = S.tmem_base;
  const uint32_t t_s = tmem, t_o = tmem + T5_TILE;  // columns of S and of O
  volatile int* abort = &S.abort;
  const uint32_t bar = smem_u32(&S.mma_done), bar_o = smem_u32(&S.o_done), bar_k = smem_u32(&S.k_full), bar_v = smem_u32(&S.v_full),
                 bar_vf = smem_u32(&S.v_free);

  // ---- row threads' view: threads r and r + 64 (r < 64) share query row i = rg * 64 + r.  Lane r
  // of tensor memory holds the leading parts' products, lane r + 64 the remainders'; thread r
  // takes columns 0..63 of a tile, thread r + 64 columns 64..127.
  const int r_loc = tid & 63, i_row = rg * 64 + r_loc, half = (tid >> 6) & 1;
  const bool row_ok = i_row < NQ;
  const int rr = row_ok ? i_row % R : 0, hl = row_ok ? i_row / R : 0;
  const int h = gk * G + hl, m = bi * R + rr, lim = L + rr;  // head, row of the forward, last visible key

  float m_run = -CUDART_INF_F;
  T5Sum l_run = {0.f, 0.f, 0.f, 0.f};  // this thread's half of the row's sum

  if (warp == 5) {
    // ---- copy warp: K and V tiles by 16-byte async copies; lane = (key % 8, chunk % 4), so that
    // a warp instruction fills all banks and reads 64 contiguous bytes per key.  A barrier
    // completes when every lane's copies of the tile have landed.
    const bf16* kbase = kv_layer + (((size_t)b * 2 + 0) * Hkv + gk) * (size_t)cap * HD;
    const bf16* vbase = kv_layer + (((size_t)b * 2 + 1) * Hkv + gk) * (size_t)cap * HD;
    auto row_src = [&](int key_abs, int which) -> const bf16* {
      if (page_table) {
        const int pg = max(page_table[(size_t)b * max_pages + key_abs / TC_PAGE_TOKENS], 0);
        return kv_layer + (((size_t)pg * 2 + which) * Hkv + gk) * (size_t)TC_PAGE_TOKENS * HD +
               (size_t)(key_abs % TC_PAGE_TOKENS) * HD;
      }
      return (which ? vbase : kbase) + (size_t)key_abs * HD;
    };
    auto load = [&](int t, int which) {
      const int key0 = k_begin + t * T5_TILE;
      for (int kg = 0; kg < T5_TILE / 8; ++kg) {
        const int key = kg * 8 + (lane & 7);
        const bf16* src = row_src(min(key0 + key, k_end - 1), which);  // past the range: a valid key (masked later)
        if (which == 0) {
#pragma unroll
          for (int c = lane >> 3; c < CH; c += 4) cp_async16(smem_u32(Ks + c * (T5_TILE * 16) + key * 16), src + c * 8);
        } else {
#pragma unroll
          for (int c = lane >> 3; c < CH; c += 4) cp_async16(smem_u32(Vraw + key * Lay::VROW + c * 16), src + c * 8);
        }
      }
      asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(which ? bar_v : bar_k) : "memory");
    };
    load(0, 0);
    load(0, 1);
    t5_fence_before();
    __syncthreads();  // (the barrier the other warps take after their set-up)
    for (int t = 0; t < n_tiles; ++t) {
      // K(t + 1) goes where K(t) was: S(t) must be complete (round t)
      if (!mbar_wait(bar, (uint32_t)t & 1u, abort)) break;
      if (t + 1 < n_tiles) load(t + 1, 0);
      // V(t + 1) goes into the raw area: the row threads must be done with it (transposition and exchange of tile t)
      if (!mbar_wait(bar_vf, (uint32_t)t & 1u, abort)) break;
      if (t + 1 < n_tiles) load(t + 1, 1);
    }
    cp_async_wait<0>();  // never leave with copies in flight
  } else if (warp < 4) {
    // q as the A operand: row r (leading parts) and row 64 + r (remainders); rows that do not exist are zero
    for (int idx = tid; idx < 64 * CH; idx += 128) {
      const int r = idx / CH, c = idx % CH, i = rg * 64 + r;
      uint4 hi = make_uint4(0u, 0u, 0u, 0u), lo = hi;
      if (i < NQ) {
        const float* q = qrot + ((size_t)(bi * R + i % R) * Hq + gk * G + i / R) * HD + c * 8;
        const float4 a = *reinterpret_cast<const float4*>(q), bq = *reinterpret_cast<const float4*>(q + 4);
        const float x[8] = {a.x, a.y, a.z, a.w, bq.x, bq.y, bq.z, bq.w};
        uint32_t hw[4], lw[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const __nv_bfloat162 hh = __floats2bfloat162_rn(x[2 * j], x[2 * j + 1]);
          const __nv_bfloat162 ll = __floats2bfloat162_rn(x[2 * j] - __low2float(hh), x[2 * j + 1] - __high2float(hh));
          hw[j] = *reinterpret_cast<const uint32_t*>(&hh);
          lw[j] = *reinterpret_cast<const uint32_t*>(&ll);
        }
        hi = make_uint4(hw[0], hw[1], hw[2], hw[3]);
        lo = make_uint4(lw[0], lw[1], lw[2], lw[3]);
      }
      *reinterpret_cast<uint4*>(Qs + c * 2048 + r * 16) = hi;
      *reinterpret_cast<uint4*>(Qs + c * 2048 + (64 + r) * 16) = lo;
    }
    fence_async_smem();
  }
  if (warp != 5) {
    t5_fence_before();
    __syncthreads();
  }
  if (warp == 4 && lane == 0) {  // S(0) = q K(0)^T
    if (mbar_wait(bar_k, 0u, abort)) {
      fence_async_smem();
      t5_fence_after();
#pragma unroll
      for (int s = 0; s < HD / 16; ++s)
        umma_bf16(t_s, umma_desc(smem_u32(Qs) + s * 4096, 2048u, 128u),
                  umma_desc(smem_u32(Ks) + s * (2 * T5_TILE * 16), (uint32_t)T5_TILE * 16u, 128u), umma_idesc(T5_TILE),
                  s > 0 ? 1u : 0u);
    }
    umma_commit(bar);
  }

  if (warp != 5) {
    for (int t = 0; t < n_tiles; ++t) {
      const int key0 = k_begin + t * T5_TILE;
      if (warp < 4) {
        // O includes tile t - 1 (the first part of round t): the transposed V and p of that tile
        // may be overwritten.  The rest of the round, S(t), finishes while V(t) is transposed.
        if (t > 0 && !mbar_wait(bar_o, (uint32_t)(t - 1) & 1u, abort)) S.abort = 1;
        if (!mbar_wait(bar_v, (uint32_t)t & 1u, abort)) S.abort = 1;  // V(t) has landed
        // V(t): [key][d] -> [key / 8][d][key % 8] with transposing matrix loads: an 8 x 8 block
        // (8 keys x 8 d) comes back with thread T holding keys 2 (T % 4), + 1 of d = T / 4, one
        // word of the operand; the 32 words of a block go to 32 different banks.
        for (int task = warp; task < (T5_TILE / 8) * (CH / 4); task += 4) {
          const int kgrp = task % (T5_TILE / 8), c4 = task / (T5_TILE / 8);
          const uint32_t src = smem_u32(Vraw) + (uint32_t)((kgrp * 8 + (lane & 7)) * Lay::VROW + (c4 * 4 + (lane >> 3)) * 16);
          uint32_t w0, w1, w2, w3;
          asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                       : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3) : "r"(src));
          uint8_t* dst = Vt + (size_t)kgrp * (HD * 16) + (size_t)(c4 * 32 + (lane >> 2)) * 16 + (lane & 3) * 4;
          *reinterpret_cast<uint32_t*>(dst) = w0;
          *reinterpret_cast<uint32_t*>(dst + 8 * 16) = w1;
          *reinterpret_cast<uint32_t*>(dst + 16 * 16) = w2;
          *reinterpret_cast<uint32_t*>(dst + 24 * 16) = w3;
        }
        if (!mbar_wait(bar, (uint32_t)t & 1u, abort)) S.abort = 1;  // round t has finished: S(t) is complete
        t5_fence_after();
        row_sync();  // the raw tile is dead: its place becomes the exchange area
        // Every thread reads its lane's columns of S: the half it keeps stays in registers, the
        // other half goes to the partner (thread r gives the upper columns, thread r + 64 the lower).
        constexpr int HC = T5_TILE / 2;  // columns per thread
        static_assert(HC == 32, "one 32-column tensor-memory load per half");
        float sv[HC];
        {
          const uint32_t lane_addr = t_s + ((uint32_t)(warp * 32) << 16);
          uint32_t v[32];
          tmem_ld32(lane_addr + (uint32_t)((1 - half) * HC), v);
          float4* dst = reinterpret_cast<float4*>(Sx + (size_t)r_loc * Lay::SX_STRIDE + (1 - half) * HC);
#pragma unroll
          for (int j = 0; j < 8; ++j)
            dst[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                                 __uint_as_float(v[4 * j + 3]));
          tmem_ld32(lane_addr + (uint32_t)(half * HC), v);
#pragma unroll
          for (int j = 0; j < 32; ++j) sv[j] = __uint_as_float(v[j]);
        }
        row_sync();
        // scores of this thread's columns, mask, maximum
        const int last_vis = min(k_end - 1, lim) - key0 - half * HC;  // last visible one of this thread's columns
        float mt = -CUDART_INF_F;
        {
          const float4* other = reinterpret_cast<const float4*>(Sx + (size_t)r_loc * Lay::SX_STRIDE + half * HC);
          float m4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
          for (int j = 0; j < HC / 4; ++j) {
            const float4 x = other[j];
            sv[4 * j] += x.x;
            sv[4 * j + 1] += x.y;
            sv[4 * j + 2] += x.z;
            sv[4 * j + 3] += x.w;
          }
          if (last_vis >= HC - 1) {
#pragma unroll
            for (int j = 0; j < HC; ++j) m4[j & 3] = fmaxf(m4[j & 3], sv[j]);
          } else {
#pragma unroll
            for (int j = 0; j < HC; ++j) {
              if (j > last_vis) sv[j] = -CUDART_INF_F;
              m4[j & 3] = fmaxf(m4[j & 3], sv[j]);
            }
          }
          mt = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
          if (!row_ok) mt = -CUDART_INF_F;
        }
        S.mx[tid] = mt;
        row_sync();  // both halves' maxima are known; the exchange area is free again
        if (tid == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_vf) : "memory");
        const float mn = fmaxf(m_run, fmaxf(S.mx[r_loc], S.mx[r_loc + 64]));
        const float corr = (m_run == -CUDART_INF_F || m_run == mn) ? 1.f : __expf(m_run - mn);
        m_run = mn;
        l_run.a *= corr;
        l_run.b *= corr;
        l_run.c *= corr;
        l_run.d *= corr;
        // p = exp(s - max) (0 where masked: exp(-inf)), its sum, and both bf16 parts into the
        // operand rows r and 64 + r, columns of this thread
        const float sub = mn == -CUDART_INF_F ? 0.f : mn;  // a row that has seen nothing yet: all scores are -inf
#pragma unroll
        for (int j = 0; j < HC; ++j) sv[j] = row_ok ? __expf(sv[j] - sub) : 0.f;
#pragma unroll
        for (int g8 = 0; g8 < HC / 8; ++g8) {
          const float* p = sv + 8 * g8;
          l_run.a += p[0] + p[4];
          l_run.b += p[1] + p[5];
          l_run.c += p[2] + p[6];
          l_run.d += p[3] + p[7];
          uint32_t hw[4], lw[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const __nv_bfloat162 hh = __floats2bfloat162_rn(p[2 * j], p[2 * j + 1]);
            const __nv_bfloat162 ll = __floats2bfloat162_rn(p[2 * j] - __low2float(hh), p[2 * j + 1] - __high2float(hh));
            hw[j] = *reinterpret_cast<const uint32_t*>(&hh);
            lw[j] = *reinterpret_cast<const uint32_t*>(&ll);
          }
          uint8_t* dst = Ps + (size_t)(half * (HC / 8) + g8) * 2048 + r_loc * 16;
          *reinterpret_cast<uint4*>(dst) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
          *reinterpret_cast<uint4*>(dst + 64 * 16) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
        }
        // a grown maximum: rescale this thread's lane of O (both lanes of a row use the row's factor)
        if (t > 0 && __any_sync(0xffffffffu, corr != 1.f)) {
#pragma unroll
          for (int c0 = 0; c0 < HD; c0 += 32) {
            uint32_t v[32];
            tmem_ld32(t_o + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * corr);
            tmem_st32(t_o + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
          }
        }
        fence_async_smem();  // p and the transposed V were written by ordinary stores
      }
      t5_fence_before();
      asm volatile("bar.sync 2, 160;" ::: "memory");  // row warps and the issuing warp
      if (S.abort) break;  // uniform
      if (warp == 4 && lane == 0) {
        // O += p V(t) and S(t + 1) = q K(t + 1)^T, alternately
        const bool more = t + 1 < n_tiles;
        bool k_ok = true;
        if (more) {
          k_ok = mbar_wait(bar_k, (uint32_t)(t + 1) & 1u, abort);
          fence_async_smem();
        }
        t5_fence_after();
        constexpr int NPV = T5_TILE / 16, NQK = HD / 16;
#pragma unroll
        for (int s = 0; s < (NPV > NQK ? NPV : NQK); ++s) {
          if (s < NPV)
            umma_bf16(t_o, umma_desc(smem_u32(Ps) + s * 4096, 2048u, 128u),
                      umma_desc(smem_u32(Vt) + s * (2 * HD * 16), (uint32_t)HD * 16u, 128u), umma_idesc(HD),
                      (t > 0 || s > 0) ? 1u : 0u);
          if (more && k_ok && s < NQK)
            umma_bf16(t_s, umma_desc(smem_u32(Qs) + s * 4096, 2048u, 128u),
                      umma_desc(smem_u32(Ks) + s * (2 * T5_TILE * 16), (uint32_t)T5_TILE * 16u, 128u),
                      umma_idesc(T5_TILE), s > 0 ? 1u : 0u);
          if (s == NPV - 1) umma_commit(bar_o);  // everything issued so far, the whole O part among it
        }
        umma_commit(bar);
      }
    }
  }

  // ---- the partial result of this key range: O (leading + remainder lanes), max, sum
  __syncthreads();
  bool fin = false;
  if (!S.abort) fin = mbar_wait(bar, (uint32_t)n_tiles & 1u, abort);
  t5_fence_after();
  if (warp < 4) {
    // the copy warp has drained its copies before it got here and the last instructions have
    // finished: the raw V, transposed V and p areas together serve as the exchange area
    float* Ox = reinterpret_cast<float*>(Vraw);
    if (fin && half == 1) {
      float* dst = Ox + (size_t)r_loc * Lay::OX_STRIDE;
#pragma unroll
      for (int c0 = 0; c0 < HD; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(t_o + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          reinterpret_cast<float4*>(dst + c0)[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                                __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
      }
      dst[HD] = (l_run.a + l_run.b) + (l_run.c + l_run.d);  // this half's share of the row's sum
    }
    row_sync();
    if (fin && half == 0) {
      float* dst = part + (((size_t)m * Hq + h) * nsplit + sp) * (HD + 2);
      const float* other = Ox + (size_t)r_loc * Lay::OX_STRIDE;
#pragma unroll
      for (int c0 = 0; c0 < HD; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(t_o + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
        if (row_ok) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float2 x = *reinterpret_cast<const float2*>(other + c0 + 2 * j);
            *reinterpret_cast<float2*>(dst + c0 + 2 * j) =
                make_float2(__uint_as_float(v[2 * j]) + x.x, __uint_as_float(v[2 * j + 1]) + x.y);
          }
        }
      }
      if (row_ok) {
        dst[HD] = m_run;
        dst[HD + 1] = ((l_run.a + l_run.b) + (l_run.c + l_run.d)) + other[HD];
      }
    }
  }
  t5_fence_before();
  __syncthreads();
  if (warp == 4) {
    t5_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)Lay::TMEM_COLS) : "memory");
  }
  if (tid == 0 && *abort) atomicOr(status, SSD_STATUS_TIMEOUT);
}

}  // namespace

bool tc_attention5_supported(int hd, int G, int R) { return (hd == 64 || hd == 128) && G * R >= 1; }

template <int HD>
static cudaError_t launch5(const float* qrot, const bf16* kv_layer, const int32_t* len, RowMap rm, int cap, int Hq,
                           int Hkv, float* part, int nsplit, int keys_per_split, const int32_t* page_table,
                           int max_pages, int32_t* status, cudaStream_t st) {
  const int NQ = (Hq / Hkv) * rm.R, n_rowgroups = (NQ + 63) / 64;
  auto kern = tc_attn5_kernel<HD>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, T5Lay<HD>::TOTAL);
  if (e != cudaSuccess) return e;
  e = tc_launch_pdl(kern, dim3(nsplit, Hkv * n_rowgroups, rm.nb), dim3(T5_THREADS), (size_t)T5Lay<HD>::TOTAL, st, qrot,
                    kv_layer, len, rm, cap, Hq, Hkv, n_rowgroups, part, nsplit, keys_per_split, page_table, max_pages,
                    status);
  if (e != cudaSuccess) return e;
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_tc_attention5(const float* qrot, const bf16* kv_layer, const int32_t* len, RowMap rm, int cap,
                                 int Hq, int Hkv, int hd, float* part, int nsplit, int keys_per_split,
                                 const int32_t* page_table, int max_pages, int32_t* status, cudaStream_t st) {
  if (hd == 128)
    return launch5<128>(qrot, kv_layer, len, rm, cap, Hq, Hkv, part, nsplit, keys_per_split, page_table, max_pages,
                        status, st);
  if (hd == 64)
    return launch5<64>(qrot, kv_layer, len, rm, cap, Hq, Hkv, part, nsplit, keys_per_split, page_table, max_pages,
                       status, st);
  return cudaErrorInvalidValue;
}

}  // namespace ssd
