// Projections of the batched verify forward on tcgen05 tensor cores with the accumulator in tensor
// memory (QKV, O, gate/up + SwiGLU, down, LM head of Eq. 4's decoder pass when more than 16 rows
// are in flight).  Layouts and the reasons for them: tc.h.
//
// One CTA = one tile of 128 weight rows x one K slice x all token rows - or, with more than 256
// token rows, two tiles x one K slice x one chunk of the rows.  Warp 0 streams the
// operands: per pipeline stage, eight of its lanes issue bulk copies of the stage's weight blocks
// (read once from HBM, marked evict-first) and of the matching activation blocks (re-read by every
// tile, so they stay in L2), in pieces of 8 KB, all completing on the stage's "full" barrier.  Warp 1 owns tensor
// memory and issues the MMAs: per k-step of 16 columns one tcgen05.mma over both parts of the
// activations (up to 256 rows: 128 x 2 Mpad x 16), or one per part and tile (128 x Mc x 16), bf16 x
// bf16 -> fp32, reading both operands straight from shared memory; a tcgen05.commit hands
// the stage back to the copy warp through its "empty" barrier, a last one tells the epilogue
// warps that the accumulator is complete.  Then all eight warps (two per quarter of the tensor-memory
// lanes) read the accumulator, 32 lanes x 32 columns at a time (lane = weight row, column = token),
// and apply the epilogue.
//
// Every wait is bounded: when one runs out the CTA raises SSD_STATUS_TIMEOUT, stops issuing, waits
// (bounded again) for the copies it has in flight, frees its tensor memory and returns.
#include <math_constants.h>

#include "kernels.h"
#include "tc.h"

namespace ssd {

namespace {

constexpr unsigned long long TC_WAIT_CYCLES = 2000000000ull;  // ~1 s
constexpr int TC_MAX_STAGES = 12;
// Operand copies are issued by several lanes of the copy warp, in pieces of at most 8 KB: measured
// on a B200, one thread issuing one large copy per operand and stage moves 35-48 GB/s into an SM,
// eight lanes issuing 8 KB pieces 46-90 GB/s.
constexpr int TC_ISSUERS = 8;
constexpr uint32_t TC_PIECE = 8192;
// SwiGLU epilogue staging: 32 token rows of 16 bytes per (column half, part), padded against bank conflicts
constexpr uint32_t TC_STG_STRIDE = 528;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
// Bounded wait; gives up (and tells the other roles through *abort) after TC_WAIT_CYCLES or when
// another role has given up.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort) {
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 15u) == 0u) {
      if (*abort) return false;
      if ((unsigned long long)(clock64() - t0) > TC_WAIT_CYCLES) {
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
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar,
                                              uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}

// Shared-memory matrix descriptor of a K-major operand without swizzle: start address, byte
// distance between core matrices along K (leading) and along the rows (stride), all in units of
// 16 bytes; bit 46 marks the descriptor format of this architecture.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lead_bytes, uint32_t stride_bytes) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lead_bytes >> 4) << 16) |
         ((uint64_t)(stride_bytes >> 4) << 32) | (1ull << 46);
}
// Instruction descriptor of kind::f16: fp32 accumulator, bf16 A and B, both K-major, M = 128.
__device__ __forceinline__ uint32_t umma_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TC_TILE_ROWS >> 4) << 24);
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
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
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

struct TcKernelParams {
  const uint8_t* w;
  const uint8_t* a;
  int n_rows, KS, M, Mpad, ld_part;  // KS = k-steps of the whole projection; ld_part = tiles * 128
  int Mc;                            // token rows of a row chunk (= Mpad up to 256 rows)
  int ntile;                         // weight-row tiles per CTA: 2 where the rows are chunked, else 1
  int sk, stages;                    // k-steps per stage, pipeline depth
  int wide;                          // 1: one instruction multiplies both parts (N over 2 * Mpad rows)
  int dual;                          // wide, and even / odd k-steps accumulate into two column sets
  int nchunks, chunk_n;              // row ranges of the activation operand per MMA (<= 256 each)
  int tmem_cols;
  int epi;
  float* part;
  float* out;
  int ldo;
  uint8_t* act_out;
  int32_t* status;
};

struct TcShared {
  unsigned long long full[TC_MAX_STAGES], empty[TC_MAX_STAGES], accum;
  uint32_t tmem_base;
  int abort;
};

__global__ void __launch_bounds__(TC_THREADS) tc_gemm_kernel(const __grid_constant__ TcKernelParams P) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int split = blockIdx.y, nsplit = gridDim.y, chunk = blockIdx.z;
  const int tile0 = (int)blockIdx.x * P.ntile;                       // first weight-row tile of this CTA
  const int n_tiles_all = P.ld_part / TC_TILE_ROWS;
  const int ntile = min(P.ntile, n_tiles_all - tile0);               // a last odd tile stands alone
  const int t0 = chunk * P.Mc;                                       // first token row of this CTA
  const int rows_here = min(P.M - t0, P.Mc);                         // valid token rows
  const uint32_t tile_w = (uint32_t)P.sk * TC_WBLOCK;                // one tile's weights of a stage
  const uint32_t stage_w = (uint32_t)P.ntile * tile_w, act_block = (uint32_t)P.Mc * 64u;
  const uint32_t stage_a = (uint32_t)P.sk * act_block;
  uint8_t* smem_w = smem;
  uint8_t* smem_a = smem + (size_t)P.stages * stage_w;
  TcShared& S = *reinterpret_cast<TcShared*>(smem_a + (size_t)P.stages * stage_a);
  const int ks0 = (int)(((long long)split * P.KS) / nsplit), ks1 = (int)(((long long)(split + 1) * P.KS) / nsplit);
  const int n_iter = (ks1 - ks0 + P.sk - 1) / P.sk;
  const bool dual = P.dual && ks1 - ks0 >= 2;  // the second column set needs a k-step of its own

  if (tid == 0) {
    for (int s = 0; s < P.stages; ++s) {
      mbar_init(smem_u32(&S.full[s]), TC_ISSUERS);
      mbar_init(smem_u32(&S.empty[s]), 1);
    }
    mbar_init(smem_u32(&S.accum), 1);
    S.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  tc_pdl_trigger();
  // The copy warp does not wait here: the first weight copies depend on nothing and go out at
  // once.  Everyone else needs the predecessor's results (or tensor memory, which must not be
  // held while the predecessor may still want it).
  if (warp != 0) tc_pdl_wait();
  if (warp == 1) {  // tensor memory: one warp allocates, the same warp frees
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&S.tmem_base)), "r"((uint32_t)P.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = S.tmem_base;
  volatile int* abort = &S.abort;

  if (warp == 0) {
    if (lane >= TC_ISSUERS) tc_pdl_wait();
    if (lane < TC_ISSUERS) {  // ---- operand copies: piece i of a stage is issued by lane i % TC_ISSUERS
      const uint64_t pol = policy_evict_first();
      const uint8_t* wsrc = P.w + ((size_t)tile0 * P.KS + ks0) * TC_WBLOCK;
      const size_t wtile = (size_t)P.KS * TC_WBLOCK;  // from one tile's weights to the next tile's
      const uint8_t* asrc = P.a + ((size_t)chunk * P.KS + ks0) * act_block;
      // One stage's pieces; which = 1: weights, 2: activations, 3: both.  A lane arrives once per
      // stage (with the weights, or with `both`), announcing all the bytes it will bring.  Each
      // tile's weights of the stage and the stage's activations are contiguous runs, cut into
      // pieces of at most 8 KB.
      auto issue = [&](int it, int which) {
        const int s = it % P.stages;
        const int nks = min(P.sk, ks1 - ks0 - it * P.sk);
        const uint32_t bar = smem_u32(&S.full[s]);
        const uint32_t wbytes = (uint32_t)nks * TC_WBLOCK, abytes = (uint32_t)nks * act_block;
        const uint32_t wp1 = (wbytes + TC_PIECE - 1) / TC_PIECE, wp = wp1 * (uint32_t)ntile;
        const uint32_t ap = (abytes + TC_PIECE - 1) / TC_PIECE;
        const uint8_t* ws = wsrc + (size_t)it * P.sk * TC_WBLOCK;
        const uint8_t* as = asrc + (size_t)it * P.sk * act_block;
        // one pass: issue, and add up what this lane announces (the arrival may follow the
        // copies: the phase cannot complete before all issuing lanes have arrived)
        uint32_t mine = 0;
        for (uint32_t i = lane; i < wp + ap; i += TC_ISSUERS) {
          if (i < wp) {
            const uint32_t tl = i >= wp1 ? 1u : 0u, off = (i - tl * wp1) * TC_PIECE;  // at most two tiles
            const uint32_t nb = min(TC_PIECE, wbytes - off);
            mine += nb;
            if (which & 1)
              bulk_g2s_hint(smem_u32(smem_w + (size_t)s * stage_w) + tl * tile_w + off, ws + (size_t)tl * wtile + off, nb,
                            bar, pol);
          } else {
            const uint32_t off = (i - wp) * TC_PIECE, nb = min(TC_PIECE, abytes - off);
            mine += nb;
            if (which & 2) bulk_g2s(smem_u32(smem_a + (size_t)s * stage_a) + off, as + off, nb, bar);
          }
        }
        if (which & 1) mbar_expect_tx(bar, mine);
      };
      // first fill of the ring: the weights at once, the activations when the predecessor is done
      const int first = min(n_iter, P.stages);
      for (int it = 0; it < first; ++it) issue(it, 1);
      tc_pdl_wait();
      for (int it = 0; it < first; ++it) issue(it, 2);
      int it = first;
      for (; it < n_iter; ++it) {
        const int s = it % P.stages, use = it / P.stages;
        if (!mbar_wait(smem_u32(&S.empty[s]), (uint32_t)(use - 1) & 1u, abort)) break;
        issue(it, 3);
      }
      if (*abort) {
        // never leave with copies in flight into this CTA's shared memory: the last uses of the
        // stages either completed long ago (the wait returns at once) or land within the limit
        for (int j = max(0, it - P.stages); j < it; ++j)
          mbar_wait(smem_u32(&S.full[j % P.stages]), (uint32_t)(j / P.stages) & 1u, abort);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {  // ---- MMA issue
      for (int it = 0; it < n_iter; ++it) {
        const int s = it % P.stages, use = it / P.stages;
        if (!mbar_wait(smem_u32(&S.full[s]), (uint32_t)use & 1u, abort)) break;
        tc_fence_after();
        const int nks = min(P.sk, ks1 - ks0 - it * P.sk);
        const uint32_t wb = smem_u32(smem_w + (size_t)s * stage_w), ab = smem_u32(smem_a + (size_t)s * stage_a);
        for (int j = 0; j < nks; ++j) {
          const uint64_t da = umma_desc(wb + (uint32_t)j * TC_WBLOCK, 2048u, 128u);
          const uint32_t blk = ab + (uint32_t)j * act_block, lead = (uint32_t)P.Mc * 32u;
          if (dual) {
            // Back-to-back instructions into the same accumulator columns wait for one another
            // (~280 cycles each, measured, against ~165 when they alternate between column
            // ranges): even k-steps add into columns [0, 2 Mc), odd ones into [2 Mc, 4 Mc).
            const int kk = it * P.sk + j;
            umma_bf16(tmem + (uint32_t)((kk & 1) * 2 * P.Mc), da, umma_desc(blk, lead, 128u), umma_idesc(2 * P.Mc),
                      kk >= 2 ? 1u : 0u);
          } else if (P.wide) {
            // the operand's 2 * Mc rows (leading parts, then remainders) in ranges of <= 256:
            // accumulator columns [0, Mc) receive W x_hi, [Mc, 2 Mc) receive W x_lo
            for (int c = 0; c < P.nchunks; ++c) {
              const int n = min(P.chunk_n, 2 * P.Mc - c * P.chunk_n);
              umma_bf16(tmem + (uint32_t)(c * P.chunk_n), da, umma_desc(blk + (uint32_t)(c * P.chunk_n) * 16u, lead, 128u),
                        umma_idesc(n), (it > 0 || j > 0) ? 1u : 0u);
            }
          } else {
            // more than 256 token rows: this CTA's chunk of Mc rows against its one or two tiles;
            // tile u accumulates in columns [u Mc, (u + 1) Mc), both parts into the same columns
#pragma unroll
            for (int part = 0; part < 2; ++part) {
              for (int u = 0; u < ntile; ++u)
                umma_bf16(tmem + (uint32_t)(u * P.Mc), umma_desc(wb + (uint32_t)u * tile_w + (uint32_t)j * TC_WBLOCK, 2048u, 128u),
                          umma_desc(blk + (uint32_t)(part * P.Mc) * 16u, lead, 128u), umma_idesc(P.Mc),
                          (it > 0 || j > 0 || part > 0) ? 1u : 0u);
            }
          }
        }
        umma_commit(smem_u32(&S.empty[s]));  // the stage is free once these MMAs have read it
      }
      umma_commit(smem_u32(&S.accum));       // also in the abort path: dealloc waits for it below
    }
  }
  {
    // ---- epilogue, by all eight warps (the copy and the issuing warp have finished their parts):
    // warp w may read the 32 tensor-memory lanes of quarter w % 4, so each quarter has two warps,
    // which take the 32-column ranges alternately
    __syncwarp();
    const int q = warp & 3, sub = warp >> 2, row = q * 32 + lane;
    const bool ok = mbar_wait(smem_u32(&S.accum), 0u, abort);
    tc_fence_after();
    if (ok && !*abort) {
     for (int u = 0; u < ntile; ++u) {
      const int tile = tile0 + u, n = tile * TC_TILE_ROWS + row;
      const uint32_t cb = (uint32_t)(u * P.Mc);  // the tile's accumulator columns (two-tile CTAs)
      for (int c0 = sub * 32; c0 < rows_here; c0 += 64) {
        uint32_t v[32];
        tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + cb + (uint32_t)c0, v);
        if (P.wide) {  // add the remainder part's products
          uint32_t w[32];
          tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(P.Mc + c0), w);
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) + __uint_as_float(w[i]));
          if (dual) {  // and the odd k-steps' column set, in a fixed order
            uint32_t x[32];
            tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(2 * P.Mc + c0), x);
            tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(3 * P.Mc + c0), w);
#pragma unroll
            for (int i = 0; i < 32; ++i)
              v[i] = __float_as_uint(__uint_as_float(v[i]) + (__uint_as_float(x[i]) + __uint_as_float(w[i])));
          }
        }
        if (P.epi == TC_EPI_PARTIAL) {
          float* dst = P.part + ((size_t)split * P.Mpad + t0 + c0) * P.ld_part + n;
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (c0 + i < rows_here) dst[(size_t)i * P.ld_part] = __uint_as_float(v[i]);
        } else if (P.epi == TC_EPI_STORE) {
          if (n < P.n_rows) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (c0 + i < rows_here) P.out[(size_t)(t0 + c0 + i) * P.ldo + n] = __uint_as_float(v[i]);
          }
        } else {
          // TC_EPI_SWIGLU: even lanes hold gate_j, odd lanes up_j, j = n / 2.  The warp's 16 columns j
          // are one k-step block of the output operand.  The two lanes of a pair share the work
          // (even lane: even tokens of the range, odd lane: odd tokens); the bf16 parts go through
          // a small staging area in shared memory (the pipeline stages are idle by now) so that
          // global memory sees whole 16-byte rows, 512 contiguous bytes per warp store, instead
          // of two-byte pieces (measured: the epilogue of a 448-row tile 41 -> 6 us).
          const int j0 = (tile * TC_TILE_ROWS + q * 32) >> 1, jl = lane >> 1, odd = lane & 1;
          uint8_t* stg = smem + (size_t)warp * (4 * TC_STG_STRIDE);
          const uint32_t my = (uint32_t)((jl >> 3) * 2) * TC_STG_STRIDE + (uint32_t)(jl & 7) * 2u;
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float a = __uint_as_float(v[i]), b = __uint_as_float(v[i + 1]);
            const float got = __shfl_xor_sync(0xffffffffu, odd ? a : b, 1);
            const float gate = odd ? got : a, up = odd ? b : got;
            const float x = __fdividef(gate, 1.f + __expf(-gate)) * up;
            const bf16 hi = __float2bfloat16_rn(x);
            const bf16 lo = __float2bfloat16_rn(x - __bfloat162float(hi));
            uint8_t* e = stg + my + (uint32_t)(i + odd) * 16u;
            *reinterpret_cast<bf16*>(e) = hi;
            *reinterpret_cast<bf16*>(e + TC_STG_STRIDE) = lo;
          }
          __syncwarp();
          if (j0 < ((P.n_rows / 2 + 15) & ~15) && c0 + lane < rows_here) {
            // the output operand has the same rows, so the same chunks, and n_rows / 2 columns
            uint8_t* blk = P.act_out + ((size_t)chunk * ((P.n_rows / 2 + 15) >> 4) + (size_t)(j0 >> 4)) * ((size_t)P.Mc * 64) +
                           (size_t)(c0 + lane) * 16;
#pragma unroll
            for (int hp = 0; hp < 4; ++hp)  // hp = half * 2 + part
              *reinterpret_cast<uint4*>(blk + (size_t)hp * ((size_t)P.Mc * 16)) =
                  *reinterpret_cast<const uint4*>(stg + (uint32_t)hp * TC_STG_STRIDE + (uint32_t)lane * 16u);
          }
          __syncwarp();
        }
      }
     }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    // the accumulator barrier completes when every MMA issued above has finished
    if (lane == 0) mbar_wait(smem_u32(&S.accum), 0u, abort);
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)P.tmem_cols) : "memory");
  }
  if (tid == 0 && *abort) atomicOr(P.status, SSD_STATUS_TIMEOUT);
}

// ---- weight packing (once per model) -----------------------------------------------------------

__global__ void tc_pack_weights_kernel(const bf16* __restrict__ w, int n_rows, int K, int KS, size_t n_chunks,
                                       uint4* __restrict__ out) {
  // one thread = one 16-byte row of a core matrix: chunk = ((tile * KS + ks) * 2 + kc) * 128 + r
  const size_t c = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= n_chunks) return;
  const int r = (int)(c & 127), kc = (int)((c >> 7) & 1);
  const size_t blk = c >> 8;
  const int ks = (int)(blk % KS), tile = (int)(blk / KS);
  const int n = tile * TC_TILE_ROWS + r, k0 = ks * 16 + kc * 8;
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (n < n_rows && k0 < K) v = *reinterpret_cast<const uint4*>(w + (size_t)n * K + k0);  // K is a multiple of 8
  out[c] = v;
}

__global__ void tc_unpack_weights_kernel(const uint4* __restrict__ packed, int n_rows, int K, int KS,
                                         size_t n_chunks, bf16* __restrict__ w) {
  const size_t c = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= n_chunks) return;
  const int r = (int)(c & 127), kc = (int)((c >> 7) & 1);
  const size_t blk = c >> 8;
  const int ks = (int)(blk % KS), tile = (int)(blk / KS);
  const int n = tile * TC_TILE_ROWS + r, k0 = ks * 16 + kc * 8;
  if (n < n_rows && k0 < K) *reinterpret_cast<uint4*>(w + (size_t)n * K + k0) = packed[c];
}

}  // namespace

cudaError_t tc_pack_weights(const bf16* w, int n_rows, int K, uint8_t* packed, cudaStream_t st) {
  const int KS = (K + 15) / 16;
  const size_t n_chunks = tc_weight_bytes(n_rows, K) / 16;
  tc_pack_weights_kernel<<<(unsigned)((n_chunks + 255) / 256), 256, 0, st>>>(w, n_rows, K, KS, n_chunks,
                                                                            reinterpret_cast<uint4*>(packed));
  count_launch();
  return cudaGetLastError();
}

cudaError_t tc_unpack_weights(const uint8_t* packed, int n_rows, int K, bf16* w, cudaStream_t st) {
  const int KS = (K + 15) / 16;
  const size_t n_chunks = tc_weight_bytes(n_rows, K) / 16;
  tc_unpack_weights_kernel<<<(unsigned)((n_chunks + 255) / 256), 256, 0, st>>>(
      reinterpret_cast<const uint4*>(packed), n_rows, K, KS, n_chunks, w);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_tc_gemm(const TcGemm& g, cudaStream_t st) {
  if (g.M < 1 || g.M > TC_MAX_ROWS || g.ksplit < 1 || (g.K & 7) || g.n_rows < 1) return cudaErrorInvalidValue;
  TcKernelParams p{};
  p.w = g.w;
  p.a = g.a;
  p.n_rows = g.n_rows;
  p.KS = (g.K + 15) / 16;
  p.M = g.M;
  p.Mpad = tc_round16(g.M);
  const int tiles = (g.n_rows + TC_TILE_ROWS - 1) / TC_TILE_ROWS;
  p.ld_part = tiles * TC_TILE_ROWS;
  p.epi = g.epi;
  p.part = g.part;
  p.out = g.out;
  p.ldo = g.ldo;
  p.act_out = g.act_out;
  p.status = g.status;
  if (g.ksplit > p.KS || (g.epi != TC_EPI_PARTIAL && g.ksplit != 1)) return cudaErrorInvalidValue;
  // pipeline: at least three stages of as many k-steps as fit (measured at 448 rows: six stages
  // of one k-step are 12 % slower than three of two - fewer, larger copies win).  A grid that exceeds the SM count
  // by a little leaves room for a second CTA per SM so that it still runs in one wave; any other
  // grid takes the whole shared memory: with few token rows the weight stream is latency-bound,
  // and what a CTA keeps in flight is what it gets.
  const TcChunks ch = tc_chunks(g.M);
  p.Mc = ch.rows;
  p.ntile = tc_tiles_per_cta(g.n_rows, g.K, g.M);
  const int grid_x = (tiles + p.ntile - 1) / p.ntile;
  const size_t per_ks = (size_t)p.ntile * TC_WBLOCK + (size_t)p.Mc * 64;
  int n_sm = 148;
  {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sm < 1)
      n_sm = 148;
  }
  const int ctas = grid_x * g.ksplit * ch.n;
  const bool two_per_sm = p.Mpad <= 128 && ctas > n_sm && ctas <= 2 * n_sm;  // 2 x 256 columns
  const size_t budget = two_per_sm ? 100 * 1024 : 216 * 1024;
  p.sk = 4;
  while (p.sk > 1 && 3 * p.sk * per_ks > budget) p.sk >>= 1;
  p.stages = (int)(budget / (p.sk * per_ks));
  if (p.stages > TC_MAX_STAGES) p.stages = TC_MAX_STAGES;
  if (p.stages < 2) return cudaErrorInvalidValue;
  p.wide = ch.n == 1;  // both parts' products fit the 512 tensor-memory columns side by side
  const int op_rows = p.wide ? 2 * p.Mc : p.ntile * p.Mc;  // accumulator columns
  p.nchunks = p.wide ? (op_rows + 255) / 256 : 1;
  p.chunk_n = p.wide ? tc_round16((op_rows + p.nchunks - 1) / p.nchunks) : p.Mc;
  p.dual = p.wide && 4 * p.Mc <= 512 && !two_per_sm;  // two CTAs on an SM have 256 columns each
  p.tmem_cols = 32;
  while (p.tmem_cols < (p.dual ? 2 : 1) * op_rows) p.tmem_cols <<= 1;
  const size_t smem = (size_t)p.stages * p.sk * per_ks + sizeof(TcShared) + 64;
  cudaError_t e = cudaFuncSetAttribute(tc_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e != cudaSuccess) return e;
  e = tc_launch_pdl(tc_gemm_kernel, dim3(grid_x, g.ksplit, ch.n), dim3(TC_THREADS), smem, st, p);
  if (e != cudaSuccess) return e;
  count_launch();
  return cudaGetLastError();
}

}  // namespace ssd
