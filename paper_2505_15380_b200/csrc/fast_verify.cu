// Persistent small-batch verify forward (Eq. 4: one causal-decoder pass over the pending token and
// the gamma draft tokens of each stream against the cached prefix), T = B * (gamma + 1) <= 16 rows.
//
// One CTA per SM lives for the whole forward.  Every warp streams its own pre-packed slice of the
// weights from HBM through a private shared-memory ring with bulk async copies that complete on
// mbarriers; a slot is refilled the moment its chunk has been consumed, whatever phase the consumer
// is in, so the weight stream runs ahead of the dependency chain across phase boundaries.  The
// ring is kept shallow on purpose: four 2 KB copies in flight per warp already saturate HBM.
// The phases of a layer (QKV projection, attention, O projection, gate/up, down) are separated by
// grid barriers on one monotonic arrival counter, with bounded waits.
//
// The forward is a chain of ~5 dependent phases per layer, each far shorter than a microsecond of
// memory time, so what bounds it is the number of instructions a warp executes per phase (eight
// warps per SM hide little latency).  Hence: activations are converted once per phase into the
// tensor-core operand layout, the weight stream is pre-cut into chunks of whole k-steps so the
// inner loop is straight-line for each tile count, and everything rare is out of line.
//
// Projections: D[token, weight row] = sum_k X[token, k] * W[row, k] on mma.m16n8k16 (bf16 inputs,
// fp32 accumulate): the 16-row A operand holds the tokens, the B operand one packed tile of 8 weight
// rows.  Activations are fp32 and enter the instruction as a two-term bf16 split (hi + lo), so the
// products are exact to ~2^-17 relative; weights are exactly their stored bf16 values.  The warps
// of a CTA split K; their partial sums are added in a fixed order in shared memory.
#include <math_constants.h>
#include <stdlib.h>

#include "fast.h"
#include "kernels.h"

namespace ssd {

namespace {

constexpr unsigned long long FAST_WAIT_CYCLES = 3000000000ull;  // ~1.5 s at 2 GHz
constexpr int FAST_KEYS_MIN = 64;                                // fewest keys worth a split of their own
constexpr float FIX_SCALE = 4294967296.f;                        // residual stream: 2^-32 fixed point
constexpr float FIX_INV_SCALE = 1.f / 4294967296.f;

enum { EPI_F_QKV = 0, EPI_F_RESID = 1, EPI_F_SWIGLU = 2, EPI_F_LOGITS = 3 };

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
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
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_u32(uint32_t* p, uint32_t v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint2 lds_v2(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Two fp32 values -> packed bf16 pair of their leading parts and of the remainders.
__device__ __forceinline__ void split2(float x, float y, uint32_t& hi, uint32_t& lo) {
  __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  float rx = x - __low2float(h), ry = y - __high2float(h);
  __nv_bfloat162 l = __floats2bfloat162_rn(rx, ry);
  hi = *reinterpret_cast<uint32_t*>(&h);
  lo = *reinterpret_cast<uint32_t*>(&l);
}
// Residual-stream word (2^-32 fixed point) -> fp32, through its two 32-bit halves.
__device__ __forceinline__ float fix_to_float(long long v) {
  const int hi = (int)(v >> 32);
  const unsigned lo = (unsigned)v;
  return fmaf(__uint2float_rn(lo), FIX_INV_SCALE, __int2float_rn(hi));
}

// Per-CTA bookkeeping in shared memory.
struct FastMisc {
  unsigned long long bars[FAST_WARPS][FAST_MAX_SLOTS];
  uint8_t chunks[FAST_WARPS][FAST_MAX_CHUNKS];  // chunk sizes (tiles) of each warp's stream
  int32_t ucnt[FOP_COUNT];
  int32_t utile[FOP_COUNT][FAST_MAX_UNITS];
  float inv_rms[FAST_MAX_T];
  float row_m[FAST_MAX_T], row_l[FAST_MAX_T], row_corr[FAST_MAX_T];
  float wred[FAST_WARPS][FAST_MAX_T];
  int32_t tok_stream[FAST_MAX_T];  // stream of each row of this forward
  int32_t tok_pos[FAST_MAX_T];     // its position len + r
  int32_t last;
};

// A warp's private weight stream and shared-memory ring; every lane keeps an identical copy in
// registers.  One chunk (whole k-steps of a round, at most FAST_SLOT_TILES tiles) fills one slot.
struct Ring {
  uint32_t ring, bars;      // shared addresses of the ring and of its mbarriers
  const uint8_t* src;       // next byte of the stream to request
  const uint8_t* tab;       // this warp's chunk sizes: [ncl] of a layer, then [nch] of the LM head
  uint32_t pc;              // index in `tab` of the next chunk to request
  uint32_t ncl, nend;       // chunks per layer; one past the last table entry to request
  uint32_t layers_left;     // passes over the layer part still to request
  uint32_t slot, parity;    // the consumer's next slot and its phase parity
  uint32_t nslot;
  uint32_t outstanding;     // copies issued and not yet waited for
  bool dead;                // a bounded wait ran out
};

// Tiles of the next chunk to request (0: the stream is exhausted).
__device__ __forceinline__ uint32_t ring_next_chunk(Ring& r) {
  if (r.pc >= r.nend) return 0u;
  const uint32_t n = r.tab[r.pc];
  ++r.pc;
  if (r.layers_left > 0 && r.pc == r.ncl) {
    if (--r.layers_left > 0) r.pc = 0;  // next layer: same chunk sizes; else fall through to the head
  }
  return n;
}
__device__ __forceinline__ void ring_request(Ring& r, uint32_t slot, int lane) {
  const uint32_t n = ring_next_chunk(r);
  if (n) {
    if (lane == 0) {
      const uint32_t bar = r.bars + slot * 8;
      mbar_expect_tx(bar, n * FAST_TILE_BYTES);
      bulk_g2s(r.ring + slot * FAST_SLOT_BYTES, r.src, n * FAST_TILE_BYTES, bar);
    }
    r.src += n * FAST_TILE_BYTES;
    r.outstanding++;
  }
}
__device__ __noinline__ bool bounded_mbar_wait(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if ((unsigned long long)(clock64() - t0) > FAST_WAIT_CYCLES) return false;
  }
  return true;
}
// Waits for the chunk in the consumer's slot.
__device__ __forceinline__ void ring_acquire(Ring& r) {
  const uint32_t bar = r.bars + r.slot * 8;
  if (!r.dead) {
    if (mbar_try_wait(bar, r.parity) || bounded_mbar_wait(bar, r.parity)) r.outstanding--;
    else r.dead = true;
  }
}
// Gives the consumed slot back: the next chunk of the stream is requested into it.
__device__ __forceinline__ void ring_release(Ring& r, int lane) {
  __syncwarp();  // every lane has read its bytes of the slot: it may be overwritten
  if (!r.dead) ring_request(r, r.slot, lane);
  if (++r.slot == r.nslot) {
    r.slot = 0;
    r.parity ^= 1u;
  }
}

__device__ __forceinline__ void trace_mark(const FastParams& P, int& n_trace) {
  if (P.trace && threadIdx.x == 0 && n_trace < P.trace_cap)
    P.trace[(size_t)blockIdx.x * P.trace_cap + n_trace++] = clock64();
}

// Grid-wide barrier on one monotonic arrival counter: it is complete when the counter has
// reached `target`.  One thread per CTA arrives (release) and polls (acquire).  A CTA whose wait
// ran out raises the failure word next to the base; every poller looks at that word now and then,
// so all CTAs give up together.  Returns false in that case.
__device__ __noinline__ bool grid_sync(const FastParams& P, uint32_t target, bool failed) {
  const int bad_in = __syncthreads_or(failed ? 1 : 0);
  bool ok = bad_in == 0;
  if (threadIdx.x == 0) {
    if (bad_in) st_release_u32(P.epoch_base + 1, 1u);
    __threadfence();
    atomicAdd(P.flags, 1u);  // result unused: a fire-and-forget reduction
    if ((int32_t)(ld_acquire_u32(P.flags) - target) < 0) {
      const long long t0 = clock64();
      uint32_t spins = 0;
      while ((int32_t)(ld_acquire_u32(P.flags) - target) < 0) {
        if ((++spins & 63u) == 0u) {
          if (ld_acquire_u32(P.epoch_base + 1) != 0u) {
            ok = false;
            break;
          }
          if ((unsigned long long)(clock64() - t0) > FAST_WAIT_CYCLES) {
            st_release_u32(P.epoch_base + 1, 1u);
            ok = false;
            break;
          }
        }
      }
    }
  }
  return __syncthreads_or(ok ? 0 : 1) == 0;
}

// ---- projections -------------------------------------------------------------------------------

// One projection of the layer: which weights, which input, which epilogue.
struct PhaseDesc {
  const void* in;     // input rows (fixed-point residual stream when in_fix, else fp32)
  const float* gain;  // RMSNorm gain (in_fix only)
  int op;             // FOP_*: whose tiles of this CTA
  int epi;            // EPI_F_*
  int in_fix;
  int ld, kb, kc;     // input row stride; first column and number of columns this CTA covers
  int n_rows;         // valid weight rows (the last tile of the LM head is padded)
  int layer;
  bf16* kv_layer;     // this layer's slice of the cache (QKV epilogue)
  float qscale;       // 1 / sqrt(head_dim)
};

// Shared-memory image of the A operand: for k-step s and lane l (g = l / 4, t = l % 4) 16 bytes
//   { hi(x[g][16s+2t..]), hi(x[g][16s+8+2t..]), lo(same), lo(same) }
// and, when more than 8 rows are in flight, 16 more bytes for row g + 8.
template <bool T16>
__device__ __forceinline__ uint32_t afrag_word(int row, int kk) {  // kk = column pair index
  constexpr int W = T16 ? 8 : 4;
  const int s = kk >> 3, t = kk & 3, which = (kk >> 2) & 1;
  return (uint32_t)(((s * 32 + (row & 7) * 4 + t) * W) + (row >> 3) * 4 + which);
}

// Residual-stream rows -> A operand of x * gain, and the rows' sums of squares, for inputs of at
// most J * 2 * FAST_THREADS columns.  All loads of a batch of rows are in flight before the first
// is used.
template <int J, bool T16>
__device__ __forceinline__ void stage_fix_rows(const longlong2* __restrict__ hin,
                                               const float2* __restrict__ gain2, uint32_t* af,
                                               FastMisc& M, int T, int half_k, int ld2, int tid) {
  constexpr int RB = 16 / J;  // rows per batch
  const int lane = tid & 31, warp = tid >> 5;
  float2 gj[J];
#pragma unroll
  for (int j = 0; j < J; ++j) {
    const int kk = j * FAST_THREADS + tid;
    gj[j] = kk < half_k ? __ldg(gain2 + kk) : make_float2(0.f, 0.f);
  }
  for (int r0 = 0; r0 < T; r0 += RB) {
    longlong2 hv[RB][J];
#pragma unroll
    for (int rr = 0; rr < RB; ++rr) {
#pragma unroll
      for (int j = 0; j < J; ++j) {
        const int kk = j * FAST_THREADS + tid;
        if (r0 + rr < T && kk < half_k) hv[rr][j] = __ldcg(hin + (r0 + rr) * ld2 + kk);
      }
    }
#pragma unroll
    for (int rr = 0; rr < RB; ++rr) {
      const int row = r0 + rr;
      if (row < T) {
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < J; ++j) {
          const int kk = j * FAST_THREADS + tid;
          if (kk < half_k) {
            const float x0 = fix_to_float(hv[rr][j].x), x1 = fix_to_float(hv[rr][j].y);
            ss = fmaf(x0, x0, fmaf(x1, x1, ss));
            uint32_t hi, lo;
            split2(x0 * gj[j].x, x1 * gj[j].y, hi, lo);
            const uint32_t wd = afrag_word<T16>(row, kk);
            af[wd] = hi;
            af[wd + 2] = lo;
          }
        }
        ss = warp_sum(ss);
        if (lane == 0) M.wred[warp][row] = ss;
      }
    }
  }
}

// Stages the input of a projection phase as the A operand in shared memory: columns
// [kb, kb + kc) of an input with row stride `ld` (written by other CTAs in an earlier phase, hence
// read past L1).  With in_fix the input is the fixed-point residual stream and the operand is
// x * gain; the rows' sums of squares go to wred (the RMS scale is applied in the epilogue, which
// is exact because it is one factor per token).
template <bool T16>
__device__ __noinline__ void stage_input(const FastParams& P, FastMisc& M, uint32_t* af,
                                         const PhaseDesc& D) {
  const int T = P.T, tid = threadIdx.x;
  const int kc = D.kc, ld = D.ld;
  if (D.in_fix) {
    const longlong2* hin = static_cast<const longlong2*>(D.in);
    const float2* gain2 = reinterpret_cast<const float2*>(D.gain);
    const int half_k = kc >> 1, ld2 = ld >> 1;
    if (half_k <= FAST_THREADS) stage_fix_rows<1, T16>(hin, gain2, af, M, T, half_k, ld2, tid);
    else if (half_k <= 2 * FAST_THREADS) stage_fix_rows<2, T16>(hin, gain2, af, M, T, half_k, ld2, tid);
    else if (half_k <= 4 * FAST_THREADS) stage_fix_rows<4, T16>(hin, gain2, af, M, T, half_k, ld2, tid);
    else stage_fix_rows<16, T16>(hin, gain2, af, M, T, half_k, ld2, tid);
  } else {
    constexpr int LB = 8;
    const float* fin = static_cast<const float*>(D.in) + D.kb;
    const int c4 = kc >> 2;
    // this thread's float4 elements: (row, col) advancing by FAST_THREADS columns with carry
    int row_l = 0, col_l = tid;
    while (col_l >= c4) { col_l -= c4; ++row_l; }
    int row_u = row_l, col_u = col_l;
    while (row_u < T) {
      float4 v[LB];
#pragma unroll
      for (int i = 0; i < LB; ++i) {
        if (row_l < T) v[i] = __ldcg(reinterpret_cast<const float4*>(fin + row_l * ld) + col_l);
        col_l += FAST_THREADS;
        while (col_l >= c4) { col_l -= c4; ++row_l; }
      }
#pragma unroll
      for (int i = 0; i < LB; ++i) {
        if (row_u < T) {
          uint32_t h0, l0, h1, l1;
          split2(v[i].x, v[i].y, h0, l0);
          split2(v[i].z, v[i].w, h1, l1);
          const uint32_t wd = afrag_word<T16>(row_u, 2 * col_u);  // pair 2c; pair 2c+1 is the next lane's
          af[wd] = h0;
          af[wd + 2] = l0;
          af[wd + (T16 ? 8 : 4)] = h1;
          af[wd + (T16 ? 8 : 4) + 2] = l1;
        }
        col_u += FAST_THREADS;
        while (col_u >= c4) { col_u -= c4; ++row_u; }
      }
    }
  }
  __syncthreads();
}

// One output element pair of a projection: token `tok`, packed weight rows n and n + 1.
__device__ __forceinline__ void epilogue_pair(const FastParams& P, const PhaseDesc& D, const FastMisc& M,
                                              int tok, int n, float c0, float c1) {
  if (D.epi == EPI_F_RESID) {
    // 64-bit integer adds commute: the K slices of different CTAs may arrive in any order and the
    // sum is still bit-reproducible
    unsigned long long* dst = reinterpret_cast<unsigned long long*>(P.hfix + (size_t)tok * P.d + n);
    atomicAdd(dst, (unsigned long long)__float2ll_rn(c0 * FIX_SCALE));
    atomicAdd(dst + 1, (unsigned long long)__float2ll_rn(c1 * FIX_SCALE));
  } else if (D.epi == EPI_F_SWIGLU) {
    P.act[(size_t)tok * P.F + (n >> 1)] = c0 / (1.f + expf(-c0)) * c1;
  } else if (D.epi == EPI_F_LOGITS) {
    if (n < D.n_rows) P.logits[(size_t)tok * P.V + n] = c0;
    if (n + 1 < D.n_rows) P.logits[(size_t)tok * P.V + n + 1] = c1;
  } else {  // EPI_F_QKV: bias, rotary embedding, q scaling, K/V append
    const int hd = P.hd, hs = P.hd_shift, half = hd >> 1, qd = P.Hq << hs, kvd = P.Hkv << hs;
    const float2 bias = *reinterpret_cast<const float2*>(P.m.bias_qkv + (size_t)D.layer * (qd + 2 * kvd) + n);
    const float x1 = c0 + bias.x, x2 = c1 + bias.y;
    const int stream = M.tok_stream[tok], pos = M.tok_pos[tok];
    if (n < qd + kvd) {
      const int j = (n & (hd - 1)) >> 1;
      const float2 cs = __ldcg(reinterpret_cast<const float2*>(P.rope_cs + ((size_t)tok * half + j) * 2));
      const float o1 = x1 * cs.x - x2 * cs.y, o2 = x2 * cs.x + x1 * cs.y;
      if (n < qd) {
        float* q = P.qrot + tok * qd + (n & ~(hd - 1));
        q[j] = o1 * D.qscale;
        q[j + half] = o2 * D.qscale;
      } else if (pos < P.cap) {
        const int gk = (n - qd) >> hs;
        bf16* kdst = D.kv_layer + (((size_t)stream * 2 + 0) * P.Hkv + gk) * (size_t)P.cap * hd + (size_t)pos * hd;
        kdst[j] = __float2bfloat16_rn(o1);
        kdst[j + half] = __float2bfloat16_rn(o2);
      } else {
        atomicOr(P.status, SSD_STATUS_KV_OVERFLOW);
      }
    } else if (pos < P.cap) {
      const int nn = n - qd - kvd, gk = nn >> hs, jj = nn & (hd - 1);
      bf16* vdst = D.kv_layer + (((size_t)stream * 2 + 1) * P.Hkv + gk) * (size_t)P.cap * hd + (size_t)pos * hd;
      *reinterpret_cast<__nv_bfloat162*>(vdst + jj) = __floats2bfloat162_rn(x1, x2);
    }
  }
}

// The tensor-core work of one round of CNT tiles over this warp's k-steps [s0, s1): straight-line
// per chunk (one ring slot = SPC whole k-steps), partial sums to shared memory at the end.
template <int CNT, bool T16>
__device__ __forceinline__ void mma_round(Ring& r, int lane, uint32_t af_lane, int s0, int s1, bool row0,
                                          bool row1, float* red_dst) {
  constexpr int SPC = FAST_SLOT_TILES / CNT;
  constexpr uint32_t STEP = T16 ? 1024u : 512u;
  constexpr int NACC = T16 ? 4 : 2;
  float acc[CNT][4];
#pragma unroll
  for (int u = 0; u < CNT; ++u) acc[u][0] = acc[u][1] = acc[u][2] = acc[u][3] = 0.f;
#pragma unroll 1
  for (int s = s0; s < s1; s += SPC) {
    ring_acquire(r);
    const uint32_t wb = r.ring + r.slot * FAST_SLOT_BYTES + lane * 8;
#pragma unroll
    for (int i = 0; i < SPC; ++i) {
      if (SPC == 1 || s + i < s1) {
        uint32_t ahi[4], alo[4];
        uint4 a = make_uint4(0u, 0u, 0u, 0u);
        if (row0) a = lds_v4(af_lane + (uint32_t)(s + i) * STEP);
        ahi[0] = a.x; ahi[2] = a.y; alo[0] = a.z; alo[2] = a.w;
        if (T16) {
          uint4 a2 = make_uint4(0u, 0u, 0u, 0u);
          if (row1) a2 = lds_v4(af_lane + (uint32_t)(s + i) * STEP + 16u);
          ahi[1] = a2.x; ahi[3] = a2.y; alo[1] = a2.z; alo[3] = a2.w;
        } else {
          ahi[1] = ahi[3] = alo[1] = alo[3] = 0u;
        }
        uint2 b[CNT];
#pragma unroll
        for (int u = 0; u < CNT; ++u) b[u] = lds_v2(wb + (uint32_t)(i * CNT + u) * FAST_TILE_BYTES);
#pragma unroll
        for (int u = 0; u < CNT; ++u) mma_bf16(acc[u], ahi, b[u].x, b[u].y);
#pragma unroll
        for (int u = 0; u < CNT; ++u) mma_bf16(acc[u], alo, b[u].x, b[u].y);
      }
    }
    ring_release(r, lane);
  }
#pragma unroll
  for (int u = 0; u < CNT; ++u) {
    float* dst = red_dst + (size_t)u * 32 * NACC;
    *reinterpret_cast<float2*>(dst) = make_float2(acc[u][0], acc[u][1]);
    if (T16) *reinterpret_cast<float2*>(dst + 2) = make_float2(acc[u][2], acc[u][3]);
  }
}

// One projection phase: stage the input, run this CTA's tiles (the warps split K), add the warps'
// partial sums in shared memory and apply the epilogue.
template <bool T16>
__device__ __forceinline__ void gemm_phase(const FastParams& P, FastMisc& M, uint8_t* uni, Ring& ring,
                                           const PhaseDesc& D) {
  constexpr int NACC = T16 ? 4 : 2;
  const int cnt_total = M.ucnt[D.op];
  if (cnt_total == 0) return;
  const int T = P.T, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2;
  const int KS = D.kc >> 4;
  uint32_t* af = reinterpret_cast<uint32_t*>(uni);                             // A operand, KS steps
  float* red = reinterpret_cast<float*>(uni + (size_t)KS * (T16 ? 1024 : 512));  // [warp][MAXU][32][NACC]
  stage_input<T16>(P, M, af, D);
  if (D.in_fix && tid < T) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < FAST_WARPS; ++w) tot += M.wred[w][tid];
    M.inv_rms[tid] = rsqrtf(tot / (float)D.kc + P.eps);
  }
  const int s0 = fast_warp_k0(warp, KS), s1 = fast_warp_k1(warp, KS);
  const uint32_t af_lane = smem_u32(af) + lane * (T16 ? 32u : 16u);
  const bool row0 = g < T, row1 = T16 && g + 8 < T;
  float* red_dst = red + ((size_t)warp * FAST_MAXU * 32 + lane) * NACC;

  for (int u0 = 0; u0 < cnt_total; u0 += FAST_MAXU) {
    const int cnt = min(FAST_MAXU, cnt_total - u0);
    switch (cnt) {
      case 1: mma_round<1, T16>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      case 2: mma_round<2, T16>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      case 3: mma_round<3, T16>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      case 4: mma_round<4, T16>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      case 5: mma_round<5, T16>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      case 6: mma_round<6, T16>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      case 7: mma_round<7, T16>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      default: mma_round<8, T16>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
    }
    __syncthreads();
    for (int idx = tid; idx < cnt * 32; idx += FAST_THREADS) {
      const int u = idx >> 5, l = idx & 31, gg = l >> 2, tt = l & 3;
      float c[NACC];
#pragma unroll
      for (int i = 0; i < NACC; ++i) c[i] = 0.f;
#pragma unroll
      for (int w = 0; w < FAST_WARPS; ++w) {  // fixed order: bit-reproducible
        const float* src = red + (((size_t)w * FAST_MAXU + u) * 32 + l) * NACC;
#pragma unroll
        for (int i = 0; i < NACC; ++i) c[i] += src[i];
      }
      const int n = M.utile[D.op][u0 + u] * 8 + 2 * tt;
      if (gg < T) {
        const float inv = D.in_fix ? M.inv_rms[gg] : 1.f;
        epilogue_pair(P, D, M, gg, n, c[0] * inv, c[1] * inv);
      }
      if (T16 && gg + 8 < T) {
        const float inv = D.in_fix ? M.inv_rms[gg + 8] : 1.f;
        epilogue_pair(P, D, M, gg + 8, n, c[NACC - 2] * inv, c[NACC - 1] * inv);
      }
    }
    if (u0 + FAST_MAXU < cnt_total) __syncthreads();
  }
}

// ---- attention ---------------------------------------------------------------------------------

// Work item = (stream, query head, key split).  The item's CTA stages KT keys / values at a time
// in shared memory, computes the scores of the stream's R rows (row r sees keys 0..len + r:
// causal inside the draft block), keeps a running max / sum per row and accumulates P * V in
// shared memory.  With more than one split the partials go to global memory and the CTA that
// arrives last for a (stream, head) merges them in split order.
template <int HD>
__device__ __noinline__ void attn_phase(const FastParams& P, FastMisc& M, uint8_t* uni, int layer) {
  constexpr int KT = 8192 / HD;         // keys per tile (a power of two >= 64)
  constexpr int KROW = HD * 2 + 16;     // padded K row in bytes (conflict-free 16-byte reads)
  const int R = P.R, nb = P.nb, Hq = P.Hq, G = Hq / P.Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int max_total = 0;
  for (int bi = 0; bi < nb; ++bi) max_total = max(max_total, min(M.tok_pos[bi * R] + R, P.cap));
  int nsplit = (max_total + FAST_KEYS_MIN - 1) / FAST_KEYS_MIN;
  nsplit = max(1, min(nsplit, min(FAST_NSPLIT_CAP, max(1, P.m.n_cta / (nb * Hq)))));
  const int items = nb * Hq * nsplit;

  float* qs = reinterpret_cast<float*>(uni);                     // [R][HD]
  uint8_t* Ks = reinterpret_cast<uint8_t*>(qs + R * HD);          // [KT][KROW]
  bf16* Vs = reinterpret_cast<bf16*>(Ks + KT * KROW);             // [KT][HD]
  float* ps = reinterpret_cast<float*>(Vs + KT * HD);             // [R][KT] scores, then weights
  float* acc_s = ps + R * KT;                                     // [R][HD] running P * V
  const bf16* kvl = P.kv + (size_t)layer * P.kv_layer_elems;

  for (int item = blockIdx.x; item < items; item += P.m.n_cta) {
    const int c = item % nsplit, hq = (item / nsplit) % Hq, bi = item / (nsplit * Hq);
    const int stream = P.b0 + bi, gk = hq / G;
    const int L = M.tok_pos[bi * R], total = min(L + R, P.cap);
    const int per = (((total + nsplit - 1) / nsplit) + 7) & ~7;
    const int k0 = c * per, k1 = min(k0 + per, total);
    __syncthreads();
    {
      constexpr int QB = FAST_MAX_T * HD / FAST_THREADS;  // covers R * HD <= 16 * HD values
      float qv[QB];
#pragma unroll
      for (int i = 0; i < QB; ++i) {
        const int idx = tid + i * FAST_THREADS;
        if (idx < R * HD) qv[i] = __ldcg(P.qrot + ((size_t)(bi * R + idx / HD) * Hq + hq) * HD + idx % HD);
      }
#pragma unroll
      for (int i = 0; i < QB; ++i) {
        const int idx = tid + i * FAST_THREADS;
        if (idx < R * HD) {
          qs[idx] = qv[i];
          acc_s[idx] = 0.f;
        }
      }
    }
    if (tid < R) {
      M.row_m[tid] = -CUDART_INF_F;
      M.row_l[tid] = 0.f;
    }
    const size_t kbase = (((size_t)stream * 2 + 0) * P.Hkv + gk) * (size_t)P.cap * HD;
    const size_t vbase = (((size_t)stream * 2 + 1) * P.Hkv + gk) * (size_t)P.cap * HD;

    for (int kt0 = k0; kt0 < k1; kt0 += KT) {
      const int nk = min(KT, k1 - kt0);
      __syncthreads();
      {
        const uint4* ksrc = reinterpret_cast<const uint4*>(kvl + kbase + (size_t)kt0 * HD);
        const uint4* vsrc = reinterpret_cast<const uint4*>(kvl + vbase + (size_t)kt0 * HD);
        constexpr int CB = KT * (HD / 8) / FAST_THREADS;  // 16-byte chunks per thread of a full tile
        uint4 kq[CB], vq[CB];
#pragma unroll
        for (int i = 0; i < CB; ++i) {
          const int idx = tid + i * FAST_THREADS;
          if (idx < nk * (HD / 8)) {
            kq[i] = __ldcg(ksrc + idx);
            vq[i] = __ldcg(vsrc + idx);
          }
        }
#pragma unroll
        for (int i = 0; i < CB; ++i) {
          const int idx = tid + i * FAST_THREADS;
          if (idx < nk * (HD / 8)) {
            *reinterpret_cast<uint4*>(Ks + (idx / (HD / 8)) * KROW + (idx % (HD / 8)) * 16) = kq[i];
            *reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(Vs) + (size_t)idx * 16) = vq[i];
          }
        }
      }
      __syncthreads();
      // scores of (row, key) pairs; a warp works on 32 consecutive keys of one row
      for (int idx = tid; idx < R * KT; idx += FAST_THREADS) {
        const int r = idx / KT, key = idx % KT;
        float sc = -CUDART_INF_F;
        if (key < nk && kt0 + key <= L + r) {
          const float* q = qs + r * HD;
          const uint8_t* krow = Ks + key * KROW;
          sc = 0.f;
#pragma unroll 2
          for (int ch = 0; ch < HD / 8; ++ch) {
            float kx[8];
            unpack8(*reinterpret_cast<const uint4*>(krow + ch * 16), kx);
            const float4 q0 = *reinterpret_cast<const float4*>(q + ch * 8);
            const float4 q1 = *reinterpret_cast<const float4*>(q + ch * 8 + 4);
            sc = fmaf(kx[0], q0.x, sc); sc = fmaf(kx[1], q0.y, sc);
            sc = fmaf(kx[2], q0.z, sc); sc = fmaf(kx[3], q0.w, sc);
            sc = fmaf(kx[4], q1.x, sc); sc = fmaf(kx[5], q1.y, sc);
            sc = fmaf(kx[6], q1.z, sc); sc = fmaf(kx[7], q1.w, sc);
          }
        }
        ps[idx] = sc;
      }
      __syncthreads();
      // running max / sum per row (one warp per row), scores -> weights in place
      for (int r = warp; r < R; r += FAST_WARPS) {
        float mt = -CUDART_INF_F;
        for (int key = lane; key < nk; key += 32) mt = fmaxf(mt, ps[r * KT + key]);
        mt = warp_max(mt);
        const float m_old = M.row_m[r], m_new = fmaxf(m_old, mt);
        float lt = 0.f;
        for (int key = lane; key < nk; key += 32) {
          const float sc = ps[r * KT + key];
          const float pw = sc == -CUDART_INF_F ? 0.f : expf(sc - m_new);
          ps[r * KT + key] = pw;
          lt += pw;
        }
        lt = warp_sum(lt);
        if (lane == 0) {
          const float corr = m_new == -CUDART_INF_F ? 0.f : expf(m_old - m_new);
          M.row_corr[r] = corr;
          M.row_m[r] = m_new;
          M.row_l[r] = M.row_l[r] * corr + lt;
        }
      }
      __syncthreads();
      // P * V for (row, dim) pairs
      for (int idx = tid; idx < R * HD; idx += FAST_THREADS) {
        const int r = idx / HD, dd = idx % HD;
        float a = acc_s[idx] * M.row_corr[r];
        const float* pr = ps + r * KT;
#pragma unroll 4
        for (int key = 0; key < nk; ++key) a = fmaf(pr[key], __bfloat162float(Vs[key * HD + dd]), a);
        acc_s[idx] = a;
      }
    }
    __syncthreads();
    for (int idx = tid; idx < R * HD; idx += FAST_THREADS) {
      const int r = idx / HD, dd = idx % HD, tok = bi * R + r;
      if (nsplit == 1) {
        P.attn_out[((size_t)tok * Hq + hq) * HD + dd] = acc_s[idx] / M.row_l[r];
      } else {
        float* dst = P.part + (((size_t)tok * Hq + hq) * FAST_NSPLIT_CAP + c) * (HD + 2);
        dst[dd] = acc_s[idx];
        if (dd == 0) {
          dst[HD] = M.row_m[r];
          dst[HD + 1] = M.row_l[r];
        }
      }
    }
    if (nsplit > 1) {
      __threadfence();
      __syncthreads();
      if (tid == 0) {
        int prev = atomicAdd(&P.attn_counters[bi * Hq + hq], 1);
        M.last = prev == nsplit - 1;
        if (M.last) P.attn_counters[bi * Hq + hq] = 0;
      }
      __syncthreads();
      if (M.last) {
        __threadfence();
        for (int idx = tid; idx < R * HD; idx += FAST_THREADS) {
          const int r = idx / HD, dd = idx % HD, tok = bi * R + r;
          const float* src = P.part + ((size_t)tok * Hq + hq) * FAST_NSPLIT_CAP * (HD + 2);
          float m_tot = -CUDART_INF_F, denom = 0.f, o = 0.f;
          constexpr int MB = 8;  // splits loaded together
          for (int sp0 = 0; sp0 < nsplit; sp0 += MB) {
            float ms[MB], ls[MB], os[MB];
#pragma unroll
            for (int i = 0; i < MB; ++i) {
              if (sp0 + i < nsplit) {
                ms[i] = __ldcg(src + (sp0 + i) * (HD + 2) + HD);
                ls[i] = __ldcg(src + (sp0 + i) * (HD + 2) + HD + 1);
                os[i] = __ldcg(src + (sp0 + i) * (HD + 2) + dd);
              }
            }
#pragma unroll
            for (int i = 0; i < MB; ++i) {
              if (sp0 + i < nsplit && ms[i] != -CUDART_INF_F) {  // running merge in split order
                const float m_new = fmaxf(m_tot, ms[i]);
                const float ca = expf(m_tot - m_new), cb = expf(ms[i] - m_new);
                denom = denom * ca + ls[i] * cb;
                o = o * ca + os[i] * cb;
                m_tot = m_new;
              }
            }
          }
          P.attn_out[((size_t)tok * Hq + hq) * HD + dd] = o / denom;
        }
      }
    }
  }
}

// ---- the kernel --------------------------------------------------------------------------------

template <bool T16>
__global__ void __launch_bounds__(FAST_THREADS, 1) fast_forward_kernel(const __grid_constant__ FastParams P) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, cta = blockIdx.x;
  FastMisc& M = *reinterpret_cast<FastMisc*>(smem + P.misc_off);
  uint8_t* uni = smem + P.union_off;
  int n_trace = 0;

  // a launch that failed earlier leaves the barrier words unusable: refuse to run on them
  if (ld_acquire_u32(P.epoch_base + 1) != 0u) {
    if (cta == 0 && tid == 0) atomicOr(P.status, SSD_STATUS_TIMEOUT);
    return;
  }

  // per-CTA tables: tile lists, chunk sizes, rows of this forward
  const size_t wi = (size_t)cta * FAST_WARPS + warp;
  if (tid < FOP_COUNT) M.ucnt[tid] = P.m.unit_cnt[cta * FOP_COUNT + tid];
  for (int i = tid; i < FOP_COUNT * FAST_MAX_UNITS; i += FAST_THREADS) {
    const int op = i / FAST_MAX_UNITS, u = i % FAST_MAX_UNITS;
    const int cnt = P.m.unit_cnt[cta * FOP_COUNT + op];
    M.utile[op][u] = u < cnt ? P.m.unit_tile[P.m.unit_off[cta * FOP_COUNT + op] + u] : 0;
  }
  for (int i = lane; i < FAST_MAX_CHUNKS / 4; i += 32)
    reinterpret_cast<uint32_t*>(M.chunks[warp])[i] =
        reinterpret_cast<const uint32_t*>(P.m.chunks + wi * FAST_MAX_CHUNKS)[i];
  if (tid < P.T) {
    const int bi = tid / P.R, r = tid % P.R;
    M.tok_stream[tid] = P.b0 + bi;
    M.tok_pos[tid] = P.len[P.b0 + bi] + r;
  }

  // this warp's ring: barriers, then the first copies
  Ring ring;
  ring.ring = smem_u32(smem) + warp * P.ring_warp_bytes;
  ring.bars = smem_u32(&M.bars[warp][0]);
  ring.src = P.m.wstream + P.m.stream_off[wi];
  ring.tab = M.chunks[warp];
  ring.ncl = (uint32_t)P.m.chunk_cnt[wi * 2];
  ring.nend = ring.ncl + (P.logits ? (uint32_t)P.m.chunk_cnt[wi * 2 + 1] : 0u);
  ring.layers_left = ring.ncl ? (uint32_t)P.L : 0u;
  ring.pc = 0;
  ring.slot = ring.parity = 0;
  ring.nslot = (uint32_t)P.nslot;
  ring.outstanding = 0;
  ring.dead = false;
  if (lane == 0) {
    for (int s = 0; s < P.nslot; ++s) mbar_init(ring.bars + s * 8, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();  // also orders this warp's chunk table before its first use
  for (int s = 0; s < P.nslot; ++s) ring_request(ring, (uint32_t)s, lane);
  const uint32_t epoch_base = ld_acquire_u32(P.epoch_base);
  uint32_t epoch = 0;
  __syncthreads();
  trace_mark(P, n_trace);

  const int T = P.T, d = P.d, qd = P.Hq * P.hd, half = P.hd >> 1;

  // phase 0: embedding rows and the rotary table of this forward's positions
  if (cta < T) {
    const int tok = cta, r = tok % P.R, stream = M.tok_stream[tok];
    int id = P.row_ids ? P.row_ids[tok]
                       : (r == 0 ? P.pending[stream] : P.draft_tokens[(size_t)stream * (P.R - 1) + r - 1]);
    if (id < 0 || id >= P.vocab_in) {
      if (tid == 0) atomicOr(P.status, SSD_STATUS_BAD_TOKEN);
      id = min(max(id, 0), P.vocab_in - 1);
    }
    const bf16* src = P.embed + (size_t)id * d;
    for (int j = tid; j < d; j += FAST_THREADS)
      P.hfix[(size_t)tok * d + j] = __float2ll_rn(__bfloat162float(src[j]) * FIX_SCALE);
    const double pos = (double)M.tok_pos[tok];
    for (int j = tid; j < half; j += FAST_THREADS) {
      double sn, cs;
      sincos(pos * P.inv_freq[j], &sn, &cs);
      P.rope_cs[((size_t)tok * half + j) * 2 + 0] = (float)cs;
      P.rope_cs[((size_t)tok * half + j) * 2 + 1] = (float)sn;
    }
  }
  trace_mark(P, n_trace);
  bool ok = grid_sync(P, epoch_base + (++epoch) * (uint32_t)P.m.n_cta, false);
  trace_mark(P, n_trace);
  // every CTA has read the base by now: publish the next launch's (this launch arrives 1 + 5 L times)
  if (ok && cta == 0 && tid == 0)
    st_release_u32(P.epoch_base, epoch_base + (uint32_t)(1 + 5 * P.L) * (uint32_t)P.m.n_cta);

  // K slice of the down projection this CTA works on
  const int dsteps = P.F >> 4, dsl = cta % P.m.down_split;
  const int dk0 = (int)(((long long)dsl * dsteps) / P.m.down_split) << 4;
  const int dk1 = (int)(((long long)(dsl + 1) * dsteps) / P.m.down_split) << 4;
  const float qscale = rsqrtf((float)P.hd);

  // 5 phases per layer (QKV, attention, O, gate/up, down), then the LM head
  const int n_phase = 5 * P.L + (P.logits ? 1 : 0);
  int l = 0, ph = 0;
#pragma unroll 1
  for (int it = 0; it < n_phase && ok; ++it) {
    if (it == 5 * P.L) ph = 5;
    if (ph == 1) {
      if (P.hd == 64) attn_phase<64>(P, M, uni, l);
      else if (P.hd == 128) attn_phase<128>(P, M, uni, l);
      else attn_phase<32>(P, M, uni, l);
    } else {
      PhaseDesc D;
      D.layer = l;
      D.gain = nullptr;
      D.kb = 0;
      D.qscale = qscale;
      D.kv_layer = P.kv + (size_t)l * P.kv_layer_elems;
      if (ph == 0) {
        D.op = FOP_QKV; D.epi = EPI_F_QKV; D.in_fix = 1; D.in = P.hfix;
        D.gain = P.m.gains + (size_t)l * 2 * d; D.ld = d; D.kc = d; D.n_rows = qd + 2 * P.Hkv * P.hd;
      } else if (ph == 2) {
        D.op = FOP_O; D.epi = EPI_F_RESID; D.in_fix = 0; D.in = P.attn_out;
        D.ld = qd; D.kc = qd; D.n_rows = d;
      } else if (ph == 3) {
        D.op = FOP_GU; D.epi = EPI_F_SWIGLU; D.in_fix = 1; D.in = P.hfix;
        D.gain = P.m.gains + (size_t)l * 2 * d + d; D.ld = d; D.kc = d; D.n_rows = 2 * P.F;
      } else if (ph == 4) {
        D.op = FOP_DOWN; D.epi = EPI_F_RESID; D.in_fix = 0; D.in = P.act;
        D.ld = P.F; D.kb = dk0; D.kc = dk1 - dk0; D.n_rows = d;
      } else {
        D.op = FOP_HEAD; D.epi = EPI_F_LOGITS; D.in_fix = 1; D.in = P.hfix; D.layer = 0;
        D.gain = P.m.gains + (size_t)P.L * 2 * d; D.ld = d; D.kc = d; D.n_rows = P.V;
      }
      gemm_phase<T16>(P, M, uni, ring, D);
    }
    trace_mark(P, n_trace);
    if (ph < 5) {
      ok = grid_sync(P, epoch_base + (++epoch) * (uint32_t)P.m.n_cta, ring.dead);
      trace_mark(P, n_trace);
      if (++ph == 5) {
        ph = 0;
        ++l;
      }
    } else if (__syncthreads_or(ring.dead ? 1 : 0)) {
      ok = false;
    }
  }
  if (!ok && tid == 0) {
    // a wait ran out here or elsewhere: make the failure sticky
    atomicOr(P.status, SSD_STATUS_TIMEOUT);
    st_release_u32(P.epoch_base + 1, 1u);
  }
  // never leave with bulk copies in flight into this CTA's shared memory
  while (ring.outstanding > 0) {
    const uint32_t bar = ring.bars + ring.slot * 8;
    if (!mbar_try_wait(bar, ring.parity) && !bounded_mbar_wait(bar, ring.parity)) break;
    ring.outstanding--;
    if (++ring.slot == ring.nslot) {
      ring.slot = 0;
      ring.parity ^= 1u;
    }
  }
}

}  // namespace

size_t fast_union_bytes(int stage_k, int hd, int T, int R) {
  const bool t16 = T > 8;
  size_t af = (size_t)(stage_k / 16) * (t16 ? 1024 : 512);
  size_t red = (size_t)FAST_WARPS * FAST_MAXU * 32 * (t16 ? 16 : 8);
  const int KT = 8192 / hd;
  size_t attn = (size_t)R * hd * 4 + (size_t)KT * (hd * 2 + 16) + (size_t)KT * hd * 2 +
                (size_t)R * KT * 4 + (size_t)R * hd * 4;
  size_t u = af + red > attn ? af + red : attn;
  return (u + 127) / 128 * 128;
}

cudaError_t launch_fast_forward(const FastParams& p_in, cudaStream_t st) {
  FastParams p = p_in;
  if (p.T < 1 || p.T > FAST_MAX_T || p.m.n_cta > FAST_MAX_CTAS || p.m.max_units > FAST_MAX_UNITS)
    return cudaErrorInvalidValue;
  const size_t uni = fast_union_bytes(p.m.max_stage_k, p.hd, p.T, p.R);
  const size_t misc = (sizeof(FastMisc) + 127) / 128 * 128;
  const size_t max_smem = 227 * 1024;
  if (uni + misc + (size_t)FAST_WARPS * 2 * FAST_SLOT_BYTES > max_smem) return cudaErrorInvalidValue;
  // A shallow ring on purpose: four 2 KB copies in flight per warp already saturate HBM, and refill
  // traffic in flight beyond that only queues ahead of the phases' latency-critical loads.
  int nslot = (int)((max_smem - uni - misc) / ((size_t)FAST_WARPS * FAST_SLOT_BYTES));
  if (nslot > FAST_RING_SLOTS) nslot = FAST_RING_SLOTS;
  p.nslot = nslot;
  p.ring_warp_bytes = nslot * FAST_SLOT_BYTES;
  p.union_off = FAST_WARPS * p.ring_warp_bytes;
  p.misc_off = p.union_off + (int)uni;
  const size_t smem = (size_t)p.misc_off + misc;
  const bool t16 = p.T > 8;
  const void* kern = t16 ? (const void*)fast_forward_kernel<true> : (const void*)fast_forward_kernel<false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  void* args[] = {(void*)&p};
  e = cudaLaunchCooperativeKernel(kern, dim3(p.m.n_cta), dim3(FAST_THREADS), args, smem, st);
  if (e != cudaSuccess) return e;
  count_launch();
  return cudaGetLastError();
}

}  // namespace ssd
