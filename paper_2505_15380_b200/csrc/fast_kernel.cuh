// Persistent small-batch verify forward (Eq. 4: one causal-decoder pass over the pending token and
// the gamma draft tokens of each stream against the cached prefix), T = B * (gamma + 1) <= 16 rows.
//
// One CTA per SM lives for the whole forward.  Every warp streams its own pre-packed slice of the
// weights from HBM through a private shared-memory ring with bulk async copies that complete on
// mbarriers; a slot is refilled the moment its chunk has been consumed, whatever phase the consumer
// is in, so the weight stream runs ahead of the dependency chain across phase boundaries.  The
// ring is kept shallow on purpose: a few KB in flight per warp already saturate HBM (measured).
// The phases of a layer (QKV projection, attention + O projection, gate/up, down) are separated by
// grid barriers on one monotonic arrival counter, with bounded waits.
//
// The forward is a chain of 4 dependent phases per layer, each far shorter than a microsecond of
// memory time, so what bounds it is latency: the instructions a warp executes per phase (eight
// warps per SM hide little) and the round trips through L2 between phases.  Hence: every activation
// is converted to the tensor-core operand layout (bf16 hi + lo) once, by the thread that produces
// it, and consumers fetch their slice with one bulk copy; the weight stream is pre-cut into chunks
// of whole k-steps so the inner loop is straight-line for each tile count; everything rare is out
// of line; attention keeps its weights in registers between its two contractions; projections
// that are split over K across CTAs (O by query head, down by column range) add into a
// fixed-point residual stream whose words carry an arrival count, so the thread that completes
// an element finishes it without a further exchange.
//
// Projections: D[token, weight row] = sum_k X[token, k] * W[row, k] on mma.m16n8k16 (bf16 inputs,
// fp32 accumulate): the 16-row A operand holds the tokens, the B operand one packed tile of 8 weight
// rows.  Activations are fp32 and enter the instruction as a two-term bf16 split (hi + lo), so the
// products are exact to ~2^-17 relative; weights are exactly their stored bf16 values.  With at
// most 8 rows both terms ride in one instruction (rows 0..7 hi, rows 8..15 lo).  The warps of a
// CTA split K; their partial sums are added in a fixed order in shared memory.
//
// This header holds the kernel template; fast_verify_*.cu instantiate its variants (rows <= 8 or
// <= 16, split or plain activations, with or without the phase trace), one pair per translation
// unit so that they compile side by side, and fast_verify.cu holds the launcher.
#pragma once
#include <math_constants.h>

#include "fast.h"
#include "kernels.h"

namespace ssd {

namespace {

constexpr unsigned long long FAST_WAIT_CYCLES = 3000000000ull;  // ~1.5 s at 2 GHz
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
// The same copy with an L2 eviction priority.  The weight stream is read once per forward and is
// six times the size of L2: marked evict-first it stops pushing out what the phases re-read (the
// operands between phases, the prefetched keys and values, the per-layer constants).
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
__device__ __forceinline__ uint32_t pack_bf16(float x, float y) {
  __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  return *reinterpret_cast<uint32_t*>(&h);
}
// Residual-stream word (2^-32 fixed point) -> fp32, through its two 32-bit halves.
__device__ __forceinline__ float fix_to_float(long long v) {
  const int hi = (int)(v >> 32);
  const unsigned lo = (unsigned)v;
  return fmaf(__uint2float_rn(lo), FIX_INV_SCALE, __int2float_rn(hi));
}

// Where each layer's part of a warp's stream starts: base + (source layer) * layer_bytes.  A model
// that inherits layers of another (a draft made of some of the target's layers) walks the same
// stream in the order of its layer map, so the source pointer jumps at layer boundaries.  Touched
// once per layer only, hence kept in shared memory (behind the warp's chunk table), not in the
// ring's registers.
struct RingSide {
  const uint8_t* base;
  const int32_t* map;   // layer -> source layer, or null: identity
  uint32_t layer_bytes;
  uint32_t cur, n_src;  // layer being requested; layers in the packed stream (the head follows them)
};

// Per-CTA bookkeeping in shared memory.
struct FastMisc {
  unsigned long long bars[FAST_WARPS][FAST_MAX_SLOTS];
  unsigned long long sbar[FAST_WARPS];          // per warp: arrival of its slice of the A operand
  // chunk sizes (tiles) of each warp's stream, followed by the warp's RingSide record
  alignas(8) uint8_t chunks[FAST_WARPS][FAST_MAX_CHUNKS + sizeof(RingSide)];
  int32_t ucnt[FOP_COUNT];
  int32_t utile[FOP_COUNT][FAST_MAX_UNITS];
  float inv_rms[FAST_MAX_T];
  float row_m[FAST_MAX_T], row_l[FAST_MAX_T], row_corr[FAST_MAX_T];
  float wred[FAST_WARPS][FAST_MAX_T];
  int32_t tok_stream[FAST_MAX_T];  // stream of each row of this forward
  int32_t tok_pos[FAST_MAX_T];     // its position len + r
};

__device__ __forceinline__ void prefetch_l2(const void* p) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

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
  bool mapped;              // the model walks another model's stream by a layer map (see RingSide)
  uint64_t policy;          // L2 eviction priority of the stream's copies, made once (making it
                            // anew for every copy cost 11 us per forward)
};

// A mapped stream (a model that inherits layers of another) at a layer boundary: where the next
// layer's chunks start.  Out of line: once per layer and warp, and only for such models.
__device__ __noinline__ const uint8_t* ring_boundary_src(const uint8_t* tab, bool more_layers) {
  RingSide* sd = reinterpret_cast<RingSide*>(const_cast<uint8_t*>(tab) + FAST_MAX_CHUNKS);
  uint32_t next = sd->n_src;  // the head's chunks follow the last source layer
  if (more_layers) {
    const uint32_t cur = sd->cur + 1;
    next = (uint32_t)sd->map[cur];
    __syncwarp();
    sd->cur = cur;            // every lane writes the same value
    __syncwarp();
  }
  return sd->base + (size_t)next * sd->layer_bytes;
}
// Tiles of the next chunk to request (0: the stream is exhausted); `boundary`: it was the last
// chunk of a layer.
__device__ __forceinline__ uint32_t ring_next_chunk(Ring& r, bool& boundary) {
  boundary = false;
  if (r.pc >= r.nend) return 0u;
  const uint32_t n = r.tab[r.pc];
  ++r.pc;
  if (r.layers_left > 0 && r.pc == r.ncl) {
    if (--r.layers_left > 0) r.pc = 0;  // next layer: same chunk sizes; else fall through to the head
    boundary = true;
  }
  return n;
}
__device__ __forceinline__ void ring_request(Ring& r, uint32_t slot, int lane) {
  bool boundary;
  const uint32_t n = ring_next_chunk(r, boundary);
  if (n) {
    if (lane == 0) {
      const uint32_t bar = r.bars + slot * 8;
      mbar_expect_tx(bar, n * FAST_TILE_BYTES);
      bulk_g2s_hint(r.ring + slot * FAST_SLOT_BYTES, r.src, n * FAST_TILE_BYTES, bar, r.policy);
    }
    r.src += n * FAST_TILE_BYTES;
    if (boundary && r.mapped) r.src = ring_boundary_src(r.tab, r.layers_left > 0);
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

template <bool TRACE>
__device__ __forceinline__ void trace_mark(const FastParams& P, int& n_trace) {
  if (TRACE && threadIdx.x == 0 && n_trace < P.trace_cap)
    P.trace[(size_t)blockIdx.x * P.trace_cap + n_trace++] = clock64();
}

// Grid-wide barrier on one monotonic arrival counter: it is complete when the counter has
// reached `target`.  One thread per CTA arrives (release reduction) and polls (acquire loads).
// A CTA whose wait ran out raises the failure word next to the base; every poller looks at that
// word now and then, so all CTAs give up together.  Returns false in that case.
__device__ __forceinline__ bool grid_sync(const FastParams& P, uint32_t target, bool failed) {
  const int bad_in = __syncthreads_or(failed ? 1 : 0);
  bool ok = bad_in == 0;
  if (threadIdx.x == 0) {
    if (bad_in) st_release_u32(P.epoch_base + 1, 1u);
    // one release reduction: orders the CTA's stores (made visible to this thread by the CTA
    // barrier above) before the arrival, without a separate fence (17 us per forward less)
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(P.flags) : "memory");
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
  const uint32_t* xin;  // operand-layout input, at this CTA's first k-step
  const long long* ssq_in;  // with in_fix: the sums of squares of the input rows
  int op;               // FOP_*: whose tiles of this CTA
  int epi;              // EPI_F_*
  int in_fix;           // the input is x * gain of an RMS norm: scale the outputs by inv_rms[row]
  int kc;               // input columns this CTA covers
  int n_rows;           // valid weight rows (the last tile of the LM head is padded)
  int layer;
  bf16* kv_layer;       // this layer's slice of the cache (QKV epilogue)
  float qscale;         // 1 / sqrt(head_dim)
  // residual epilogues: the operand the finished rows become for the next projection
  uint32_t* xout;
  long long* ssq_out;
  const float* gain_next;
  int cinc;             // this CTA's increment of an element's arrival count (see resid_tile)
};

// Operand layout of the activations (the A operand of the projections), in global memory where a
// producer writes it and in shared memory where the consumers copy it: for k-step s and lane l
// (g = l / 4, t = l % 4) 16 bytes
//   { hi(x[g][16s+2t..]), hi(x[g][16s+8+2t..]), lo(same), lo(same) }
// (hi = bf16 leading part, lo = bf16 of the remainder) and, when more than 8 rows are in flight,
// 16 more bytes for row g + 8.  Every value is converted once, by the thread that produces it,
// instead of once per consuming CTA.
template <bool T16, bool LO>
struct Lay {
  static constexpr int WH = LO ? 4 : 2;          // words per (k-step, lane, row half)
  static constexpr int W = WH * (T16 ? 2 : 1);   // words per (k-step, lane)
  static constexpr int STEP = 32 * W * 4;        // bytes per k-step
  // With at most 8 rows in flight the 16-row A operand has room for both parts of a split
  // activation: rows 0..7 carry the bf16 leading parts, rows 8..15 the remainders of the same
  // rows, so one instruction multiplies both and the two halves of the result are added at the end.
  static constexpr bool MERGE = LO && !T16;
};
template <bool T16, bool LO>
__device__ __forceinline__ uint32_t afrag_word(int row, int kk) {  // kk = column pair index
  const int s = kk >> 3, t = kk & 3, which = (kk >> 2) & 1;
  return (uint32_t)(((s * 32 + (row & 7) * 4 + t) * Lay<T16, LO>::W) + (row >> 3) * Lay<T16, LO>::WH + which);
}
// One row half of this lane's share of a k-step of an operand in shared memory -> registers of
// the A fragment (h = 0: rows g, registers 0 and 2; h = 1: rows g + 8, registers 1 and 3).
template <bool LO>
__device__ __forceinline__ void load_afrag(uint32_t addr, int h, uint32_t (&ahi)[4], uint32_t (&alo)[4]) {
  if (LO) {
    const uint4 a = lds_v4(addr);
    ahi[h] = a.x; ahi[2 + h] = a.y; alo[h] = a.z; alo[2 + h] = a.w;
  } else {
    const uint2 a = lds_v2(addr);
    ahi[h] = a.x; ahi[2 + h] = a.y;
  }
}
// Columns (k, k + 1), k even, of row `row`.
template <bool T16, bool LO>
__device__ __forceinline__ void write_frag_pair(uint32_t* buf, int row, int k, float x0, float x1) {
  const uint32_t wd = afrag_word<T16, LO>(row, k >> 1);
  if (LO) {
    uint32_t hi, lo;
    split2(x0, x1, hi, lo);
    buf[wd] = hi;
    buf[wd + 2] = lo;
  } else {
    buf[wd] = pack_bf16(x0, x1);
  }
}
// One column of row `row` (two 2-byte stores).
template <bool T16, bool LO>
__device__ __forceinline__ void write_frag_elem(uint32_t* buf, int row, int k, float x) {
  const bf16 h = __float2bfloat16_rn(x);
  bf16* w = reinterpret_cast<bf16*>(buf + afrag_word<T16, LO>(row, k >> 1)) + (k & 1);
  w[0] = h;
  if (LO) w[4] = __float2bfloat16_rn(x - __bfloat162float(h));  // two words on
}

// inv_rms[t] = rsqrt(mean(x[t]^2) + eps) from the sums of squares the producers left, one 64-bit
// fixed-point word (2^-32) per 64 columns and row; one warp per row.  The loads are issued at the
// start of the phase and summed after the tensor-core work, so their latency stays off the
// critical path.
constexpr int SSQ_COLS = 64;  // columns per word
struct SsqLoads {
  long long v[2];  // rows warp and warp + FAST_WARPS: word `lane`
};
__device__ __forceinline__ void ssq_issue(SsqLoads& q, const long long* __restrict__ ssq, int nwords, int T) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int row = warp + h * FAST_WARPS;
    q.v[h] = 0;
    if (row < T && lane < nwords) q.v[h] = __ldcg(ssq + lane * FAST_MAX_T + row);
  }
}
__device__ __forceinline__ void ssq_finish(const SsqLoads& q, const long long* __restrict__ ssq, int nwords, int T,
                                           int K, float eps, FastMisc& M) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int row = warp + h * FAST_WARPS;
    if (row < T) {  // uniform per warp
      long long v = q.v[h];
      for (int wd = lane + 32; wd < nwords; wd += 32) v += __ldcg(ssq + wd * FAST_MAX_T + row);
      // the words are exact (integer sums), so a fixed shuffle tree over their fp32 values gives
      // the same result in every run; half the instructions of a 64-bit tree
      float f = fix_to_float(v);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) f += __shfl_xor_sync(0xffffffffu, f, o);
      if (lane == 0) M.inv_rms[row] = rsqrtf(f / (float)K + eps);
    }
  }
}

// The constants the QKV epilogue needs for one output pair of token `tok`: the biases of packed
// rows n, n + 1 and the rotation (cos, sin) of the token's position.  The threads that run the
// first pass of the epilogue load theirs at the start of the phase, off the critical path.
struct QkvConsts {
  float2 bias, cs;
};
__device__ __forceinline__ QkvConsts qkv_consts(const FastParams& P, const PhaseDesc& D, int tok, int n) {
  const int hd = P.hd, hs = P.hd_shift, qd = P.Hq << hs, kvd = P.Hkv << hs;
  QkvConsts q;
  q.bias = *reinterpret_cast<const float2*>(P.m.bias_qkv + (size_t)D.layer * (qd + 2 * kvd) + n);
  q.cs = make_float2(1.f, 0.f);
  if (n < qd + kvd)
    q.cs = __ldcg(reinterpret_cast<const float2*>(P.rope_cs + ((size_t)tok * (hd >> 1) + ((n & (hd - 1)) >> 1)) * 2));
  return q;
}

// One output element pair of a projection: token `tok`, packed weight rows n and n + 1.
template <bool T16, bool LO>
__device__ __forceinline__ void epilogue_pair(const FastParams& P, const PhaseDesc& D, const FastMisc& M,
                                              int tok, int n, float c0, float c1, const QkvConsts& qc) {
  if (D.epi == EPI_F_SWIGLU) {
    write_frag_elem<T16, LO>(P.xd, tok, n >> 1, __fdividef(c0, 1.f + __expf(-c0)) * c1);
  } else if (D.epi == EPI_F_LOGITS) {
    if (n < D.n_rows) P.logits[(size_t)tok * P.V + n] = c0;
    if (n + 1 < D.n_rows) P.logits[(size_t)tok * P.V + n + 1] = c1;
  } else {  // EPI_F_QKV: bias, rotary embedding, q scaling, K/V append
    const int hd = P.hd, hs = P.hd_shift, half = hd >> 1, qd = P.Hq << hs, kvd = P.Hkv << hs;
    const float x1 = c0 + qc.bias.x, x2 = c1 + qc.bias.y;
    const int stream = M.tok_stream[tok], pos = M.tok_pos[tok];
    if (n < qd + kvd) {
      const int j = (n & (hd - 1)) >> 1;
      const float2 cs = qc.cs;
      const float o1 = x1 * cs.x - x2 * cs.y, o2 = x2 * cs.x + x1 * cs.y;
      if (n < qd) {
        const int col = (n & ~(hd - 1)) + j;  // q, pre-scaled, as the operand of the score contraction
        write_frag_elem<T16, LO>(P.xq, tok, col, o1 * D.qscale);
        write_frag_elem<T16, LO>(P.xq, tok, col + half, o2 * D.qscale);
      } else if (pos >= 0 && pos < P.cap) {
        const int gk = (n - qd) >> hs;
        bf16* kdst = D.kv_layer + (((size_t)stream * 2 + 0) * P.Hkv + gk) * (size_t)P.cap * hd + (size_t)pos * hd;
        kdst[j] = __float2bfloat16_rn(o1);
        kdst[j + half] = __float2bfloat16_rn(o2);
      } else {
        atomicOr(P.status, SSD_STATUS_KV_OVERFLOW);
      }
    } else if (pos >= 0 && pos < P.cap) {
      const int nn = n - qd - kvd, gk = nn >> hs, jj = nn & (hd - 1);
      bf16* vdst = D.kv_layer + (((size_t)stream * 2 + 1) * P.Hkv + gk) * (size_t)P.cap * hd + (size_t)pos * hd;
      *reinterpret_cast<__nv_bfloat162*>(vdst + jj) = __floats2bfloat162_rn(x1, x2);
    }
  }
}

// Residual epilogue of one output tile (8 columns of h), per lane = (row g, column pair t): the
// projection outputs are added to the residual stream with 64-bit integer atomics.  A word holds
// the value in 2^-32 fixed point above a 4-bit arrival count: integer adds commute, so the K
// slices of different CTAs may arrive in any order and the sum is still bit-reproducible, and the
// count tells the thread whose add completes an element that it holds the finished value (the
// slices' count increments are +1, and 1 - nsplit for slice 0: they sum to zero, and no partial
// sum is a multiple of 16).  That thread turns the element into the operand of the next
// projection (x * gain as bf16 hi / lo in operand layout) and adds x^2 to the row's sums of
// squares for the RMS norm, in fixed point as well.
template <bool T16, bool LO>
struct ResidAdds {
  long long inc[T16 ? 2 : 1][2], old[T16 ? 2 : 1][2];
  float2 gn;
};
template <bool T16, bool LO>
__device__ __forceinline__ void resid_issue(const FastParams& P, const PhaseDesc& D, int tile, int lane,
                                            const float* c, ResidAdds<T16, LO>& A, const float2* gn_ready = nullptr) {
  constexpr int NH = T16 ? 2 : 1;
  const int gg = lane >> 2, tt = lane & 3, n = tile * 8 + 2 * tt, T = P.T;
  // the gains of the next norm for these two columns: a cold load, taken at the start of the
  // phase where the caller could
  A.gn = gn_ready ? *gn_ready : __ldg(reinterpret_cast<const float2*>(D.gain_next + n));
#pragma unroll
  for (int h = 0; h < NH; ++h) {
    if (gg + 8 * h < T) {
      unsigned long long* hp = reinterpret_cast<unsigned long long*>(P.hfix + (size_t)(gg + 8 * h) * P.d + n);
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        A.inc[h][j] = __float2ll_rn(c[2 * h + j] * FIX_SCALE) * 16 + D.cinc;
        A.old[h][j] = (long long)atomicAdd(hp + j, (unsigned long long)A.inc[h][j]);
      }
    }
  }
}
template <bool T16, bool LO>
__device__ __forceinline__ void resid_finish(const FastParams& P, const PhaseDesc& D, int tile, int lane,
                                             const ResidAdds<T16, LO>& A) {
  constexpr int NH = T16 ? 2 : 1;
  const int gg = lane >> 2, tt = lane & 3, n = tile * 8 + 2 * tt, T = P.T;
#pragma unroll
  for (int h = 0; h < NH; ++h) {
    const int row = gg + 8 * h;
    if (row < T) {
      long long sq = 0;
      bool any = false;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const long long now = A.old[h][j] + A.inc[h][j];
        if ((now & 15) == 0) {  // this add completed the element
          const float x = fix_to_float(now >> 4);
          write_frag_elem<T16, LO>(D.xout, row, n + j, x * (j ? A.gn.y : A.gn.x));
          sq += __float2ll_rn(x * x * FIX_SCALE);
          any = true;
        }
      }
      if (any)
        atomicAdd(reinterpret_cast<unsigned long long*>(D.ssq_out + (n / SSQ_COLS) * FAST_MAX_T + row),
                  (unsigned long long)sq);
    }
  }
}
template <bool T16, bool LO>
__device__ __forceinline__ void resid_tile(const FastParams& P, const PhaseDesc& D, int tile, int lane,
                                           const float* c, const float2* gn_ready = nullptr) {
  ResidAdds<T16, LO> A;
  resid_issue<T16, LO>(P, D, tile, lane, c, A, gn_ready);
  resid_finish<T16, LO>(P, D, tile, lane, A);
}

// The tensor-core work of one round of CNT tiles over this warp's k-steps [s0, s1): straight-line
// per chunk (one ring slot = SPC whole k-steps), partial sums to shared memory at the end.
template <int CNT, bool T16, bool LO>
__device__ __forceinline__ void mma_round(Ring& r, int lane, uint32_t af_lane, int s0, int s1, bool row0,
                                          bool row1, float* red_dst) {
  constexpr int SPC = FAST_SLOT_TILES / CNT;
  constexpr uint32_t STEP = Lay<T16, LO>::STEP;
  constexpr int NACC = T16 ? 4 : 2;
  constexpr bool MERGE = Lay<T16, LO>::MERGE;
  constexpr bool TWO = LO && !MERGE && CNT <= 4;  // few tiles: the hi and lo terms in separate accumulators
  float acc[CNT][4], acl[TWO ? CNT : 1][4];
#pragma unroll
  for (int u = 0; u < CNT; ++u) acc[u][0] = acc[u][1] = acc[u][2] = acc[u][3] = 0.f;
#pragma unroll
  for (int u = 0; u < (TWO ? CNT : 1); ++u) acl[u][0] = acl[u][1] = acl[u][2] = acl[u][3] = 0.f;
#pragma unroll 1
  for (int s = s0; s < s1; s += SPC) {
    ring_acquire(r);
    const uint32_t wb = r.ring + r.slot * FAST_SLOT_BYTES + lane * 8;
#pragma unroll
    for (int i = 0; i < SPC; ++i) {
      if (SPC > 1 && s + i >= s1) break;  // the last chunk of the slice may hold fewer k-steps
      {
        uint32_t ahi[4] = {0u, 0u, 0u, 0u}, alo[4] = {0u, 0u, 0u, 0u};
        if (row0) load_afrag<LO>(af_lane + (uint32_t)(s + i) * STEP, 0, ahi, alo);
        if (T16 && row1) load_afrag<LO>(af_lane + (uint32_t)(s + i) * STEP + Lay<T16, LO>::WH * 4, 1, ahi, alo);
        uint2 b[CNT];
#pragma unroll
        for (int u = 0; u < CNT; ++u) b[u] = lds_v2(wb + (uint32_t)(i * CNT + u) * FAST_TILE_BYTES);
        if (MERGE) {
          ahi[1] = alo[0];
          ahi[3] = alo[2];
        }
#pragma unroll
        for (int u = 0; u < CNT; ++u) mma_bf16(acc[u], ahi, b[u].x, b[u].y);
        if (LO && !MERGE) {
#pragma unroll
          for (int u = 0; u < CNT; ++u) mma_bf16(TWO ? acl[u] : acc[u], alo, b[u].x, b[u].y);
        }
      }
    }
    ring_release(r, lane);
  }
  if (TWO) {
#pragma unroll
    for (int u = 0; u < CNT; ++u) {
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[u][i] += acl[u][i];
    }
  }
#pragma unroll
  for (int u = 0; u < CNT; ++u) {
    float* dst = red_dst + (size_t)u * 32 * NACC;
    if (MERGE) {
      acc[u][0] += acc[u][2];
      acc[u][1] += acc[u][3];
    }
    *reinterpret_cast<float2*>(dst) = make_float2(acc[u][0], acc[u][1]);
    if (T16) *reinterpret_cast<float2*>(dst + 2) = make_float2(acc[u][2], acc[u][3]);
  }
}

// One projection phase: copy the input operand to shared memory, run this CTA's tiles (the warps
// split K), add the warps' partial sums in shared memory and apply the epilogue.
template <bool T16, bool LO>
__device__ __forceinline__ void gemm_phase(const FastParams& P, FastMisc& M, uint8_t* uni, Ring& ring,
                                           const PhaseDesc& D, uint32_t& stage_parity) {
  constexpr int NACC = T16 ? 4 : 2;
  const int cnt_total = M.ucnt[D.op];
  if (cnt_total == 0) return;
  const int T = P.T, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2;
  const int KS = D.kc >> 4;
  uint32_t* af = reinterpret_cast<uint32_t*>(uni);                             // A operand, KS steps
  float* red = reinterpret_cast<float*>(uni + (size_t)KS * Lay<T16, LO>::STEP);  // [warp][MAXU][32][NACC]
  const int s0 = fast_warp_k0(warp, KS), s1 = fast_warp_k1(warp, KS);
  SsqLoads ssq;
  if (D.in_fix) ssq_issue(ssq, D.ssq_in, (P.d + SSQ_COLS - 1) / SSQ_COLS, T);
  const bool row0 = g < T, row1 = T16 && g + 8 < T;
  QkvConsts qc0, qc1;  // of this thread's outputs in the first pass of the first round's epilogue
  qc0.bias = qc0.cs = qc1.bias = qc1.cs = make_float2(0.f, 0.f);
  if (D.epi == EPI_F_QKV && tid < min(FAST_MAXU, cnt_total) * 32) {
    const int n = M.utile[D.op][warp] * 8 + 2 * (lane & 3);
    if (row0) qc0 = qkv_consts(P, D, g, n);
    if (row1) qc1 = qkv_consts(P, D, g + 8, n);
  }
  float2 gn0 = make_float2(0.f, 0.f);  // residual epilogue, first pass: this thread's two gains
  if (D.epi == EPI_F_RESID && tid < min(FAST_MAXU, cnt_total) * 32)
    gn0 = __ldg(reinterpret_cast<const float2*>(D.gain_next + M.utile[D.op][warp] * 8 + 2 * (lane & 3)));
  // this warp's k-steps of the operand: one bulk copy from L2 (the producers' stores were made
  // visible by the grid barrier; the proxy fence orders that observation before the async read)
  const uint32_t sbar = smem_u32(&M.sbar[warp]);
  const uint32_t stage_bytes = (uint32_t)(s1 - s0) * Lay<T16, LO>::STEP;
  if (stage_bytes && lane == 0) {
    asm volatile("fence.proxy.async.global;" ::: "memory");  // global space only: the full form cost 40 us per forward
    mbar_expect_tx(sbar, stage_bytes);
    bulk_g2s(smem_u32(af) + (uint32_t)s0 * Lay<T16, LO>::STEP,
             reinterpret_cast<const uint8_t*>(D.xin) + (size_t)s0 * Lay<T16, LO>::STEP, stage_bytes, sbar);
  }
  if (stage_bytes) {
    if (!mbar_try_wait(sbar, stage_parity) && !bounded_mbar_wait(sbar, stage_parity)) ring.dead = true;
    stage_parity ^= 1u;
  }
  const uint32_t af_lane = smem_u32(af) + lane * (Lay<T16, LO>::W * 4);
  float* red_dst = red + ((size_t)warp * FAST_MAXU * 32 + lane) * NACC;

  for (int u0 = 0; u0 < cnt_total; u0 += FAST_MAXU) {
    const int cnt = min(FAST_MAXU, cnt_total - u0);
    switch (cnt) {
      case 1: mma_round<1, T16, LO>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      case 2: mma_round<2, T16, LO>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      case 3: mma_round<3, T16, LO>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      case 4: mma_round<4, T16, LO>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      case 5: mma_round<5, T16, LO>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      case 6: mma_round<6, T16, LO>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      case 7: mma_round<7, T16, LO>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      case 8: mma_round<8, T16, LO>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      case 9: mma_round<9, T16, LO>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
      default: mma_round<10, T16, LO>(ring, lane, af_lane, s0, s1, row0, row1, red_dst); break;
    }
    if (D.in_fix && u0 == 0) ssq_finish(ssq, D.ssq_in, (P.d + SSQ_COLS - 1) / SSQ_COLS, T, D.kc, P.eps, M);
    __syncthreads();
    for (int idx = tid; idx < cnt * 32; idx += FAST_THREADS) {  // whole warps: one tile per warp pass
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
      const int tile = M.utile[D.op][u0 + u];
      const bool first = u0 == 0 && idx == tid;  // the pass whose constants were loaded ahead
      if (D.epi == EPI_F_RESID) {
        resid_tile<T16, LO>(P, D, tile, l, c, first ? &gn0 : nullptr);
      } else {
        const int n = tile * 8 + 2 * tt;
        if (gg < T) {
          const float inv = D.in_fix ? M.inv_rms[gg] : 1.f;
          QkvConsts qc = qc0;
          if (D.epi == EPI_F_QKV && !first) qc = qkv_consts(P, D, gg, n);
          epilogue_pair<T16, LO>(P, D, M, gg, n, c[0] * inv, c[1] * inv, qc);
        }
        if (T16 && gg + 8 < T) {
          const float inv = D.in_fix ? M.inv_rms[gg + 8] : 1.f;
          QkvConsts qc = qc1;
          if (D.epi == EPI_F_QKV && !first) qc = qkv_consts(P, D, gg + 8, n);
          epilogue_pair<T16, LO>(P, D, M, gg + 8, n, c[NACC - 2] * inv, c[NACC - 1] * inv, qc);
        }
      }
    }
    if (u0 + FAST_MAXU < cnt_total) __syncthreads();
  }
}

// ---- attention ---------------------------------------------------------------------------------

__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t addr, uint32_t& r0, uint32_t& r1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}

// Attention and O projection, one phase.  The K of the O projection is split over the CTAs by
// groups of query heads (the slices of FOP_O), so a CTA needs the attention output of its own
// heads only: every CTA of a slice computes that attention itself (the same work in each of
// them), keeps the result in shared memory as the A operand, multiplies it with its tiles of W_o
// and adds the products to the residual stream.  No exchange between attention and projection.
//
// Attention of one (stream, head): every warp works through its own 16-key tiles from start to
// end (keys 16 w, 16 w + 128, ..): it stages the tile's keys / values (bf16, as cached) in its
// private part of shared memory, computes the scores S[row, key] = q[row, :] . K[key, :] on the
// tensor cores (q arrives pre-split in operand layout from the QKV epilogue), keeps a running max /
// sum per row in registers, and accumulates O[row, :] += P[row, key] V[key, :] with P taken
// straight from the score registers (split into bf16 hi + lo) and V read with a transposing
// matrix load.  One CTA barrier later the eight warps' partials are combined.  Row r of a stream
// sees keys 0..len + r: causal inside the draft block.  The operand rows are the forward's rows
// (all streams); rows of other streams are masked out.
//
// O projection: the warps split the CTA's tiles (tile u: warp u % 8), two tiles at a time so that
// the residual adds of both are in flight together.
//
// KSPLIT (long prefixes): the CTAs of a slice do not repeat each other's work; CTA j of the J that
// share the slice walks every J-th 128-key pass only, leaves its un-normalised partial (max, sum,
// output) in global memory, and the J of them meet on the slice's own arrival counter - a wait of
// about ten CTAs on one word, not a grid barrier - before each merges all J partials in a fixed
// order.  Costs one more exchange through L2 per layer, saves (J - 1) / J of the key walk.
template <int HD, bool T16, bool LO, bool KSPLIT>
__device__ __forceinline__ void attn_o_phase(const FastParams& P, FastMisc& M, uint8_t* uni, Ring& ring,
                                             const PhaseDesc& D, int layer, uint32_t ks_base) {
  constexpr int ROWB = HD * 2 + 16;       // padded K / V row in bytes (conflict-free fragment loads)
  constexpr int NH = T16 ? 2 : 1;         // row halves: rows g and g + 8
  constexpr int W = Lay<T16, LO>::W;      // words per (k-step, lane) of an operand
  constexpr int WH = Lay<T16, LO>::WH;
  constexpr bool MERGE = Lay<T16, LO>::MERGE;
  constexpr int KSTEPS = HD / 16;
  constexpr int DT = HD / 8;              // 8-dim tiles of the output
  constexpr int CH = HD / 8;              // 16-byte chunks per row
  constexpr int LPL = 16 * CH / 32;       // 16-byte loads per lane for 16 rows
  constexpr int NROW = 8 * NH;            // rows held
  const int cnt = M.ucnt[FOP_O];
  if (cnt == 0 && !KSPLIT) return;  // key split: a CTA without tiles of W_o still takes its share of the keys
  const int R = P.R, nb = P.nb, Hq = P.Hq, G = Hq / P.Hkv, T = P.T;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int hps = Hq / P.m.o_split, slice = (int)blockIdx.x % P.m.o_split, KS = hps * KSTEPS;
  // key split: this CTA's rank among the J CTAs of its slice
  const int jr = KSPLIT ? (int)blockIdx.x / P.m.o_split : 0;
  const int J = KSPLIT ? (P.m.n_cta - slice + P.m.o_split - 1) / P.m.o_split : 1;
  const int key_step = 16 * FAST_WARPS * J;
  float* my_part = KSPLIT ? P.attn_part + (size_t)blockIdx.x * hps * FAST_MAX_T * (HD + 2) : nullptr;

  uint32_t* qsm = reinterpret_cast<uint32_t*>(uni);                       // q operand, KSTEPS steps
  uint8_t* kv_w = uni + KSTEPS * 32 * W * 4 + warp * (2 * 16 * ROWB);     // this warp's K then V tile
  float* cm = reinterpret_cast<float*>(uni + KSTEPS * 32 * W * 4 + FAST_WARPS * 2 * 16 * ROWB);  // [warp][NROW]
  float* cl = cm + FAST_WARPS * NROW;
  uint32_t* osm = reinterpret_cast<uint32_t*>(cl + FAST_WARPS * NROW);     // attention output, KS steps
  // a warp's partial output [NROW][HD] takes the place of its K / V tiles once its keys are done
  static_assert(NROW * HD * 4 <= 2 * 16 * ROWB, "partial output must fit the warp's staging area");
  constexpr int CO_W = 2 * 16 * ROWB / 4;                                  // floats between warps' partials
  float* co = reinterpret_cast<float*>(uni + KSTEPS * 32 * W * 4);
  const uint32_t q_lane = smem_u32(qsm) + lane * (W * 4);
  const uint32_t k_lane = smem_u32(kv_w) + g * ROWB + t * 4;
  const uint32_t v_lane = smem_u32(kv_w) + 16 * ROWB + (lane & 15) * ROWB;
  const bf16* kvl = P.kv + (size_t)layer * P.kv_layer_elems;

  for (int item = 0; item < hps * nb; ++item) {
    const int hl = item / nb, bi = item % nb, hq = slice * hps + hl;
    const int stream = P.b0 + bi, gk = hq / G, t_lo = bi * R, t_hi = t_lo + R;
    const int L = M.tok_pos[t_lo], k1 = min(L + R, P.cap);
    const uint4* kg = reinterpret_cast<const uint4*>(kvl + (((size_t)stream * 2 + 0) * P.Hkv + gk) * (size_t)P.cap * HD);
    const uint4* vg = reinterpret_cast<const uint4*>(kvl + (((size_t)stream * 2 + 1) * P.Hkv + gk) * (size_t)P.cap * HD);

    // first tile of this warp: loads in flight before anything else
    int key0 = 16 * warp + 16 * FAST_WARPS * jr;
    uint4 kq[LPL], vq[LPL];
#pragma unroll
    for (int i = 0; i < LPL; ++i) {
      const int idx = lane + 32 * i, key = key0 + idx / CH;
      kq[i] = vq[i] = make_uint4(0u, 0u, 0u, 0u);
      if (key < k1) {
        kq[i] = __ldcg(kg + (size_t)key * CH + idx % CH);
        vq[i] = __ldcg(vg + (size_t)key * CH + idx % CH);
      }
    }
    if (item > 0) __syncthreads();  // the previous item is done with the shared memory (the first
                                    // item starts right behind a grid barrier)
    {                 // q of this head (operand layout, bf16 hi / lo as the QKV epilogue left it)
      const uint4* src = reinterpret_cast<const uint4*>(P.xq + (size_t)hq * KSTEPS * 32 * W);
      for (int i = tid; i < KSTEPS * 32 * W / 4; i += FAST_THREADS) reinterpret_cast<uint4*>(qsm)[i] = __ldcg(src + i);
    }
    if (layer + 1 < P.L && (int)blockIdx.x < P.m.o_split && hq % G == 0) {
      // the same keys and values of the next layer (the cached prefix does not change during the
      // forward): one CTA per KV head pulls them into L2 now, one 128-byte line per thread and pass
      const uint8_t* nk_ = reinterpret_cast<const uint8_t*>(kg) + P.kv_layer_elems * 2;
      const uint8_t* nv_ = reinterpret_cast<const uint8_t*>(vg) + P.kv_layer_elems * 2;
      const int lines = (k1 * HD * 2 + 127) >> 7;
      for (int i = tid; i < lines; i += FAST_THREADS) {
        prefetch_l2(nk_ + (size_t)i * 128);
        prefetch_l2(nv_ + (size_t)i * 128);
      }
    }
    __syncthreads();

    float m_run[NH], l_run[NH], o[DT][4];
#pragma unroll
    for (int h = 0; h < NH; ++h) { m_run[h] = -CUDART_INF_F; l_run[h] = 0.f; }
#pragma unroll
    for (int dt = 0; dt < DT; ++dt) o[dt][0] = o[dt][1] = o[dt][2] = o[dt][3] = 0.f;

    for (; key0 < k1; key0 += key_step) {
      __syncwarp();
#pragma unroll
      for (int i = 0; i < LPL; ++i) {
        const int idx = lane + 32 * i;
        *reinterpret_cast<uint4*>(kv_w + (idx / CH) * ROWB + (idx % CH) * 16) = kq[i];
        *reinterpret_cast<uint4*>(kv_w + 16 * ROWB + (idx / CH) * ROWB + (idx % CH) * 16) = vq[i];
      }
      __syncwarp();
      {  // the next tile's loads, in flight during this tile's arithmetic
        const int nkey0 = key0 + key_step;
#pragma unroll
        for (int i = 0; i < LPL; ++i) {
          const int idx = lane + 32 * i, key = nkey0 + idx / CH;
          kq[i] = vq[i] = make_uint4(0u, 0u, 0u, 0u);
          if (key < k1) {
            kq[i] = __ldcg(kg + (size_t)key * CH + idx % CH);
            vq[i] = __ldcg(vg + (size_t)key * CH + idx % CH);
          }
        }
      }
      // scores: thread holds rows g (and g + 8) x keys 8j + 2t, 8j + 2t + 1 of the tile
      float sc[2][4];
#pragma unroll
      for (int j = 0; j < 2; ++j) sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f;
#pragma unroll
      for (int s = 0; s < KSTEPS; ++s) {
        uint32_t ahi[4] = {0u, 0u, 0u, 0u}, alo[4] = {0u, 0u, 0u, 0u};
        load_afrag<LO>(q_lane + s * (32 * W * 4), 0, ahi, alo);
        if (T16) load_afrag<LO>(q_lane + s * (32 * W * 4) + WH * 4, 1, ahi, alo);
        if (MERGE) {
          ahi[1] = alo[0];
          ahi[3] = alo[2];
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const uint32_t b0 = lds_u32(k_lane + j * 8 * ROWB + s * 32), b1 = lds_u32(k_lane + j * 8 * ROWB + s * 32 + 16);
          mma_bf16(sc[j], ahi, b0, b1);
          if (LO && !MERGE) mma_bf16(sc[j], alo, b0, b1);
        }
      }
      if (MERGE) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          sc[j][0] += sc[j][2];
          sc[j][1] += sc[j][3];
        }
      }
      // mask, running max / sum, weights as the A operand of the second contraction
      uint32_t phi[4], plo[4];
#pragma unroll
      for (int h = 0; h < NH; ++h) {
        const int tok = g + 8 * h;
        const bool rowok = tok >= t_lo && tok < t_hi;
        float mt = -CUDART_INF_F;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            const int key = key0 + 8 * j + 2 * t + i;
            if (!(rowok && key < k1 && key <= L + (tok - t_lo))) sc[j][2 * h + i] = -CUDART_INF_F;
            mt = fmaxf(mt, sc[j][2 * h + i]);
          }
        }
        mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 1));
        mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 2));
        const float m_new = fmaxf(m_run[h], mt);
        const float corr = m_new == -CUDART_INF_F ? 0.f : __expf(m_run[h] - m_new);
        float pw[2][2], ls = 0.f;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            pw[j][i] = sc[j][2 * h + i] == -CUDART_INF_F ? 0.f : __expf(sc[j][2 * h + i] - m_new);
            ls += pw[j][i];
          }
        }
        ls += __shfl_xor_sync(0xffffffffu, ls, 1);
        ls += __shfl_xor_sync(0xffffffffu, ls, 2);
        l_run[h] = l_run[h] * corr + ls;
        m_run[h] = m_new;
#pragma unroll
        for (int dt = 0; dt < DT; ++dt) {
          o[dt][2 * h] *= corr;
          o[dt][2 * h + 1] *= corr;
          if (MERGE) {
            o[dt][2] *= corr;
            o[dt][3] *= corr;
          }
        }
        if (LO) {
          split2(pw[0][0], pw[0][1], phi[h], plo[h]);          // keys 2t, 2t + 1
          split2(pw[1][0], pw[1][1], phi[2 + h], plo[2 + h]);  // keys 8 + 2t, 8 + 2t + 1
        } else {
          phi[h] = pack_bf16(pw[0][0], pw[0][1]);
          phi[2 + h] = pack_bf16(pw[1][0], pw[1][1]);
          plo[h] = plo[2 + h] = 0u;
        }
      }
      if (!T16) phi[1] = phi[3] = plo[1] = plo[3] = 0u;
      if (MERGE) {
        phi[1] = plo[0];
        phi[3] = plo[2];
      }
#pragma unroll
      for (int dt = 0; dt < DT; ++dt) {
        uint32_t b0, b1;
        ldmatrix_x2_trans(v_lane + dt * 16, b0, b1);
        mma_bf16(o[dt], phi, b0, b1);
        if (LO && !MERGE) mma_bf16(o[dt], plo, b0, b1);
      }
    }
    if (MERGE) {
#pragma unroll
      for (int dt = 0; dt < DT; ++dt) {
        o[dt][0] += o[dt][2];
        o[dt][1] += o[dt][3];
      }
    }
    // this warp's partial -> shared memory; then all warps combine
    __syncwarp();  // every lane is done with the warp's last K / V tile
    if (t == 0) {
#pragma unroll
      for (int h = 0; h < NH; ++h) {
        cm[warp * NROW + g + 8 * h] = m_run[h];
        cl[warp * NROW + g + 8 * h] = l_run[h];
      }
    }
#pragma unroll
    for (int dt = 0; dt < DT; ++dt) {
#pragma unroll
      for (int h = 0; h < NH; ++h)
        *reinterpret_cast<float2*>(co + (size_t)warp * CO_W + (g + 8 * h) * HD + dt * 8 + 2 * t) =
            make_float2(o[dt][2 * h], o[dt][2 * h + 1]);
    }
    __syncthreads();
    for (int idx = tid; idx < R * (HD / 2); idx += FAST_THREADS) {  // (row of the stream, dim pair)
      const int r = idx / (HD / 2), dd = (idx % (HD / 2)) * 2, tok = t_lo + r;
      float mw[FAST_WARPS], m = -CUDART_INF_F;
#pragma unroll
      for (int w = 0; w < FAST_WARPS; ++w) {
        mw[w] = cm[w * NROW + tok];
        m = fmaxf(m, mw[w]);
      }
      float l = 0.f, o0 = 0.f, o1 = 0.f;
#pragma unroll
      for (int w = 0; w < FAST_WARPS; ++w) {  // fixed order: bit-reproducible
        const float e = mw[w] == -CUDART_INF_F ? 0.f : __expf(mw[w] - m);
        const float2 ov = *reinterpret_cast<const float2*>(co + (size_t)w * CO_W + tok * HD + dd);
        l = fmaf(cl[w * NROW + tok], e, l);
        o0 = fmaf(ov.x, e, o0);
        o1 = fmaf(ov.y, e, o1);
      }
      if (KSPLIT) {  // this CTA's share of the keys only: leave (max, sum, output) for the merge
        float* dst = my_part + ((size_t)hl * FAST_MAX_T + tok) * (HD + 2);
        *reinterpret_cast<float2*>(dst + dd) = make_float2(o0, o1);
        if (dd == 0) {
          dst[HD] = m;
          dst[HD + 1] = l;
        }
      } else {
        const float il = 1.f / l;
        write_frag_pair<T16, LO>(osm, tok, hl * HD + dd, o0 * il, o1 * il);
      }
    }
  }
  __syncthreads();
  if (KSPLIT) {
    // the J CTAs of the slice meet: release arrival on the slice's monotonic counter, bounded poll
    const uint32_t target = ks_base + (uint32_t)(layer + 1) * (uint32_t)J;
    bool ok = true;
    if (tid == 0) {
      uint32_t* cnt = P.attn_cnt + slice;
      asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(cnt) : "memory");
      const long long t0 = clock64();
      uint32_t spins = 0;
      while ((int32_t)(ld_acquire_u32(cnt) - target) < 0) {
        if ((++spins & 63u) == 0u &&
            (ld_acquire_u32(P.epoch_base + 1) != 0u || (unsigned long long)(clock64() - t0) > FAST_WAIT_CYCLES)) {
          ok = false;
          break;
        }
      }
    }
    if (__syncthreads_or(ok ? 0 : 1)) ring.dead = true;  // the next grid barrier spreads the failure
    if (cnt == 0) return;
    // (max, sum) of every (split, row): one round of independent loads into shared memory, then
    // each split's weight exp(m_j - m) / sum, so that the pass over the outputs has no chain of
    // dependent loads
    float* wj = reinterpret_cast<float*>(uni + KSTEPS * 32 * W * 4);  // [hps * T][J], in the K / V staging area
    const int nrow = hps * nb * R;
    for (int idx = tid; idx < nrow * J; idx += FAST_THREADS) {
      const int j = idx % J, row = idx / J, r = row % R, it2 = row / R, hl = it2 / nb, tok = (it2 % nb) * R + r;
      const float* src = P.attn_part + ((size_t)((slice + j * P.m.o_split) * hps + hl) * FAST_MAX_T + tok) * (HD + 2);
      const float2 ml = __ldcg(reinterpret_cast<const float2*>(src + HD));
      wj[(size_t)row * 2 * J + j] = ml.x;
      wj[(size_t)row * 2 * J + J + j] = ml.y;
    }
    __syncthreads();
    for (int row = tid; row < nrow; row += FAST_THREADS) {
      float* mrow = wj + (size_t)row * 2 * J;
      float m = -CUDART_INF_F, l = 0.f;
      for (int j = 0; j < J; ++j) m = fmaxf(m, mrow[j]);
      for (int j = 0; j < J; ++j) {  // fixed order: bit-reproducible
        const float e = mrow[j] == -CUDART_INF_F ? 0.f : __expf(mrow[j] - m);
        l = fmaf(mrow[J + j], e, l);
        mrow[j] = e;
      }
      const float il = 1.f / l;
      for (int j = 0; j < J; ++j) mrow[j] *= il;
    }
    __syncthreads();
    for (int idx = tid; idx < nrow * (HD / 2); idx += FAST_THREADS) {
      const int dd = (idx % (HD / 2)) * 2, row = idx / (HD / 2), r = row % R, it2 = row / R;
      const int hl = it2 / nb, tok = (it2 % nb) * R + r;
      const float* mrow = wj + (size_t)row * 2 * J;
      const float* src = P.attn_part + ((size_t)(slice * hps + hl) * FAST_MAX_T + tok) * (HD + 2) + dd;
      const size_t jstride = (size_t)P.m.o_split * hps * FAST_MAX_T * (HD + 2);
      float o0 = 0.f, o1 = 0.f;
#pragma unroll 4
      for (int j = 0; j < J; ++j) {  // fixed order
        const float2 ov = __ldcg(reinterpret_cast<const float2*>(src + (size_t)j * jstride));
        o0 = fmaf(ov.x, mrow[j], o0);
        o1 = fmaf(ov.y, mrow[j], o1);
      }
      write_frag_pair<T16, LO>(osm, tok, hl * HD + dd, o0, o1);
    }
    __syncthreads();
  }

  // O projection of this CTA's tiles over the slice's KS k-steps
  const uint32_t o_lane = smem_u32(osm) + lane * (W * 4);
  const bool row0 = g < T, row1 = T16 && g + 8 < T;
  int left = fast_warp_tiles(warp, cnt) * KS, in_chunk = 0;
  uint32_t wb = 0;
  for (int u = warp; u < cnt; u += 2 * FAST_WARPS) {
    const int np = u + FAST_WARPS < cnt ? 2 : 1;
    float acc[2][4], acl[2][4];
#pragma unroll
    for (int p = 0; p < 2; ++p) {
      acc[p][0] = acc[p][1] = acc[p][2] = acc[p][3] = 0.f;
      acl[p][0] = acl[p][1] = acl[p][2] = acl[p][3] = 0.f;
    }
    if (hps == 1) {
      // One head per slice (any GPU with at least as many SMs as query heads): KSTEPS k-steps, and
      // a pair of tiles never straddles a chunk, so both run as independent chains, unrolled.  With
      // a single tile the second chain multiplies whatever follows in shared memory, unused.
      if (in_chunk == 0) {
        ring_acquire(ring);
        in_chunk = min(FAST_O_CHUNK, left);
        left -= in_chunk;
        wb = ring.ring + ring.slot * FAST_SLOT_BYTES + lane * 8;
      }
#pragma unroll
      for (int s = 0; s < KSTEPS; ++s) {
        uint32_t ahi[4] = {0u, 0u, 0u, 0u}, alo[4] = {0u, 0u, 0u, 0u};
        if (row0) load_afrag<LO>(o_lane + s * (32 * W * 4), 0, ahi, alo);
        if (row1) load_afrag<LO>(o_lane + s * (32 * W * 4) + WH * 4, 1, ahi, alo);
        if (MERGE) {
          ahi[1] = alo[0];
          ahi[3] = alo[2];
        }
#pragma unroll
        for (int p = 0; p < 2; ++p) {
          const uint2 bw = lds_v2(wb + (p * KSTEPS + s) * FAST_TILE_BYTES);
          mma_bf16(acc[p], ahi, bw.x, bw.y);
          if (LO && !MERGE) mma_bf16(acl[p], alo, bw.x, bw.y);
        }
      }
      wb += np * KSTEPS * FAST_TILE_BYTES;
      in_chunk -= np * KSTEPS;
      if (in_chunk == 0) ring_release(ring, lane);
    } else {
#pragma unroll
    for (int p = 0; p < 2; ++p) {
      if (p < np) {
#pragma unroll 1
        for (int s = 0; s < KS; ++s) {
          if (in_chunk == 0) {
            ring_acquire(ring);
            in_chunk = min(FAST_O_CHUNK, left);
            left -= in_chunk;
            wb = ring.ring + ring.slot * FAST_SLOT_BYTES + lane * 8;
          }
          uint32_t ahi[4] = {0u, 0u, 0u, 0u}, alo[4] = {0u, 0u, 0u, 0u};
          if (row0) load_afrag<LO>(o_lane + s * (32 * W * 4), 0, ahi, alo);
          if (row1) load_afrag<LO>(o_lane + s * (32 * W * 4) + WH * 4, 1, ahi, alo);
          if (MERGE) {
            ahi[1] = alo[0];
            ahi[3] = alo[2];
          }
          const uint2 bw = lds_v2(wb);
          wb += FAST_TILE_BYTES;
          mma_bf16(acc[p], ahi, bw.x, bw.y);
          if (LO && !MERGE) mma_bf16(acl[p], alo, bw.x, bw.y);
          if (--in_chunk == 0) ring_release(ring, lane);
        }
      }
    }
    }
    ResidAdds<T16, LO> ra[2];
#pragma unroll
    for (int p = 0; p < 2; ++p) {
      if (p < np) {
        float c[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) c[i] = acc[p][i] + acl[p][i];
        if (MERGE) {
          c[0] += c[2];
          c[1] += c[3];
        }
        resid_issue<T16, LO>(P, D, M.utile[FOP_O][u + p * FAST_WARPS], lane, c, ra[p]);
      }
    }
#pragma unroll
    for (int p = 0; p < 2; ++p)
      if (p < np) resid_finish<T16, LO>(P, D, M.utile[FOP_O][u + p * FAST_WARPS], lane, ra[p]);
  }
}

// What the phases of one CTA share for the whole forward.
struct PhaseCtx {
  float qscale;
  int dk0, dk1, dsl;  // K slice of the down projection this CTA works on
  int qd;
  uint32_t ks_base;   // key-split variant: value of this slice's arrival counter at the launch's start
};

// Phase PH of layer l: 0 QKV, 1 attention + O projection, 2 gate/up, 3 down, 4 LM head.
template <int PH, bool T16, bool LO, bool KSPLIT>
__device__ __forceinline__ void run_phase(const FastParams& P, FastMisc& M, uint8_t* uni, Ring& ring,
                                          const PhaseCtx& C, int l, uint32_t& stage_parity) {
  const int d = P.d;
  PhaseDesc D;
  D.layer = l;
  D.qscale = C.qscale;
  D.kv_layer = P.kv + (size_t)l * P.kv_layer_elems;
  D.xin = nullptr;
  D.ssq_in = nullptr;
  D.xout = nullptr;
  D.ssq_out = nullptr;
  D.gain_next = nullptr;
  D.cinc = 0;
  D.in_fix = 0;
  D.kc = 0;
  D.n_rows = d;
  if (PH == 1) {
    D.op = FOP_O; D.epi = EPI_F_RESID;
    D.xout = P.xb; D.ssq_out = P.ssq_b; D.gain_next = P.m.gains + (size_t)l * 2 * d + d;
    D.cinc = (int)blockIdx.x % P.m.o_split == 0 ? 1 - P.m.o_split : 1;
    if (P.hd == 64) attn_o_phase<64, T16, LO, KSPLIT>(P, M, uni, ring, D, l, C.ks_base);
    else if (P.hd == 128) attn_o_phase<128, T16, LO, KSPLIT>(P, M, uni, ring, D, l, C.ks_base);
    else attn_o_phase<32, T16, LO, KSPLIT>(P, M, uni, ring, D, l, C.ks_base);
    return;
  }
  if (PH == 0) {
    D.op = FOP_QKV; D.epi = EPI_F_QKV; D.in_fix = 1; D.xin = P.xa; D.ssq_in = P.ssq_a;
    D.kc = d; D.n_rows = C.qd + 2 * P.Hkv * P.hd;
  } else if (PH == 2) {
    D.op = FOP_GU; D.epi = EPI_F_SWIGLU; D.in_fix = 1; D.xin = P.xb; D.ssq_in = P.ssq_b;
    D.kc = d; D.n_rows = 2 * P.F;
  } else if (PH == 3) {
    D.op = FOP_DOWN; D.epi = EPI_F_RESID;
    D.xin = P.xd + (size_t)(C.dk0 >> 4) * (32 * Lay<T16, LO>::W); D.kc = C.dk1 - C.dk0;
    D.xout = P.xa; D.ssq_out = P.ssq_a; D.cinc = C.dsl == 0 ? 1 - P.m.down_split : 1;
    D.gain_next = P.m.gains + (size_t)(l + 1) * 2 * d;  // next layer's input norm, or the final norm
  } else {
    D.op = FOP_HEAD; D.epi = EPI_F_LOGITS; D.in_fix = 1; D.xin = P.xa; D.ssq_in = P.ssq_a;
    D.layer = 0; D.kc = d; D.n_rows = P.V;
  }
  gemm_phase<T16, LO>(P, M, uni, ring, D, stage_parity);
}

// ---- the kernel --------------------------------------------------------------------------------

template <bool T16, bool LO, bool TRACE, bool KSPLIT>
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
  ring.tab = M.chunks[warp];
  ring.ncl = (uint32_t)P.m.chunk_cnt[wi * 2];
  ring.nend = ring.ncl + (P.logits ? (uint32_t)P.m.chunk_cnt[wi * 2 + 1] : 0u);
  ring.layers_left = ring.ncl ? (uint32_t)P.L : 0u;
  ring.pc = 0;
  ring.slot = ring.parity = 0;
  ring.nslot = (uint32_t)P.nslot;
  ring.outstanding = 0;
  ring.dead = false;
  ring.policy = policy_evict_first();
  uint32_t stage_parity = 0;
  if (lane == 0) {
    mbar_init(smem_u32(&M.sbar[warp]), 1);
    for (int s = 0; s < P.nslot; ++s) mbar_init(ring.bars + s * 8, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();  // also orders this warp's chunk table before its first use
  {
    uint32_t lb = 0;
    for (uint32_t i = 0; i < ring.ncl; ++i) lb += ring.tab[i];
    lb *= FAST_TILE_BYTES;
    const uint8_t* base = P.m.wstream + P.m.stream_off[wi];
    if (lane == 0) {
      RingSide* sd = reinterpret_cast<RingSide*>(M.chunks[warp] + FAST_MAX_CHUNKS);
      sd->base = base;
      sd->map = P.layer_map;
      sd->layer_bytes = lb;
      sd->cur = 0;
      sd->n_src = (uint32_t)P.n_src_layers;
    }
    __syncwarp();
    ring.mapped = P.layer_map != nullptr;
    ring.src = base;
    if (ring.mapped) ring.src = base + (size_t)(ring.ncl ? P.layer_map[0] : P.n_src_layers) * lb;
  }
  for (int s = 0; s < P.nslot; ++s) ring_request(ring, (uint32_t)s, lane);
  const uint32_t epoch_base = ld_acquire_u32(P.epoch_base);
  // key-split variant: the slice counters are quiet between launches, and no CTA gets past the
  // first grid barrier before every CTA has read its slice's value here
  const uint32_t ks_base = KSPLIT ? ld_acquire_u32(P.attn_cnt + cta % P.m.o_split) : 0u;
  uint32_t epoch = 0;
  __syncthreads();
  trace_mark<TRACE>(P, n_trace);

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
    const __nv_bfloat162* src = reinterpret_cast<const __nv_bfloat162*>(P.embed + (size_t)id * d);
    const float2* g0 = reinterpret_cast<const float2*>(P.m.gains);  // first layer's input norm
    for (int kk0 = 0; kk0 < (d >> 1); kk0 += FAST_THREADS) {         // column pairs; a warp = 64 columns
      const int kk = kk0 + tid;
      long long ss = 0;
      if (kk < (d >> 1)) {
        const float2 x = __bfloat1622float2(src[kk]);
        const float2 gn = __ldg(g0 + kk);
        *reinterpret_cast<longlong2*>(P.hfix + (size_t)tok * d + 2 * kk) =
            make_longlong2(__float2ll_rn(x.x * FIX_SCALE) * 16, __float2ll_rn(x.y * FIX_SCALE) * 16);
        write_frag_pair<T16, LO>(P.xa, tok, 2 * kk, x.x * gn.x, x.y * gn.y);
        ss = __float2ll_rn(x.x * x.x * FIX_SCALE) + __float2ll_rn(x.y * x.y * FIX_SCALE);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      if (lane == 0 && kk < (d >> 1)) P.ssq_a[(kk >> 5) * FAST_MAX_T + tok] = ss;
    }
    const double pos = (double)M.tok_pos[tok];
    for (int j = tid; j < half; j += FAST_THREADS) {
      double sn, cs;
      sincos(pos * P.inv_freq[j], &sn, &cs);
      P.rope_cs[((size_t)tok * half + j) * 2 + 0] = (float)cs;
      P.rope_cs[((size_t)tok * half + j) * 2 + 1] = (float)sn;
    }
  }
  trace_mark<TRACE>(P, n_trace);
  bool ok = grid_sync(P, epoch_base + (++epoch) * (uint32_t)P.m.n_cta, false);
  trace_mark<TRACE>(P, n_trace);
  // every CTA has read the base by now: publish the next launch's (this launch arrives 1 + 4 L times)
  if (ok && cta == 0 && tid == 0)
    st_release_u32(P.epoch_base, epoch_base + (uint32_t)(1 + 4 * P.L) * (uint32_t)P.m.n_cta);

  // K slice of the down projection this CTA works on
  const int dsteps = P.F >> 4, dsl = cta % P.m.down_split;
  const int dk0 = (int)(((long long)dsl * dsteps) / P.m.down_split) << 4;
  const int dk1 = (int)(((long long)(dsl + 1) * dsteps) / P.m.down_split) << 4;
  const float qscale = rsqrtf((float)P.hd);

  // 4 phases per layer (QKV, attention + O, gate/up, down), then the LM head.  Each phase is its
  // own call site, so that what a phase is (its projection, input, epilogue) is known at compile
  // time there: every instruction between two barriers is on the critical path.
  const int n_ssq = (d + SSQ_COLS - 1) / SSQ_COLS * FAST_MAX_T;
  const PhaseCtx C{qscale, dk0, dk1, dsl, qd, ks_base};
#pragma unroll 1
  for (int l = 0; l < P.L && ok; ++l) {
    if (l + 1 < P.L && cta == l % P.m.n_cta) {
      // the small per-layer constants are read once per forward, so they would miss all the way
      // to HBM in the middle of an epilogue: one CTA pulls the next layer's into L2 ahead of time
      const int nq = (P.Hq + 2 * P.Hkv) * P.hd;
      const uint8_t* bq = reinterpret_cast<const uint8_t*>(P.m.bias_qkv + (size_t)(l + 1) * nq);
      const uint8_t* gq = reinterpret_cast<const uint8_t*>(P.m.gains + (size_t)(l + 1) * 2 * d);
      for (int i = tid; i < ((nq * 4 + 127) >> 7); i += FAST_THREADS) prefetch_l2(bq + (size_t)i * 128);
      for (int i = tid; i < ((3 * d * 4 + 127) >> 7); i += FAST_THREADS) prefetch_l2(gq + (size_t)i * 128);
    }
    // A set of sums of squares is cleared while it is idle: the one the O projection adds to
    // during the QKV phase, the one the down projection adds to during the attention + O phase.
    if (cta == P.m.n_cta - 1)
      for (int i = tid; i < n_ssq; i += FAST_THREADS) P.ssq_b[i] = 0;
    run_phase<0, T16, LO, KSPLIT>(P, M, uni, ring, C, l, stage_parity);
    trace_mark<TRACE>(P, n_trace);
    ok = grid_sync(P, epoch_base + (++epoch) * (uint32_t)P.m.n_cta, ring.dead);
    trace_mark<TRACE>(P, n_trace);
    if (!ok) break;
    if (cta == P.m.n_cta - 1)
      for (int i = tid; i < n_ssq; i += FAST_THREADS) P.ssq_a[i] = 0;
    run_phase<1, T16, LO, KSPLIT>(P, M, uni, ring, C, l, stage_parity);
    trace_mark<TRACE>(P, n_trace);
    ok = grid_sync(P, epoch_base + (++epoch) * (uint32_t)P.m.n_cta, ring.dead);
    trace_mark<TRACE>(P, n_trace);
    if (!ok) break;
    run_phase<2, T16, LO, KSPLIT>(P, M, uni, ring, C, l, stage_parity);
    trace_mark<TRACE>(P, n_trace);
    ok = grid_sync(P, epoch_base + (++epoch) * (uint32_t)P.m.n_cta, ring.dead);
    trace_mark<TRACE>(P, n_trace);
    if (!ok) break;
    run_phase<3, T16, LO, KSPLIT>(P, M, uni, ring, C, l, stage_parity);
    trace_mark<TRACE>(P, n_trace);
    ok = grid_sync(P, epoch_base + (++epoch) * (uint32_t)P.m.n_cta, ring.dead);
    trace_mark<TRACE>(P, n_trace);
  }
  if (ok && P.logits) {
    run_phase<4, T16, LO, KSPLIT>(P, M, uni, ring, C, 0, stage_parity);
    trace_mark<TRACE>(P, n_trace);
    if (__syncthreads_or(ring.dead ? 1 : 0)) ok = false;
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

// The kernel variant for a launch, from the translation unit that instantiates it.
template <bool T16, bool LO>
inline const void* fast_kernel_variant(bool trace) {
  return trace ? (const void*)fast_forward_kernel<T16, LO, true, false>
               : (const void*)fast_forward_kernel<T16, LO, false, false>;
}
// The key-split variant (long prefixes): split activations, no trace.
template <bool T16>
inline const void* fast_kernel_keysplit_variant() {
  return (const void*)fast_forward_kernel<T16, true, false, true>;
}

}  // namespace

}  // namespace ssd
