// Batched verify forward (Eq. 4 for more than 16 rows: many streams, or a prefill chunk) on the
// 5th-generation tensor cores: declarations shared by the tcgen05 projection kernel (tc_gemm.cu),
// the row-wise kernels around it (tc_rows.cu), the batched attention (tc_attention.cu) and the
// host code that strings them together (api.cu).
//
// Projections run "swapped": D[weight row, token] = sum_k W[row, k] * X[token, k].  A CTA owns a
// tile of 128 weight rows - the M of one tcgen05.mma, so a tile's accumulator fills the 128 lanes
// of tensor memory - and all tokens (the instruction's N, up to 256 per instruction, more as
// several column ranges of the same accumulator).  Weights are therefore read from HBM exactly
// once per forward, whatever the number of rows.  Both operands are staged in shared memory by
// plain bulk copies: weights are packed once, at model creation, and activations are written by
// their producers, in the layout the instruction's shared-memory descriptors expect, so that no
// tensor map and no swizzle is involved:
//
//   canonical K-major layout without swizzle: a "core matrix" is 8 rows x 16 bytes (8 bf16 along
//   K), stored as 128 contiguous bytes; the descriptor gives the byte distance between core
//   matrices that are neighbours along K ("leading" offset) and along the rows ("stride" offset).
//
//   weights, per (tile of 128 rows, k-step of 16 columns) one 4 KB block:
//       byte(r, k) = (k / 8) * 2048 + r * 16 + (k % 8) * 2           leading 2048, stride 128
//   activations (Mpad token rows, a multiple of 16): up to 256 rows are one chunk of Mc = Mpad
//   rows; more are ceil(Mpad / 256) chunks of Mc = Mpad / chunks (rounded up to 16) rows each.
//   A chunk is stored whole, per k-step one block of Mc * 64 bytes:
//       byte(part, t, k) = ((t / Mc) * KS + k / 16) * Mc * 64
//                          + ((k / 8) % 2) * Mc * 32 + part * Mc * 16 + (t % Mc) * 16 + (k % 8) * 2
//   (KS = k-steps of the operand), so that a CTA that multiplies one chunk of rows - see below -
//   reads its share of a k-step as one contiguous run,
//   with part 0 = bf16 leading part of the fp32 activation, part 1 = bf16 of the remainder: the
//   tensor cores multiply both with the exact bf16 weights, so products are exact to ~2^-17
//   relative, as in the small-batch kernel.  The two parts of a token sit Mpad rows apart in one
//   2 * Mpad-row operand: with up to 256 token rows one instruction multiplies both (N = 2 Mpad,
//   the two halves of the accumulator are added in the epilogue), which matters because an
//   instruction costs ~190 cycles whatever its N (measured); with more rows the two parts are
//   separate instructions into the same accumulator columns, and a CTA owns TWO tiles of weight
//   rows x one chunk of token rows (2 x Mc <= 512 accumulator columns): at 448 rows the
//   projections are bound by the operand traffic from L2 into the SMs, and two tiles per CTA
//   share every activation block they load (5.5 KB per instruction instead of 8).
//
// K is split across CTAs where a projection has too few row tiles to occupy the GPU; the partial
// sums go to a workspace and the row-wise kernel that consumes the projection adds them in a
// fixed order (bit-reproducible, no atomics).
#pragma once
#include <stdint.h>

#include "common.cuh"

namespace ssd {

constexpr int TC_TILE_ROWS = 128;                 // weight rows per tile = M of the MMA
constexpr int TC_WBLOCK = TC_TILE_ROWS * 16 * 2;  // bytes of one (tile, k-step) weight block
constexpr int TC_MAX_ROWS = 512;                  // token rows per forward (tensor-memory columns)
constexpr int TC_THREADS = 256;                   // copy warp, MMA warp, six more; all eight run the epilogue

enum TcEpilogue {
  TC_EPI_PARTIAL = 0,  // part[split][token][row] = acc                (summed by the consumer)
  TC_EPI_STORE = 1,    // out[token * ldo + row] = acc                  (LM head -> logits)
  TC_EPI_SWIGLU = 2    // rows interleaved (gate_j, up_j): packed[token, j] = SiLU(gate) * up
};

// Programmatic dependent launch: the kernels of the batched forward form one dependency chain
// of ~200 short launches.  Each lets its successor start launching at once (tc_pdl_trigger) and
// waits for its predecessor's results only where it first needs them (tc_pdl_wait, which returns
// when the whole preceding grid has completed and its writes are visible), so launch latency and
// set-up - and, in the projections, the first weight copies, which depend on nothing - overlap the
// predecessor's tail.  Nothing that blocks on a shared resource (tensor memory) is taken before
// the wait.  Without the launch attribute both instructions do nothing.
#ifdef __CUDACC__
__device__ __forceinline__ void tc_pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void tc_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
template <typename... KArgs, typename... Args>
inline cudaError_t tc_launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                 Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}
#endif

inline int tc_round16(int m) { return (m + 15) / 16 * 16; }
inline size_t tc_weight_bytes(int n_rows, int K) {
  return (size_t)((n_rows + TC_TILE_ROWS - 1) / TC_TILE_ROWS) * ((K + 15) / 16) * TC_WBLOCK;
}
// Row chunks of a packed activation operand of M rows (see the layout above).
struct TcChunks {
  int n, rows;  // chunks, rows per chunk (a multiple of 16)
};
inline TcChunks tc_chunks(int M) {
  const int Mpad = tc_round16(M);
  TcChunks c;
  c.n = Mpad <= 256 ? 1 : (Mpad + 255) / 256;
  c.rows = c.n == 1 ? Mpad : tc_round16((Mpad + c.n - 1) / c.n);
  return c;
}
// Bytes of a packed activation operand of K columns for M rows.
inline size_t tc_act_bytes(int M, int K) {
  const TcChunks c = tc_chunks(M);
  return (size_t)((K + 15) / 16) * c.n * c.rows * 64;
}
// Byte offset of element (part, t, k) of a packed operand with chunks of Mc rows and KS k-steps.
#ifdef __CUDACC__
__host__ __device__
#endif
inline size_t tc_act_off(int Mc, int KS, int part, int t, int k) {
  const int ch = t / Mc, tl = t - ch * Mc;
  return ((size_t)ch * KS + (size_t)(k >> 4)) * ((size_t)Mc * 64) + (size_t)((k >> 3) & 1) * ((size_t)Mc * 32) +
         (size_t)part * ((size_t)Mc * 16) + (size_t)tl * 16 + (size_t)(k & 7) * 2;
}
// The same offset in two terms, for code that writes many columns of one row: the row's term
// (its chunk and its place in it) and the column's.
#ifdef __CUDACC__
__host__ __device__
#endif
inline size_t tc_act_row_off(int Mc, int KS, int t) {
  const int ch = t / Mc, tl = t - ch * Mc;
  return (size_t)ch * KS * ((size_t)Mc * 64) + (size_t)tl * 16;
}
#ifdef __CUDACC__
__host__ __device__
#endif
inline size_t tc_act_col_off(int Mc, int k) {
  return (size_t)(k >> 4) * ((size_t)Mc * 64) + (size_t)((k >> 3) & 1) * ((size_t)Mc * 32) + (size_t)(k & 7) * 2;
}
// Weight-row tiles per CTA: two where the token rows come in chunks (more than 256 rows) and the
// projection is long (many tiles, or a deep K): the tiles then share the activation blocks the
// CTA loads.  A short projection keeps one tile per CTA, which doubles its CTAs per K slice, so
// that half as many slices - and half the partial sums, whose stores and re-reads are what such
// a projection mostly costs - occupy the GPU.
inline int tc_tiles_per_cta(int n_rows, int K, int M) {
  const int tiles = (n_rows + TC_TILE_ROWS - 1) / TC_TILE_ROWS;
  return tc_chunks(M).n > 1 && (tiles >= 64 || K > 4096) ? 2 : 1;
}
// K slices for a projection of n_rows x K over M token rows on n_sm SMs: enough CTAs to occupy
// the GPU, at least four k-steps each.
inline int tc_ksplit(int n_rows, int K, int M, int n_sm) {
  const int tiles = (n_rows + TC_TILE_ROWS - 1) / TC_TILE_ROWS, ks = (K + 15) / 16;
  const int ntile = tc_tiles_per_cta(n_rows, K, M);
  int s = n_sm / ((tiles + ntile - 1) / ntile * tc_chunks(M).n);
  if (s > ks / 4) s = ks / 4;
  return s < 1 ? 1 : s;
}

struct TcGemm {
  const uint8_t* w;   // packed weights of the projection
  const uint8_t* a;   // packed activations
  int n_rows, K;      // weight rows, input columns
  int M;              // token rows
  int ksplit;
  int epi;
  float* part;        // TC_EPI_PARTIAL: [ksplit][Mpad][tiles * 128]
  float* out;         // TC_EPI_STORE
  int ldo;
  uint8_t* act_out;   // TC_EPI_SWIGLU: packed operand of n_rows / 2 columns
  int32_t* status;
};

// tc_gemm.cu
cudaError_t tc_pack_weights(const bf16* w_rowmajor, int n_rows, int K, uint8_t* packed, cudaStream_t st);
cudaError_t tc_unpack_weights(const uint8_t* packed, int n_rows, int K, bf16* w_rowmajor, cudaStream_t st);
cudaError_t launch_tc_gemm(const TcGemm& g, cudaStream_t st);

// tc_rows.cu
// h[m, :] += sum of `nsplit` partial projections (part may be null); then the RMS norm of the row
// times `gain`, written as a packed operand (hi + lo) of d columns.  h_in may differ from h (the
// first layer reads the embedding rows).
void launch_tc_norm_pack(float* h, const float* part, int nsplit, int ld_part, int M, int d,
                         const bf16* gain, float eps, uint8_t* apack, cudaStream_t st);
// Packs fp32 rows x[M, K] as an operand (used by tests of the projection kernel).
void launch_tc_pack_rows(const float* x, int M, int K, uint8_t* apack, cudaStream_t st);
// q/k/v = sum of partials + bias; rotary embedding; q (scaled) to qrot [M, Hq * hd] fp32, K and V
// appended to the cache at len + r.
// Paged cache (page_table non-null): kv_layer is the layer's page pool [page][2][Hkv][64][hd] and
// token t of stream b lives in page page_table[b * max_pages + t / 64], slot t % 64.
constexpr int TC_PAGE_TOKENS = 64;
void launch_tc_qkv_post(const float* part, int nsplit, int ld_part, int Mpad, const bf16* bias,
                        const float* cs, float* qrot, bf16* kv_layer, const int32_t* len, RowMap rm,
                        int cap, int Hq, int Hkv, int hd, const int32_t* page_table, int max_pages,
                        int32_t* status, cudaStream_t st);
// Page bookkeeping of a paged cache.  ensure: every stream of the forward owns pages for its
// first len + R slots (taken from the free stack).  release: pages wholly beyond a stream's
// committed length go back to the free stack - the O(1) rollback of a paged cache.
void launch_page_ensure(const int32_t* len, RowMap rm, int32_t* page_table, int32_t* pages_used,
                        int32_t* free_stack, int32_t* free_top, int max_pages, int32_t* status,
                        cudaStream_t st);
void launch_page_release(const int32_t* len, int B, int32_t* page_table, int32_t* pages_used,
                         int32_t* free_stack, int32_t* free_top, int max_pages, cudaStream_t st);

// tc_attention.cu: verify attention for all streams of the forward (causal inside the block, GQA),
// split over the keys; the merged result is written as the packed operand of the O projection.
cudaError_t launch_tc_attention(const float* qrot, const bf16* kv_layer, const int32_t* len, RowMap rm,
                                int cap, int Hq, int Hkv, int hd, float* part, int nsplit,
                                int keys_per_split, uint8_t* apack_out, int Mpad,
                                const int32_t* page_table, int max_pages, int which_kernel, int32_t* status,
                                cudaStream_t st);
int tc_attention_ctas_per_sm(int hd);  // CTAs of the attention kernel an SM holds at once
// tc_attention5.cu: the same partial results (one per row, head and key split) on tcgen05 tensor
// cores, for head sizes 64 and 128.  It costs less per key and more per CTA than the warp-level
// kernel (measured: 3.0 against 3.5 us per 64 keys, ~6 us more to start and finish), so
// launch_tc_attention uses it from TC_ATTN5_MIN_KEYS keys per CTA on (which_kernel 0), always
// (2, where the head size allows) or never (1).
constexpr int TC_ATTN5_MIN_KEYS = 1024;
cudaError_t launch_tc_attention5(const float* qrot, const bf16* kv_layer, const int32_t* len, RowMap rm, int cap,
                                 int Hq, int Hkv, int hd, float* part, int nsplit, int keys_per_split,
                                 const int32_t* page_table, int max_pages, int32_t* status, cudaStream_t st);

}  // namespace ssd
