// Persistent small-batch verify kernel ("fast path"): shared definitions of the host-side plan /
// weight packer (fast_pack.cu) and of the kernel (fast_kernel.cuh) and its launcher (fast_verify.cu).
//
// The verify forward of Eq. 4 over T = B * (gamma + 1) <= 16 rows is bound by streaming every
// weight byte once and, because each of its ~120 phases depends on the one before, by how few
// instructions a phase needs.  The fast path keeps one CTA per SM alive for the whole forward;
// each of its warps owns a private, contiguous byte stream of weights in HBM that it pulls through
// a private shared-memory ring with bulk async copies.  The streams hold the weights pre-tiled in
// the operand order of the warp-level tensor-core instruction (8 weight rows x 16 k, 256 bytes a
// tile) and pre-cut into chunks of whole k-steps, so a tile goes from shared memory to the
// instruction with one 8-byte load per lane and the inner loop has no bookkeeping.
#pragma once
#include <stdint.h>

#include <vector>

#include "common.cuh"

namespace ssd {

constexpr int FAST_WARPS = 8;  // warps per CTA; they split K of every projection
constexpr int FAST_THREADS = FAST_WARPS * 32;
constexpr int FAST_TILE_BYTES = 256;  // one operand tile: 8 weight rows x 16 k, bf16
constexpr int FAST_SLOT_TILES = 20;  // a ring slot holds one chunk of at most this many tiles
constexpr int FAST_SLOT_BYTES = FAST_TILE_BYTES * FAST_SLOT_TILES;
// Chunks of the O projection's stream (runs of a warp's own tiles): a power of two, so that a pair
// of output tiles with 2, 4 or 8 k-steps each never straddles two chunks.
constexpr int FAST_O_CHUNK = 16;
constexpr int FAST_MAX_SLOTS = 8;     // most ring slots per warp (barrier storage)
constexpr int FAST_RING_SLOTS = 3;    // ring slots per warp actually used
constexpr int FAST_MAXU = 10;         // output tiles a CTA accumulates at once (one "round")
constexpr int FAST_MAX_UNITS = 64;    // output tiles per CTA and op (table size in shared memory)
constexpr int FAST_MAX_CHUNKS = 128;  // chunks per warp: one layer's plus the LM head's
constexpr int FAST_MAX_T = 16;        // rows per forward
constexpr int FAST_MAX_CTAS = 256;

enum FastOpId { FOP_QKV = 0, FOP_O = 1, FOP_GU = 2, FOP_DOWN = 3, FOP_HEAD = 4, FOP_COUNT = 5 };

struct FastOpShape {
  int n_rows;   // output features (weight rows) in packed order
  int K;        // input features
  int n_tiles;  // ceil(n_rows / 8)
  int ksteps;   // K / 16
  int ksplit;   // CTA c works on K slice c % ksplit (1: every CTA covers all of K)
  int by_tile;  // 0: the warps of a CTA split the K slice; 1: they split the CTA's tiles (tile u goes
                // to warp u % FAST_WARPS, which covers the whole K slice)
};

// K slice (in steps of 16 columns) of an op that CTA `cta` works on.
inline int fast_slice_k0(const FastOpShape& s, int cta) {
  return (int)(((long long)(cta % s.ksplit) * s.ksteps) / s.ksplit);
}
inline int fast_slice_k1(const FastOpShape& s, int cta) {
  return (int)(((long long)(cta % s.ksplit + 1) * s.ksteps) / s.ksplit);
}

// First and one-past-last k-step that warp w covers of a CTA's slice of `ksteps` steps.
__host__ __device__ inline int fast_warp_k0(int w, int ksteps) {
  return (int)(((long long)w * ksteps) / FAST_WARPS);
}
__host__ __device__ inline int fast_warp_k1(int w, int ksteps) {
  return (int)(((long long)(w + 1) * ksteps) / FAST_WARPS);
}
// k-steps per chunk for a round of `cnt` tiles (a chunk never holds more than FAST_SLOT_TILES).
__host__ __device__ inline int fast_steps_per_chunk(int cnt) { return FAST_SLOT_TILES / cnt; }

// Tiles of a CTA's `cnt` that warp w owns when the warps split the tiles.
__host__ __device__ inline int fast_warp_tiles(int w, int cnt) {
  return cnt > w ? (cnt - w + FAST_WARPS - 1) / FAST_WARPS : 0;
}

// Which output tiles each CTA owns for each op, and where each warp's byte stream lives.
struct FastPlan {
  int n_cta = 0;
  int n_layers = 0;
  FastOpShape ops[FOP_COUNT];
  std::vector<int32_t> unit_cnt;   // [n_cta][FOP_COUNT]
  std::vector<int32_t> unit_off;   // [n_cta][FOP_COUNT] start in unit_tile
  std::vector<int32_t> unit_tile;  // tile indices, grouped by (cta, op)
  std::vector<uint64_t> stream_off;  // [n_cta][FAST_WARPS] byte offset of the warp's stream
  // chunk sizes (in tiles) of a warp's stream: first one layer's chunks, then the LM head's
  std::vector<uint8_t> chunks;       // [n_cta][FAST_WARPS][FAST_MAX_CHUNKS]
  std::vector<int32_t> chunk_cnt;    // [n_cta][FAST_WARPS][2]: chunks per layer, chunks of the head
  int max_chunks = 0;                // largest per-layer + head chunk count of any warp
  uint64_t total_bytes = 0;
};

bool fast_supported(const ssd_model_config& c);
int fast_down_split(const ssd_model_config& c);
// K slices of the O projection = groups of query heads; a slice's CTAs compute the attention of
// its heads themselves, so the O projection needs no exchange after the attention.
int fast_o_split(const ssd_model_config& c, int n_cta);
FastPlan fast_make_plan(const ssd_model_config& c, int n_cta);
// Packs the bf16 weights of the flat host blob (layout of ssd_model_create) into the per-warp
// streams described by `plan` (out has plan.total_bytes bytes).
void fast_pack_streams(const ssd_model_config& c, const FastPlan& plan, const uint16_t* blob,
                       uint8_t* out);
long long fast_unpack_streams(const ssd_model_config& c, const FastPlan& plan, const uint8_t* streams,
                              uint16_t* blob_out);
// Biases of q/k/v in packed row order and the three kinds of norm gains, as fp32:
//   bias [L][n_qkv]; gains [L][2][d] followed by the final norm's [d].
void fast_pack_aux(const ssd_model_config& c, const uint16_t* blob, std::vector<float>& bias,
                   std::vector<float>& gains);

// Device-side view of a packed model.
struct FastModelDev {
  const uint8_t* wstream;
  const uint64_t* stream_off;
  const uint8_t* chunks;
  const int32_t* chunk_cnt;
  const int32_t* unit_cnt;
  const int32_t* unit_off;
  const int32_t* unit_tile;
  const float* bias_qkv;
  const float* gains;
  int n_cta;
  int max_units;    // most tiles any CTA owns for one op
  int down_split;   // K slices of the down projection
  int o_split;      // K slices (groups of query heads) of the O projection
  int max_stage_k;  // widest input slice a CTA stages in shared memory
};

struct FastParams {
  FastModelDev m;
  const bf16* embed;
  const double* inv_freq;
  int L, d, Hq, Hkv, hd, hd_shift, F, V, vocab_in;  // hd = 1 << hd_shift
  // A model that inherits layers of another: layer l runs the packed weights of source layer
  // layer_map[l] (null: identity); n_src_layers = layers in the packed streams, before the head.
  const int32_t* layer_map;
  int n_src_layers;
  float eps;
  // streams
  bf16* kv;
  unsigned long long kv_layer_elems;
  int cap;
  const int32_t* len;
  const int32_t* pending;
  int32_t* status;
  // rows of this forward: streams b0 .. b0+nb-1, R rows each
  int b0, nb, R, T;
  const int32_t* row_ids;       // explicit ids [nb * R], or null: row 0 = pending, rows 1.. = draft
  const int32_t* draft_tokens;  // [B, gamma] when row_ids is null
  // workspace
  long long* hfix;  // residual stream [T][d]: 2^-32 fixed point above a 4-bit arrival count
  float *rope_cs, *logits;  // logits null: skip the LM head
  // Inputs of the projections, written by their producers already in the tensor-core operand layout
  // (bf16 leading part + remainder, see fast_kernel.cuh): the RMS-norm inputs x * gain of the QKV /
  // LM-head projection (xa) and of gate/up (xb), SiLU(g) * u (xd); and
  // per 64 columns and row the sums of squares that go with xa / xb.
  uint32_t *xa, *xb, *xd, *xq;  // xq: the rotated, scaled queries
  long long *ssq_a, *ssq_b;  // [ceil(d / 64)][FAST_MAX_T], 2^-32 fixed point
  // key-split attention (long prefixes): per CTA the un-normalised partials of its heads' rows
  // [n_cta][heads per slice][FAST_MAX_T][hd + 2], and one monotonic arrival counter per slice;
  // key_split != 0 selects the kernel variant that uses them
  float* attn_part;
  uint32_t* attn_cnt;
  int key_split;
  uint32_t* flags;       // [0] grid-barrier arrival counter, monotonic across launches
  uint32_t* epoch_base;  // [0] counter value at the start of the next launch, [1] nonzero after a failure
  // optional trace: thread 0 of CTA c stores clock64() at trace[c * trace_cap + i] for its i-th
  // phase boundary (before and after every grid barrier); null: off
  long long* trace;
  int trace_cap;
  // 0: activations enter the tensor cores rounded to bf16 (one instruction per tile and k-step);
  // 1: as bf16 leading part + bf16 remainder (two instructions, close to fp32 inputs)
  int split_act;
  // shared-memory carve-up (bytes)
  int nslot, ring_warp_bytes, union_off, misc_off;
};

size_t fast_union_bytes(int stage_k, int head_dim, int T, int o_steps, bool split);
cudaError_t launch_fast_forward(const FastParams& p, cudaStream_t st);

}  // namespace ssd
