// Host side of the persistent small-batch verify kernel: which output tiles every CTA owns, and
// the packing of the weights into per-warp byte streams in tensor-core operand order.
//
// Packed row order of each projection of the decoder (Sec. 3.1 of the paper; Qwen2.5-style):
//   QKV  : q heads, then k heads, then v heads; inside every q and k head the rotary partners
//          (j, j + hd/2) are made adjacent (packed row 2j = original row j, 2j+1 = j + hd/2), so
//          the two values one rotation needs land in one thread's accumulator pair.
//   GU   : gate_j and up_j adjacent (row 2j = gate_j, 2j+1 = up_j), same reason for SiLU(g)*u.
//   O, DOWN, HEAD : original order.
// A tile covers 8 packed rows x 16 k.  Lane l of a warp (g = l / 4, t = l % 4) owns 8 bytes:
//   W[row0 + g][k0 + 2t, 2t+1] and W[row0 + g][k0 + 8 + 2t, 2t+1]
// which is the "col" B operand of mma.m16n8k16 (the activations are the 16-row A operand).
//
// Order of a warp's stream: layers; ops (QKV, O, gate/up, down); rounds of FAST_MAXU of the CTA's
// tiles; the warp's k-steps; the round's tiles.  The stream is cut into chunks of whole k-steps of
// at most FAST_SLOT_TILES tiles: one chunk is one bulk copy into one ring slot.  The O projection
// is the exception: its K is split by groups of query heads over the CTAs, the warps of a CTA split
// its tiles (warp w: tiles w, w + FAST_WARPS, ..), each tile with all k-steps of the slice in
// order, and the chunks are simply runs of FAST_O_CHUNK tiles of that sequence.
#include <string.h>

#include <algorithm>
#include <numeric>

#include "fast.h"

namespace ssd {

namespace {

struct BlobView {
  // element offsets into the flat blob
  size_t embed;
  struct Layer {
    size_t norm1, wq, bq, wk, bk, wv, bv, wo, norm2, wg, wu, wd;
  };
  std::vector<Layer> layers;
  size_t norm_f, head;
};

BlobView view_blob(const ssd_model_config& c) {
  BlobView v;
  size_t d = c.d_model, qd = (size_t)c.n_q_heads * c.head_dim, kvd = (size_t)c.n_kv_heads * c.head_dim;
  size_t F = c.d_ffn, off = 0;
  auto take = [&](size_t n) { size_t o = off; off += n; return o; };
  v.embed = take((size_t)(c.vocab_out + c.vocab_text) * d);
  v.layers.resize(c.n_layers);
  for (auto& L : v.layers) {
    L.norm1 = take(d);
    L.wq = take(qd * d);
    L.bq = take(qd);
    L.wk = take(kvd * d);
    L.bk = take(kvd);
    L.wv = take(kvd * d);
    L.bv = take(kvd);
    L.wo = take(d * qd);
    L.norm2 = take(d);
    L.wg = take(F * d);
    L.wu = take(F * d);
    L.wd = take(d * F);
  }
  v.norm_f = take(d);
  v.head = take((size_t)c.vocab_out * d);
  return v;
}

// Original row of packed row n inside a head-structured block with rotary interleave.
inline int rope_unpack_row(int n, int hd) {
  int hh = n / hd, w = n % hd;
  return hh * hd + (w >> 1) + (w & 1) * (hd >> 1);
}

// Pointer to packed row n of op `op` in layer l (nullptr: a padding row of zeros).
const uint16_t* packed_row(const ssd_model_config& c, const BlobView& v, const uint16_t* blob,
                           int op, int l, int n) {
  const size_t d = c.d_model, qd = (size_t)c.n_q_heads * c.head_dim;
  const size_t kvd = (size_t)c.n_kv_heads * c.head_dim, F = c.d_ffn;
  switch (op) {
    case FOP_QKV: {
      const BlobView::Layer& L = v.layers[l];
      if ((size_t)n < qd) return blob + L.wq + (size_t)rope_unpack_row(n, c.head_dim) * d;
      if ((size_t)n < qd + kvd) return blob + L.wk + (size_t)rope_unpack_row(n - (int)qd, c.head_dim) * d;
      if ((size_t)n < qd + 2 * kvd) return blob + L.wv + ((size_t)n - qd - kvd) * d;
      return nullptr;
    }
    case FOP_O:
      return (size_t)n < d ? blob + v.layers[l].wo + (size_t)n * qd : nullptr;
    case FOP_GU:
      if ((size_t)n >= 2 * F) return nullptr;
      return blob + ((n & 1) ? v.layers[l].wu : v.layers[l].wg) + (size_t)(n >> 1) * d;
    case FOP_DOWN:
      return (size_t)n < d ? blob + v.layers[l].wd + (size_t)n * F : nullptr;
    case FOP_HEAD:
      return n < c.vocab_out ? blob + v.head + (size_t)n * d : nullptr;
  }
  return nullptr;
}

float bf16_bits_to_float(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

}  // namespace

bool fast_supported(const ssd_model_config& c) {
  if (c.weight_dtype != 1) return false;
  if (c.head_dim != 32 && c.head_dim != 64 && c.head_dim != 128) return false;
  const int qd = c.n_q_heads * c.head_dim;
  if ((c.d_model & 15) || (c.d_ffn & 15) || (qd & 15)) return false;
  if (c.d_model > 8192 || qd > 8192 || c.n_q_heads > 64) return false;
  return true;
}

int fast_o_split(const ssd_model_config& c, int n_cta) {
  // whole heads per slice; at most 16 slices, the most the 4-bit arrival count of a residual
  // element can tell apart (and every slice needs a CTA)
  int s = 1;
  for (int v = 1; v <= c.n_q_heads && v <= n_cta && v <= 16; ++v)
    if (c.n_q_heads % v == 0) s = v;
  return s;
}

int fast_down_split(const ssd_model_config& c) {
  // slices of at most 640 input columns: a CTA stages its slice of the activations in shared
  // memory, and short slices keep that copy off the critical path (8 slices measured best for F = 4864)
  int s = 1;
  while (c.d_ffn / s > 640 && s < 16) s *= 2;
  return s;
}

FastPlan fast_make_plan(const ssd_model_config& c, int n_cta) {
  FastPlan p;
  p.n_cta = n_cta;
  p.n_layers = c.n_layers;
  const int d = c.d_model, qd = c.n_q_heads * c.head_dim, kvd = c.n_kv_heads * c.head_dim, F = c.d_ffn;
  auto shape = [](int rows, int K, int split) { return FastOpShape{rows, K, (rows + 7) / 8, K / 16, split, 0}; };
  p.ops[FOP_QKV] = shape(qd + 2 * kvd, d, 1);
  p.ops[FOP_O] = shape(d, qd, fast_o_split(c, n_cta));
  p.ops[FOP_O].by_tile = 1;
  p.ops[FOP_GU] = shape(2 * F, d, 1);
  p.ops[FOP_DOWN] = shape(d, F, std::min(fast_down_split(c), n_cta));
  p.ops[FOP_HEAD] = shape(c.vocab_out, d, 1);

  // The tiles of an op (of each K slice of it) go to the slice's CTAs in contiguous runs; the CTAs
  // least loaded so far (streamed k-steps per layer) take the remainder, so that every CTA streams
  // about the same number of bytes.  The op with the finest grain (gate/up) is placed last.
  std::vector<std::vector<std::vector<int32_t>>> own(n_cta, std::vector<std::vector<int32_t>>(FOP_COUNT));
  std::vector<long long> load(n_cta, 0);
  const int order_ops[FOP_COUNT] = {FOP_DOWN, FOP_QKV, FOP_O, FOP_GU, FOP_HEAD};
  for (int oi = 0; oi < FOP_COUNT; ++oi) {
    const int op = order_ops[oi];
    const FastOpShape& s = p.ops[op];
    for (int slice = 0; slice < s.ksplit; ++slice) {
      std::vector<int> group;
      for (int cta = slice; cta < n_cta; cta += s.ksplit) group.push_back(cta);
      const int n = (int)group.size(), base = s.n_tiles / n, rem = s.n_tiles % n;
      std::stable_sort(group.begin(), group.end(), [&](int a, int b) { return load[a] < load[b]; });
      int next = 0;
      for (int i = 0; i < n; ++i) {
        const int cta = group[i], cnt = base + (i < rem ? 1 : 0);
        for (int j = 0; j < cnt; ++j) own[cta][op].push_back(next++);
        load[cta] += (long long)cnt * (fast_slice_k1(s, cta) - fast_slice_k0(s, cta));
      }
    }
  }
  p.unit_cnt.assign((size_t)n_cta * FOP_COUNT, 0);
  p.unit_off.assign((size_t)n_cta * FOP_COUNT, 0);
  for (int cta = 0; cta < n_cta; ++cta)
    for (int op = 0; op < FOP_COUNT; ++op) {
      p.unit_cnt[(size_t)cta * FOP_COUNT + op] = (int32_t)own[cta][op].size();
      p.unit_off[(size_t)cta * FOP_COUNT + op] = (int32_t)p.unit_tile.size();
      p.unit_tile.insert(p.unit_tile.end(), own[cta][op].begin(), own[cta][op].end());
    }

  // streams and their chunk tables
  const size_t nw = (size_t)n_cta * FAST_WARPS;
  p.stream_off.assign(nw, 0);
  p.chunks.assign(nw * FAST_MAX_CHUNKS, 0);
  p.chunk_cnt.assign(nw * 2, 0);
  uint64_t off = 0;
  for (int cta = 0; cta < n_cta; ++cta)
    for (int w = 0; w < FAST_WARPS; ++w) {
      const size_t i = (size_t)cta * FAST_WARPS + w;
      uint64_t tiles_layer = 0, tiles_head = 0;
      std::vector<uint8_t> ch_layer, ch_head;
      for (int op = 0; op < FOP_COUNT; ++op) {
        const int slice_steps = fast_slice_k1(p.ops[op], cta) - fast_slice_k0(p.ops[op], cta);
        const int ns = fast_warp_k1(w, slice_steps) - fast_warp_k0(w, slice_steps);
        const int cnt_total = (int)own[cta][op].size();
        std::vector<uint8_t>& ch = op == FOP_HEAD ? ch_head : ch_layer;
        if (p.ops[op].by_tile) {
          const int nt = fast_warp_tiles(w, cnt_total) * slice_steps;
          for (int t0 = 0; t0 < nt; t0 += FAST_O_CHUNK) ch.push_back((uint8_t)std::min(FAST_O_CHUNK, nt - t0));
          tiles_layer += (uint64_t)nt;
          continue;
        }
        for (int u0 = 0; u0 < cnt_total; u0 += FAST_MAXU) {
          const int cnt = std::min(FAST_MAXU, cnt_total - u0), spc = fast_steps_per_chunk(cnt);
          for (int s = 0; s < ns; s += spc) ch.push_back((uint8_t)(std::min(spc, ns - s) * cnt));
        }
        (op == FOP_HEAD ? tiles_head : tiles_layer) += (uint64_t)cnt_total * ns;
      }
      p.stream_off[i] = off;
      off += (tiles_layer * c.n_layers + tiles_head) * FAST_TILE_BYTES;
      p.chunk_cnt[i * 2 + 0] = (int32_t)ch_layer.size();
      p.chunk_cnt[i * 2 + 1] = (int32_t)ch_head.size();
      const int total = (int)(ch_layer.size() + ch_head.size());
      p.max_chunks = std::max(p.max_chunks, total);
      if (total <= FAST_MAX_CHUNKS) {
        std::copy(ch_layer.begin(), ch_layer.end(), p.chunks.begin() + i * FAST_MAX_CHUNKS);
        std::copy(ch_head.begin(), ch_head.end(), p.chunks.begin() + i * FAST_MAX_CHUNKS + ch_layer.size());
      }
    }
  p.total_bytes = off;
  return p;
}

namespace {

// One operand tile (8 packed rows from row0, k-step ks) to / from 256 bytes of a stream.
void emit_tile(const ssd_model_config& c, const BlobView& v, const uint16_t* blob, int op, int l, int row0,
               int ks, uint32_t* dst) {
  for (int g = 0; g < 8; ++g) {
    const uint16_t* row = packed_row(c, v, blob, op, l, row0 + g);
    for (int t = 0; t < 4; ++t) {
      uint32_t lo = 0, hi = 0;
      if (row) {
        const uint16_t* a = row + (size_t)ks * 16 + 2 * t;
        lo = (uint32_t)a[0] | ((uint32_t)a[1] << 16);
        hi = (uint32_t)a[8] | ((uint32_t)a[9] << 16);
      }
      dst[(g * 4 + t) * 2 + 0] = lo;
      dst[(g * 4 + t) * 2 + 1] = hi;
    }
  }
}
void scatter_tile(const ssd_model_config& c, const BlobView& v, uint16_t* blob_out, int op, int l, int row0,
                  int ks, const uint32_t* src) {
  for (int g = 0; g < 8; ++g) {
    uint16_t* row = const_cast<uint16_t*>(packed_row(c, v, blob_out, op, l, row0 + g));
    if (!row) continue;
    for (int t = 0; t < 4; ++t) {
      const uint32_t lo = src[(g * 4 + t) * 2], hi = src[(g * 4 + t) * 2 + 1];
      uint16_t* a = row + (size_t)ks * 16 + 2 * t;
      a[0] = (uint16_t)lo; a[1] = (uint16_t)(lo >> 16);
      a[8] = (uint16_t)hi; a[9] = (uint16_t)(hi >> 16);
    }
  }
}

}  // namespace

void fast_pack_streams(const ssd_model_config& c, const FastPlan& plan, const uint16_t* blob,
                       uint8_t* out) {
  const BlobView v = view_blob(c);
  for (int cta = 0; cta < plan.n_cta; ++cta)
    for (int w = 0; w < FAST_WARPS; ++w) {
      uint32_t* dst = reinterpret_cast<uint32_t*>(out + plan.stream_off[(size_t)cta * FAST_WARPS + w]);
      for (int l = 0; l <= c.n_layers; ++l) {
        const int op_begin = l < c.n_layers ? 0 : FOP_HEAD, op_end = l < c.n_layers ? FOP_HEAD : FOP_COUNT;
        const int ll = l < c.n_layers ? l : 0;
        for (int op = op_begin; op < op_end; ++op) {
          const FastOpShape& s = plan.ops[op];
          const int cnt = plan.unit_cnt[(size_t)cta * FOP_COUNT + op];
          const int32_t* tiles = plan.unit_tile.data() + plan.unit_off[(size_t)cta * FOP_COUNT + op];
          const int sk0 = fast_slice_k0(s, cta), slice_steps = fast_slice_k1(s, cta) - sk0;
          if (s.by_tile) {
            for (int u = w; u < cnt; u += FAST_WARPS)
              for (int ks = sk0; ks < sk0 + slice_steps; ++ks) {
                emit_tile(c, v, blob, op, ll, tiles[u] * 8, ks, dst);
                dst += FAST_TILE_BYTES / 4;
              }
            continue;
          }
          const int k0 = sk0 + fast_warp_k0(w, slice_steps), k1 = sk0 + fast_warp_k1(w, slice_steps);
          for (int u0 = 0; u0 < cnt; u0 += FAST_MAXU)
            for (int ks = k0; ks < k1; ++ks)
              for (int u = u0; u < std::min(cnt, u0 + FAST_MAXU); ++u) {
                emit_tile(c, v, blob, op, ll, tiles[u] * 8, ks, dst);
                dst += FAST_TILE_BYTES / 4;
              }
        }
      }
    }
}

// Inverse of fast_pack_streams, written as a consumer would walk the streams (chunk by chunk, a
// chunk being whole k-steps of one round, or a run of a warp's own tiles): scatters every tile
// back into a flat blob of the ssd_model_create layout.  Returns the number of chunks whose size
// disagrees with the walk.
long long fast_unpack_streams(const ssd_model_config& c, const FastPlan& plan, const uint8_t* streams,
                              uint16_t* blob_out) {
  const BlobView v = view_blob(c);
  long long bad = 0;
  for (int cta = 0; cta < plan.n_cta; ++cta)
    for (int w = 0; w < FAST_WARPS; ++w) {
      const size_t wi = (size_t)cta * FAST_WARPS + w;
      const uint8_t* tab = plan.chunks.data() + wi * FAST_MAX_CHUNKS;
      const int ncl = plan.chunk_cnt[wi * 2], nch = plan.chunk_cnt[wi * 2 + 1];
      const uint32_t* src = reinterpret_cast<const uint32_t*>(streams + plan.stream_off[wi]);
      for (int l = 0; l <= c.n_layers; ++l) {
        int ci = l < c.n_layers ? 0 : ncl;  // chunk cursor in the table
        const int op_begin = l < c.n_layers ? 0 : FOP_HEAD, op_end = l < c.n_layers ? FOP_HEAD : FOP_COUNT;
        const int ll = l < c.n_layers ? l : 0;
        for (int op = op_begin; op < op_end; ++op) {
          const FastOpShape& s = plan.ops[op];
          const int cnt_total = plan.unit_cnt[(size_t)cta * FOP_COUNT + op];
          const int32_t* tiles = plan.unit_tile.data() + plan.unit_off[(size_t)cta * FOP_COUNT + op];
          const int sk0 = fast_slice_k0(s, cta), steps = fast_slice_k1(s, cta) - sk0;
          if (s.by_tile) {
            int left = fast_warp_tiles(w, cnt_total) * steps, in_chunk = 0, u = w, ks = 0;
            while (left > 0) {
              if (in_chunk == 0) {
                in_chunk = std::min(FAST_O_CHUNK, left);
                if (tab[ci++] != in_chunk) ++bad;
              }
              scatter_tile(c, v, blob_out, op, ll, tiles[u] * 8, sk0 + ks, src);
              src += FAST_TILE_BYTES / 4;
              --in_chunk;
              --left;
              if (++ks == steps) {
                ks = 0;
                u += FAST_WARPS;
              }
            }
            continue;
          }
          const int s0 = sk0 + fast_warp_k0(w, steps), s1 = sk0 + fast_warp_k1(w, steps);
          for (int u0 = 0; u0 < cnt_total; u0 += FAST_MAXU) {
            const int cnt = std::min(FAST_MAXU, cnt_total - u0), spc = fast_steps_per_chunk(cnt);
            for (int sb = s0; sb < s1; sb += spc) {
              const int nst = std::min(spc, s1 - sb);
              if (tab[ci++] != nst * cnt) ++bad;
              for (int i = 0; i < nst; ++i)
                for (int u = 0; u < cnt; ++u) {
                  scatter_tile(c, v, blob_out, op, ll, tiles[u0 + u] * 8, sb + i, src);
                  src += FAST_TILE_BYTES / 4;
                }
            }
          }
        }
        if (l < c.n_layers ? ci != ncl : ci != ncl + nch) ++bad;
      }
    }
  return bad;
}

void fast_pack_aux(const ssd_model_config& c, const uint16_t* blob, std::vector<float>& bias,
                   std::vector<float>& gains) {
  const BlobView v = view_blob(c);
  const int d = c.d_model, qd = c.n_q_heads * c.head_dim, kvd = c.n_kv_heads * c.head_dim;
  const int nq = qd + 2 * kvd;
  bias.assign((size_t)c.n_layers * nq, 0.f);
  gains.assign((size_t)c.n_layers * 2 * d + d, 0.f);
  for (int l = 0; l < c.n_layers; ++l) {
    const BlobView::Layer& L = v.layers[l];
    float* b = bias.data() + (size_t)l * nq;
    for (int n = 0; n < qd; ++n) b[n] = bf16_bits_to_float(blob[L.bq + rope_unpack_row(n, c.head_dim)]);
    for (int n = 0; n < kvd; ++n) b[qd + n] = bf16_bits_to_float(blob[L.bk + rope_unpack_row(n, c.head_dim)]);
    for (int n = 0; n < kvd; ++n) b[qd + kvd + n] = bf16_bits_to_float(blob[L.bv + n]);
    float* g = gains.data() + (size_t)l * 2 * d;
    for (int j = 0; j < d; ++j) {
      g[j] = bf16_bits_to_float(blob[L.norm1 + j]);
      g[d + j] = bf16_bits_to_float(blob[L.norm2 + j]);
    }
  }
  float* gf = gains.data() + (size_t)c.n_layers * 2 * d;
  for (int j = 0; j < d; ++j) gf[j] = bf16_bits_to_float(blob[v.norm_f + j]);
}

}  // namespace ssd
