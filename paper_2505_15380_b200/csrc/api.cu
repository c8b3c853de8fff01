// C ABI of the SSD verify library: handles, argument checks, and the launch sequence of one
// decoder forward (Sec. 3.1 decoder; Eq. 4) followed by the acceptance kernel (Eq. 5-6).
#include <math.h>
#include <stdio.h>
#include <string.h>
#include <stdint.h>

#include <new>

#include "fast.h"
#include "kernels.h"
#include "tc.h"

using namespace ssd;

namespace {

thread_local char g_cuda_err[256] = "";

int cuda_fail(cudaError_t e, const char* what) {
  snprintf(g_cuda_err, sizeof(g_cuda_err), "%.120s: %.120s", what, cudaGetErrorString(e));
  return SSD_ERR_CUDA;
}
#define SSD_CUDA(call)                                  \
  do {                                                  \
    cudaError_t e_ = (call);                            \
    if (e_ != cudaSuccess) return cuda_fail(e_, #call); \
  } while (0)

inline size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

constexpr size_t PREFILL_ROWS = 64;  // least rows a bf16 streams object can run in one forward
// Streams with room for this many tokens run the persistent kernel's key-split variant: from a
// few hundred keys on, ten CTAs sharing a head's keys and meeting once costs less than each of
// them walking all keys (0.8 us per 128 keys and layer against ~1.5 us for the exchange).
constexpr int KEYSPLIT_MIN_CAPACITY = 768;

bool cfg_ok(const ssd_model_config* c) {
  if (!c) return false;
  if (c->n_layers < 1 || c->d_model < 8 || c->n_q_heads < 1 || c->n_kv_heads < 1) return false;
  if (c->head_dim != 32 && c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->n_q_heads % c->n_kv_heads) return false;
  if (c->n_q_heads / c->n_kv_heads > 16) return false;
  if ((c->d_model & 7) || (c->d_ffn & 7) || c->d_ffn < 8) return false;
  if (c->vocab_out < 2 || c->vocab_text < 0) return false;
  if ((size_t)c->vocab_out * 4 > 180 * 1024) return false;  // a logit row must fit in shared memory
  if (c->weight_dtype != 0 && c->weight_dtype != 1) return false;
  if (c->qkv_bias != 1) return false;
  if (!(c->rope_theta > 0.f) || !(c->rms_eps >= 0.f)) return false;
  return true;
}

struct LayerOff {
  size_t norm1, w_qkv, b_qkv, w_o, norm2, w_gu, w_d;
};
struct ArenaPlan {
  size_t embed, norm_f, head, inv_freq, total;
  std::vector<LayerOff> layers;
  // weights packed for the persistent small-batch kernel (bf16 models only)
  bool fast;
  size_t f_stream, f_stream_off, f_chunks, f_chunk_cnt, f_unit_cnt, f_unit_off, f_unit_tile, f_bias,
      f_gains;
  // weights packed for the tensor-core projections of batched forwards (bf16 models only)
  bool tc;
  std::vector<LayerOff> tc_layers;  // w_qkv, w_o, w_gu, w_d used
  size_t tc_head;
};

// CTAs of the persistent kernel: one per SM of the current device (148 when none is present, the
// SM count of a B200, so that sizes can be computed without a GPU).
int fast_cta_count() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
    cudaGetLastError();
    return 148;
  }
  return sms > FAST_MAX_CTAS ? FAST_MAX_CTAS : sms;
}

ArenaPlan plan_arena(const ssd_model_config& c, const FastPlan* fp = nullptr) {
  ArenaPlan p;
  size_t el = c.weight_dtype == 0 ? 4 : 2, off = 0;
  size_t d = c.d_model, qd = (size_t)c.n_q_heads * c.head_dim, kvd = (size_t)c.n_kv_heads * c.head_dim;
  size_t F = c.d_ffn;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  p.embed = take((size_t)(c.vocab_out + c.vocab_text) * d * el);
  p.layers.resize(c.n_layers);
  for (auto& L : p.layers) {
    L.norm1 = take(d * el);
    L.w_qkv = take((qd + 2 * kvd) * d * el);
    L.b_qkv = take((qd + 2 * kvd) * el);
    L.w_o = take(d * qd * el);
    L.norm2 = take(d * el);
    L.w_gu = take(2 * F * d * el);
    L.w_d = take(d * F * el);
  }
  p.norm_f = take(d * el);
  p.head = take((size_t)c.vocab_out * d * el);
  p.inv_freq = take((size_t)(c.head_dim / 2) * sizeof(double));
  p.fast = fast_supported(c);
  if (p.fast) {
    FastPlan local;
    if (!fp) {
      local = fast_make_plan(c, fast_cta_count());
      fp = &local;
    }
    const size_t nq = (size_t)(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
    p.f_stream = take(fp->total_bytes);
    p.f_stream_off = take(fp->stream_off.size() * 8);
    p.f_chunks = take(fp->chunks.size());
    p.f_chunk_cnt = take(fp->chunk_cnt.size() * 4);
    p.f_unit_cnt = take(fp->unit_cnt.size() * 4);
    p.f_unit_off = take(fp->unit_off.size() * 4);
    p.f_unit_tile = take(fp->unit_tile.size() * 4);
    p.f_bias = take((size_t)c.n_layers * nq * 4);
    p.f_gains = take(((size_t)c.n_layers * 2 + 1) * d * 4);
  }
  p.tc = c.weight_dtype == 1;
  if (p.tc) {
    p.tc_layers.resize(c.n_layers);
    for (auto& L : p.tc_layers) {
      L.w_qkv = take(tc_weight_bytes((int)(qd + 2 * kvd), (int)d));
      L.w_o = take(tc_weight_bytes((int)d, (int)qd));
      L.w_gu = take(tc_weight_bytes((int)(2 * F), (int)d));
      L.w_d = take(tc_weight_bytes((int)d, (int)F));
    }
    p.tc_head = take(tc_weight_bytes(c.vocab_out, (int)d));
  }
  p.total = off;
  return p;
}

size_t blob_elems(const ssd_model_config& c) {
  size_t d = c.d_model, qd = (size_t)c.n_q_heads * c.head_dim, kvd = (size_t)c.n_kv_heads * c.head_dim;
  size_t F = c.d_ffn;
  size_t per_layer = d + qd * d + qd + 2 * (kvd * d + kvd) + d * qd + d + 3 * F * d;
  return (size_t)(c.vocab_out + c.vocab_text) * d + per_layer * c.n_layers + d + (size_t)c.vocab_out * d;
}

struct WsPlan {
  size_t len, pending, status, counters, row_ids, accept_flags;
  size_t h, qkv, qrot, rope_cs, part, logits, row_stats, xn, attn_out, act;
  size_t st_tokens, st_k, st_y, st_probs, st_uni;
  size_t hfix, flags, epoch_base, xa, xb, xd, xq, ssq_a, ssq_b;
  size_t tc_xa, tc_xattn, tc_xact, tc_part;
  size_t attn_part, attn_cnt;
  size_t page_table, pages_used, free_stack, free_top;
  size_t total;
  int max_rows, nsplit_max;
};

WsPlan plan_ws(const ssd_model_config& c, int B, int max_gamma, int cap, int n_pages = 0, int max_pages = 0) {
  WsPlan p;
  size_t off = 0;
  size_t d = c.d_model, qd = (size_t)c.n_q_heads * c.head_dim, kvd = (size_t)c.n_kv_heads * c.head_dim;
  size_t F = c.d_ffn, V = c.vocab_out;
  size_t M = (size_t)B * (max_gamma + 1);
  // bf16 models: room for prefill chunks large enough for the tensor-core forward
  if (c.weight_dtype == 1 && M < PREFILL_ROWS) M = PREFILL_ROWS;
  p.max_rows = (int)M;
  p.nsplit_max = (cap + ATTN_CHUNK - 1) / ATTN_CHUNK;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  p.len = take(B * 4);
  p.pending = take(B * 4);
  p.status = take(4);
  p.counters = take(B * 4);
  p.row_ids = take(M * 4);
  p.accept_flags = take(M * 4);
  p.h = take(M * d * 4);
  p.qkv = take(M * (qd + 2 * kvd) * 4);
  p.qrot = take(M * qd * 4);
  p.rope_cs = take(M * c.head_dim * 4);
  p.part = take(M * c.n_q_heads * (size_t)p.nsplit_max * (c.head_dim + 2) * 4);
  p.logits = take(M * V * 4);
  p.row_stats = take(M * 8 * 4);  // eight statistics words per row (sampler.cu)
  p.xn = take(M * d * 4);
  p.attn_out = take(M * qd * 4);
  p.act = take(M * F * 4);
  // host-call staging: [tokens | uniforms] and [k | y] are each one contiguous run, so that the
  // host-buffer entry moves them with one copy each way
  p.st_tokens = take((size_t)B * max_gamma * 4 + M * 2 * 4);
  p.st_k = take((size_t)2 * B * 4);
  p.st_y = p.st_k + (size_t)B * 4;
  p.st_probs = take((size_t)B * max_gamma * V * 4);
  p.st_uni = p.st_tokens + (size_t)B * max_gamma * 4;
  p.hfix = take((size_t)FAST_MAX_T * d * 8);
  // operand-layout activations: per 16 columns 32 lanes x 32 bytes (16 rows, bf16 hi + lo)
  p.xa = take(d * 64);
  p.xb = take(d * 64);
  p.xq = take(qd * 64);
  p.xd = take(F * 64);
  p.ssq_a = take((d / 64 + 1) * FAST_MAX_T * 8);
  p.ssq_b = take((d / 64 + 1) * FAST_MAX_T * 8);
  p.flags = take(64);
  p.epoch_base = take(2 * 4);
  p.attn_part = p.attn_cnt = 0;
  if (fast_supported(c)) {  // key-split attention of the persistent kernel
    const int hps = c.n_q_heads / fast_o_split(c, fast_cta_count());
    p.attn_part = take((size_t)FAST_MAX_CTAS * hps * FAST_MAX_T * (c.head_dim + 2) * 4);
    p.attn_cnt = take((size_t)FAST_MAX_CTAS * 4);
  }
  p.page_table = p.pages_used = p.free_stack = p.free_top = 0;
  if (n_pages > 0) {
    p.page_table = take((size_t)B * max_pages * 4);
    p.pages_used = take((size_t)B * 4);
    p.free_stack = take((size_t)n_pages * 4);
    p.free_top = take(4);
  }
  p.tc_xa = p.tc_xattn = p.tc_xact = p.tc_part = 0;
  if (c.weight_dtype == 1 && M > FAST_MAX_T && M <= TC_MAX_ROWS) {
    const int Mpad = tc_round16((int)M), n_sm = fast_cta_count();
    // the row chunks of an operand depend on the rows of the forward: room for the largest
    size_t rows_max = 0;
    for (int mp = 16; mp <= Mpad; mp += 16) {
      const TcChunks ch = tc_chunks(mp);
      rows_max = std::max(rows_max, (size_t)ch.n * ch.rows);
    }
    p.tc_xa = take((size_t)((d + 15) / 16) * rows_max * 64);
    p.tc_xattn = take((size_t)((qd + 15) / 16) * rows_max * 64);
    p.tc_xact = take((size_t)((F + 15) / 16) * rows_max * 64);
    size_t part = 0;
    const int rows[3] = {(int)(qd + 2 * kvd), (int)d, (int)d}, ks[3] = {(int)d, (int)qd, (int)F};
    for (int i = 0; i < 3; ++i) {
      const size_t tiles = (rows[i] + TC_TILE_ROWS - 1) / TC_TILE_ROWS;
      for (int mp = 16; mp <= Mpad; mp += 16) {  // the K split depends on the rows of the forward
        const size_t b = (size_t)tc_ksplit(rows[i], ks[i], mp, n_sm) * mp * tiles * TC_TILE_ROWS * 4;
        part = b > part ? b : part;
      }
    }
    p.tc_part = take(part);
  }
  p.total = off;
  return p;
}

bool streams_args_ok(const ssd_model_config* c, int B, int max_gamma, int cap) {
  return cfg_ok(c) && B >= 1 && B <= 4096 && max_gamma >= 1 && max_gamma + 1 <= R_MAX &&
         cap >= max_gamma + 1 && cap <= (1 << 20);
}

bool same_shape(const ssd_model_config& a, const ssd_model_config& b) {
  return a.n_layers == b.n_layers && a.d_model == b.d_model && a.n_q_heads == b.n_q_heads &&
         a.n_kv_heads == b.n_kv_heads && a.head_dim == b.head_dim && a.d_ffn == b.d_ffn &&
         a.vocab_out == b.vocab_out && a.vocab_text == b.vocab_text &&
         a.weight_dtype == b.weight_dtype;
}

// One decoder forward over the rows described by rm (ids already in s->row_ids).  Appends the
// rows' K/V at len + r; when logits_out is non-null also runs the final norm and the LM head.
// The persistent kernel covers forwards of at most FAST_MAX_T rows over a bf16 model.
bool use_fast(const ssd_model* m, const ssd_streams* s, RowMap rm) {
  return m->fast.enabled && s->path == 0 && !s->paged && rm.nb * rm.R <= FAST_MAX_T;
}

int forward_fast(const ssd_model* m, ssd_streams* s, RowMap rm, const int32_t* row_ids,
                 const int32_t* draft_tokens, float* logits_out, cudaStream_t st) {
  const ssd_model_config& c = m->cfg;
  const ssd_fast_model& f = m->fast;
  FastParams p{};
  p.m.wstream = f.wstream;
  p.m.stream_off = f.stream_off;
  p.m.chunks = f.chunks;
  p.m.chunk_cnt = f.chunk_cnt;
  p.m.unit_cnt = f.unit_cnt;
  p.m.unit_off = f.unit_off;
  p.m.unit_tile = f.unit_tile;
  p.m.bias_qkv = f.bias_qkv;
  p.m.gains = f.gains;
  p.m.n_cta = f.n_cta;
  p.m.max_units = f.max_units;
  p.m.down_split = f.down_split;
  p.m.o_split = f.o_split;
  p.m.max_stage_k = f.max_stage_k;
  p.layer_map = f.layer_map;
  p.n_src_layers = f.n_src_layers;
  p.embed = (const bf16*)m->embed;
  p.inv_freq = m->inv_freq;
  p.L = c.n_layers;
  p.d = c.d_model;
  p.Hq = c.n_q_heads;
  p.Hkv = c.n_kv_heads;
  p.hd = c.head_dim;
  p.hd_shift = c.head_dim == 32 ? 5 : c.head_dim == 64 ? 6 : 7;
  p.F = c.d_ffn;
  p.V = c.vocab_out;
  p.vocab_in = c.vocab_out + c.vocab_text;
  p.eps = c.rms_eps;
  p.kv = (bf16*)s->kv;
  p.kv_layer_elems = s->kv_layer_elems;
  p.cap = s->cap;
  p.len = s->len;
  p.pending = s->pending;
  p.status = s->status;
  p.b0 = rm.b0;
  p.nb = rm.nb;
  p.R = rm.R;
  p.T = rm.nb * rm.R;
  p.row_ids = row_ids;
  p.draft_tokens = draft_tokens;
  p.hfix = s->hfix;
  p.rope_cs = s->rope_cs;
  p.xa = s->xa;
  p.xb = s->xb;
  p.xq = s->xq;
  p.xd = s->xd;
  p.ssq_a = s->ssq_a;
  p.ssq_b = s->ssq_b;
  p.logits = logits_out;
  p.flags = s->flags;
  p.epoch_base = s->epoch_base;
  p.attn_part = s->attn_part;
  p.attn_cnt = s->attn_cnt;
  p.key_split = s->key_split;
  p.split_act = s->split_act;
  p.trace = s->trace;
  p.trace_cap = s->trace_cap;
  SSD_CUDA(launch_fast_forward(p, st));
  return SSD_OK;
}

// Forwards of more than FAST_MAX_T rows over a bf16 model: projections on the tcgen05 tensor cores
// (each weight byte read once), attention on the warp-level tensor-core instruction.
bool use_tc(const ssd_model* m, const ssd_streams* s, RowMap rm) {
  const int M = rm.nb * rm.R;
  if (s->paged) return true;  // the paged cache exists on this path only (sizes checked at creation)
  return m->tc.enabled && s->path == 0 && s->tc_part && M > FAST_MAX_T && M <= TC_MAX_ROWS && M <= s->max_rows;
}

int forward_tc(const ssd_model* m, ssd_streams* s, RowMap rm, float* logits_out, cudaStream_t st) {
  const ssd_model_config& c = m->cfg;
  const int M = rm.nb * rm.R, Mpad = tc_round16(M), d = c.d_model;
  const int qd = c.n_q_heads * c.head_dim, kvd = c.n_kv_heads * c.head_dim, F = c.d_ffn, nq = qd + 2 * kvd;
  const int n_sm = m->tc.n_sm;
  auto ld_of = [](int rows) { return (rows + TC_TILE_ROWS - 1) / TC_TILE_ROWS * TC_TILE_ROWS; };
  const int ks_qkv = tc_ksplit(nq, d, M, n_sm), ks_o = tc_ksplit(d, qd, M, n_sm), ks_d = tc_ksplit(d, F, M, n_sm);
  // key splits of the attention: whole 64-key tiles, and no more CTAs in all than the SMs hold
  // at once (a second, partly filled wave would cost as much as the first)
  const int G = c.n_q_heads / c.n_kv_heads, rowgroups = (G * rm.R + 63) / 64;
  long long want = ((long long)tc_attention_ctas_per_sm(c.head_dim) * n_sm) /
                   ((long long)rm.nb * c.n_kv_heads * rowgroups);  // splits that still fit one wave
  if (want < 1) want = 1;
  long long kps = ((s->cap + want - 1) / want + 63) / 64 * 64;
  if (kps < 64) kps = 64;
  while ((s->cap + kps - 1) / kps > 128) kps += 64;  // the merge kernel's table of splits
  const int nsplit = (int)((s->cap + kps - 1) / kps);
  if (M > s->max_rows || M > TC_MAX_ROWS) return SSD_ERR_BAD_PARAM;
  if (s->paged)  // every stream of this forward owns pages for the rows it is about to append
    launch_page_ensure(s->len, rm, s->page_table, s->pages_used, s->free_stack, s->free_top, s->max_pages,
                       s->status, st);
  launch_embed(1, m->embed, c.vocab_out + c.vocab_text, d, s->row_ids, M, s->h, s->status, st);
  launch_rope_table(s->len, rm, m->inv_freq, c.head_dim / 2, s->rope_cs, st);
  const float* part = nullptr;
  int nsp = 0, ldp = 0;
  TcGemm g{};
  g.M = M;
  g.status = s->status;
  for (int l = 0; l < c.n_layers; ++l) {
    const LayerW& w = m->layers[l];
    const ssd_tc_layer& t = m->tc.layers[l];
    bf16* kv_layer = (bf16*)(s->kv + (size_t)l * s->kv_layer_elems * s->el);
    launch_tc_norm_pack(s->h, part, nsp, ldp, M, d, (const bf16*)w.norm1, c.rms_eps, s->tc_xa, st);
    g.w = t.w_qkv; g.a = s->tc_xa; g.n_rows = nq; g.K = d; g.ksplit = ks_qkv; g.epi = TC_EPI_PARTIAL; g.part = s->tc_part;
    SSD_CUDA(launch_tc_gemm(g, st));
    launch_tc_qkv_post(s->tc_part, ks_qkv, ld_of(nq), Mpad, (const bf16*)w.b_qkv, s->rope_cs, s->qrot, kv_layer,
                       s->len, rm, s->cap, c.n_q_heads, c.n_kv_heads, c.head_dim, s->page_table, s->max_pages,
                       s->status, st);
    SSD_CUDA(launch_tc_attention(s->qrot, kv_layer, s->len, rm, s->cap, c.n_q_heads, c.n_kv_heads, c.head_dim,
                                 s->part, nsplit, (int)kps, s->tc_xattn, Mpad, s->page_table, s->max_pages, s->attn_kernel,
                                 s->status, st));
    g.w = t.w_o; g.a = s->tc_xattn; g.n_rows = d; g.K = qd; g.ksplit = ks_o;
    SSD_CUDA(launch_tc_gemm(g, st));
    launch_tc_norm_pack(s->h, s->tc_part, ks_o, ld_of(d), M, d, (const bf16*)w.norm2, c.rms_eps, s->tc_xa, st);
    g.w = t.w_gu; g.a = s->tc_xa; g.n_rows = 2 * F; g.K = d; g.ksplit = 1; g.epi = TC_EPI_SWIGLU; g.act_out = s->tc_xact;
    SSD_CUDA(launch_tc_gemm(g, st));
    g.w = t.w_d; g.a = s->tc_xact; g.n_rows = d; g.K = F; g.ksplit = ks_d; g.epi = TC_EPI_PARTIAL;
    SSD_CUDA(launch_tc_gemm(g, st));
    part = s->tc_part;
    nsp = ks_d;
    ldp = ld_of(d);
  }
  if (logits_out) {
    launch_tc_norm_pack(s->h, part, nsp, ldp, M, d, (const bf16*)m->norm_f, c.rms_eps, s->tc_xa, st);
    g.w = m->tc.head; g.a = s->tc_xa; g.n_rows = c.vocab_out; g.K = d; g.ksplit = 1; g.epi = TC_EPI_STORE;
    g.out = logits_out; g.ldo = c.vocab_out;
    SSD_CUDA(launch_tc_gemm(g, st));
  }
  SSD_CUDA(cudaGetLastError());
  return SSD_OK;
}

int forward(const ssd_model* m, ssd_streams* s, RowMap rm, float* logits_out, cudaStream_t st) {
  if (s->paged) return forward_tc(m, s, rm, logits_out, st);
  if (use_fast(m, s, rm)) return forward_fast(m, s, rm, s->row_ids, nullptr, logits_out, st);
  if (use_tc(m, s, rm)) return forward_tc(m, s, rm, logits_out, st);
  const ssd_model_config& c = m->cfg;
  const int dt = c.weight_dtype, M = rm.nb * rm.R, d = c.d_model;
  const int qd = c.n_q_heads * c.head_dim, kvd = c.n_kv_heads * c.head_dim, F = c.d_ffn;
  launch_embed(dt, m->embed, c.vocab_out + c.vocab_text, d, s->row_ids, M, s->h, s->status, st);
  launch_rope_table(s->len, rm, m->inv_freq, c.head_dim / 2, s->rope_cs, st);
  for (int l = 0; l < c.n_layers; ++l) {
    const LayerW& w = m->layers[l];
    void* kv_layer = s->kv + (size_t)l * s->kv_layer_elems * s->el;
    launch_rmsnorm(dt, s->h, w.norm1, s->xn, M, d, c.rms_eps, st);
    SSD_CUDA(launch_gemm_simt(dt, EPI_STORE_F32, s->xn, d, w.w_qkv, w.b_qkv, s->qkv,
                              qd + 2 * kvd, M, qd + 2 * kvd, d, st));
    launch_qkv_post(dt, s->qkv, s->rope_cs, s->qrot, kv_layer, s->len, rm, s->cap, c.n_q_heads,
                    c.n_kv_heads, c.head_dim, s->status, st);
    SSD_CUDA(launch_attention_simt(dt, s->qrot, kv_layer, s->len, rm, s->cap, c.n_q_heads,
                                   c.n_kv_heads, c.head_dim, s->part, s->nsplit_max, s->attn_out,
                                   st));
    SSD_CUDA(launch_gemm_simt(dt, EPI_RESIDUAL, s->attn_out, qd, w.w_o, nullptr, s->h, d,
                              M, d, qd, st));
    launch_rmsnorm(dt, s->h, w.norm2, s->xn, M, d, c.rms_eps, st);
    SSD_CUDA(launch_gemm_simt(dt, EPI_SWIGLU, s->xn, d, w.w_gu, nullptr, s->act, F, M,
                              2 * F, d, st));
    SSD_CUDA(launch_gemm_simt(dt, EPI_RESIDUAL, s->act, F, w.w_d, nullptr, s->h, d, M, d,
                              F, st));
  }
  if (logits_out) {
    launch_rmsnorm(dt, s->h, m->norm_f, s->xn, M, d, c.rms_eps, st);
    SSD_CUDA(launch_gemm_simt(dt, EPI_STORE_F32, s->xn, d, m->head, nullptr, logits_out,
                              c.vocab_out, M, c.vocab_out, d, st));
  }
  SSD_CUDA(cudaGetLastError());
  return SSD_OK;
}

// One autoregressive step of the draft model for every stream (Eq. 2-3): feeds n_in ids per
// stream (ids [B, n_in], or null with n_in = 1: each stream's pending token), commits them, and
// draws x ~ p from the transformed last row.  Token and row are written with the given strides.
int draft_step_impl(ssd_model* draft, ssd_streams* ds, const int32_t* ids, int n_in, const float* uniform,
                    const ssd_verify_params* params, int32_t* out_token, int tok_stride, float* out_prob,
                    size_t prob_stride, cudaStream_t st) {
  const int V = draft->cfg.vocab_out;
  const RowMap rm{0, ds->B, n_in};
  int rc;
  if (use_fast(draft, ds, rm)) {  // explicit ids, or row 0 = pending when there are none
    rc = forward_fast(draft, ds, rm, ids, nullptr, ds->logits, st);
  } else {
    SSD_CUDA(cudaMemcpyAsync(ds->row_ids, ids ? ids : ds->pending, (size_t)ds->B * n_in * 4,
                             cudaMemcpyDeviceToDevice, st));
    rc = forward(draft, ds, rm, ds->logits, st);
  }
  if (rc != SSD_OK) return rc;
  launch_advance_all(ds->len, ds->B, n_in, ds->cap, ds->status, st);
  SSD_CUDA(launch_draft_sampler(ds->logits + (size_t)(n_in - 1) * V, n_in * V, V, uniform, ds->B,
                                1.0f / params->temperature, params->top_k, params->top_p, out_token, tok_stride, out_prob,
                                prob_stride, ds->pending, ds->status, st));
  return SSD_OK;
}

int params_ok(const ssd_streams* s, const ssd_verify_params* p, bool need_gamma) {
  if (!p) return SSD_ERR_NULL;
  if (need_gamma && (p->gamma < 1 || p->gamma > s->max_gamma)) return SSD_ERR_BAD_GAMMA;
  if (!(p->temperature > 0.f) || !isfinite(p->temperature)) return SSD_ERR_BAD_PARAM;
  if (!(p->beta >= 0.f) || !isfinite(p->beta)) return SSD_ERR_BAD_PARAM;
  if (!(p->top_p >= 0.f) || !isfinite(p->top_p)) return SSD_ERR_BAD_PARAM;
  if (p->ras_window < 0 || p->ras_window > 32 || (p->ras_window > 0 && (!p->dev_recent_tokens || !(p->ras_tau >= 0.f))))
    return SSD_ERR_BAD_PARAM;
  return SSD_OK;
}

}  // namespace

namespace ssd {
int report_cuda_error(cudaError_t e, const char* what) { return cuda_fail(e, what); }
}  // namespace ssd

extern "C" {

size_t ssd_model_arena_bytes(const ssd_model_config* cfg) {
  if (!cfg_ok(cfg)) return 0;
  return plan_arena(*cfg).total;
}

int ssd_model_create(const ssd_model_config* cfg, const void* host_weights, size_t nbytes,
                     void* dev_arena, size_t arena_bytes, ssd_model** out) {
  if (!cfg || !host_weights || !dev_arena || !out) return SSD_ERR_NULL;
  if (!cfg_ok(cfg)) return SSD_ERR_BAD_CONFIG;
  if ((uintptr_t)dev_arena & 255) return SSD_ERR_MISALIGNED;
  const ssd_model_config& c = *cfg;
  FastPlan fplan;
  const bool fast = fast_supported(c);
  if (fast) fplan = fast_make_plan(c, fast_cta_count());
  ArenaPlan p = plan_arena(c, fast ? &fplan : nullptr);
  const size_t el = c.weight_dtype == 0 ? 4 : 2;
  if (arena_bytes < p.total) return SSD_ERR_TOO_SMALL;
  if (nbytes != blob_elems(c) * el) return SSD_ERR_BAD_CONFIG;
  ssd_model* m = new (std::nothrow) ssd_model();
  if (!m) return SSD_ERR_CUDA;
  m->cfg = c;
  m->el = (int)el;
  m->arena = (char*)dev_arena;
  const char* src = (const char*)host_weights;
  char* A = m->arena;
  const size_t d = c.d_model, qd = (size_t)c.n_q_heads * c.head_dim, kvd = (size_t)c.n_kv_heads * c.head_dim;
  const size_t F = c.d_ffn;
  cudaError_t e = cudaSuccess;
  auto put = [&](size_t dst_off, size_t elems) {
    if (e == cudaSuccess) e = cudaMemcpy(A + dst_off, src, elems * el, cudaMemcpyHostToDevice);
    src += elems * el;
  };
  put(p.embed, (size_t)(c.vocab_out + c.vocab_text) * d);
  m->embed = A + p.embed;
  m->layers.resize(c.n_layers);
  for (int l = 0; l < c.n_layers; ++l) {
    const LayerOff& o = p.layers[l];
    put(o.norm1, d);
    put(o.w_qkv, qd * d);                        // wq
    put(o.b_qkv, qd);                            // bq
    put(o.w_qkv + qd * d * el, kvd * d);         // wk
    put(o.b_qkv + qd * el, kvd);                 // bk
    put(o.w_qkv + (qd + kvd) * d * el, kvd * d); // wv
    put(o.b_qkv + (qd + kvd) * el, kvd);         // bv
    put(o.w_o, d * qd);
    put(o.norm2, d);
    // gate and up rows interleaved (row 2j = gate_j, row 2j+1 = up_j) so that one thread / one
    // accumulator tile owns both halves of SiLU(gate) * up
    if (e == cudaSuccess)
      e = cudaMemcpy2D(A + o.w_gu, 2 * d * el, src, d * el, d * el, F, cudaMemcpyHostToDevice);
    src += F * d * el;
    if (e == cudaSuccess)
      e = cudaMemcpy2D(A + o.w_gu + d * el, 2 * d * el, src, d * el, d * el, F, cudaMemcpyHostToDevice);
    src += F * d * el;
    put(o.w_d, d * F);
    m->layers[l] = LayerW{A + o.norm1, A + o.w_qkv, A + o.b_qkv, A + o.w_o, A + o.norm2, A + o.w_gu, A + o.w_d};
  }
  put(p.norm_f, d);
  put(p.head, (size_t)c.vocab_out * d);
  m->norm_f = A + p.norm_f;
  m->head = A + p.head;
  std::vector<double> inv(c.head_dim / 2);
  for (int j = 0; j < c.head_dim / 2; ++j)
    inv[j] = pow((double)c.rope_theta, -2.0 * j / (double)c.head_dim);
  if (e == cudaSuccess)
    e = cudaMemcpy(A + p.inv_freq, inv.data(), inv.size() * sizeof(double), cudaMemcpyHostToDevice);
  m->inv_freq = (const double*)(A + p.inv_freq);
  if (fast && e == cudaSuccess) {
    // second copy of the projection weights, tiled and ordered for the persistent kernel
    std::vector<uint8_t> packed(fplan.total_bytes);
    std::vector<float> bias, gains;
    fast_pack_streams(c, fplan, (const uint16_t*)host_weights, packed.data());
    fast_pack_aux(c, (const uint16_t*)host_weights, bias, gains);
    auto up = [&](size_t dst_off, const void* srcp, size_t bytes) {
      if (e == cudaSuccess && bytes) e = cudaMemcpy(A + dst_off, srcp, bytes, cudaMemcpyHostToDevice);
    };
    up(p.f_stream, packed.data(), packed.size());
    up(p.f_stream_off, fplan.stream_off.data(), fplan.stream_off.size() * 8);
    up(p.f_chunks, fplan.chunks.data(), fplan.chunks.size());
    up(p.f_chunk_cnt, fplan.chunk_cnt.data(), fplan.chunk_cnt.size() * 4);
    up(p.f_unit_cnt, fplan.unit_cnt.data(), fplan.unit_cnt.size() * 4);
    up(p.f_unit_off, fplan.unit_off.data(), fplan.unit_off.size() * 4);
    up(p.f_unit_tile, fplan.unit_tile.data(), fplan.unit_tile.size() * 4);
    up(p.f_bias, bias.data(), bias.size() * 4);
    up(p.f_gains, gains.data(), gains.size() * 4);
    ssd_fast_model& f = m->fast;
    f.wstream = (const uint8_t*)(A + p.f_stream);
    f.stream_off = (const uint64_t*)(A + p.f_stream_off);
    f.chunks = (const uint8_t*)(A + p.f_chunks);
    f.chunk_cnt = (const int32_t*)(A + p.f_chunk_cnt);
    f.unit_cnt = (const int32_t*)(A + p.f_unit_cnt);
    f.unit_off = (const int32_t*)(A + p.f_unit_off);
    f.unit_tile = (const int32_t*)(A + p.f_unit_tile);
    f.bias_qkv = (const float*)(A + p.f_bias);
    f.gains = (const float*)(A + p.f_gains);
    f.n_cta = fplan.n_cta;
    f.n_src_layers = c.n_layers;
    f.down_split = fplan.ops[FOP_DOWN].ksplit;
    f.o_split = fplan.ops[FOP_O].ksplit;
    f.max_units = 0;
    for (int32_t v : fplan.unit_cnt) f.max_units = v > f.max_units ? v : f.max_units;
    int down_w = 0;
    for (int cta = 0; cta < fplan.n_cta; ++cta) {
      int w = (fast_slice_k1(fplan.ops[FOP_DOWN], cta) - fast_slice_k0(fplan.ops[FOP_DOWN], cta)) * 16;
      down_w = w > down_w ? w : down_w;
    }
    f.max_stage_k = c.d_model;
    if (c.n_q_heads * c.head_dim > f.max_stage_k) f.max_stage_k = c.n_q_heads * c.head_dim;
    if (down_w > f.max_stage_k) f.max_stage_k = down_w;
    f.enabled = f.max_units <= FAST_MAX_UNITS && fplan.max_chunks <= FAST_MAX_CHUNKS;
  }
  if (p.tc && e == cudaSuccess) {
    // third arrangement of the projection weights: 128-row tiles in the tensor cores' canonical
    // shared-memory layout, made on the device from the row-major copy
    ssd_tc_model& t = m->tc;
    t.n_sm = fast_cta_count();
    t.layers.resize(c.n_layers);
    auto pack = [&](const void* src, int rows, int K, size_t dst_off) {
      if (e == cudaSuccess) e = tc_pack_weights((const bf16*)src, rows, K, (uint8_t*)(A + dst_off), 0);
      return (const uint8_t*)(A + dst_off);
    };
    for (int l = 0; l < c.n_layers; ++l) {
      const LayerW& w = m->layers[l];
      const LayerOff& o = p.tc_layers[l];
      t.layers[l].w_qkv = pack(w.w_qkv, (int)(qd + 2 * kvd), (int)d, o.w_qkv);
      t.layers[l].w_o = pack(w.w_o, (int)d, (int)qd, o.w_o);
      t.layers[l].w_gu = pack(w.w_gu, (int)(2 * F), (int)d, o.w_gu);
      t.layers[l].w_d = pack(w.w_d, (int)d, (int)F, o.w_d);
    }
    t.head = pack(m->head, c.vocab_out, (int)d, p.tc_head);
    t.enabled = e == cudaSuccess;
  }
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    delete m;
    return cuda_fail(e, "ssd_model_create copy");
  }
  *out = m;
  return SSD_OK;
}

size_t ssd_model_inherited_arena_bytes(const ssd_model* source, int32_t n_layers) {
  if (!source || n_layers < 1 || n_layers > 4096) return 0;
  const ssd_model_config& c = source->cfg;
  const size_t nq = (size_t)(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim, d = c.d_model;
  return align_up((size_t)n_layers * 4) + align_up((size_t)n_layers * nq * 4) +
         align_up(((size_t)n_layers * 2 + 1) * d * 4);
}

int ssd_model_create_inherited(const ssd_model* source, const int32_t* host_layer_map, int32_t n_layers,
                               void* dev_arena, size_t arena_bytes, ssd_model** out) {
  if (!source || !host_layer_map || !dev_arena || !out) return SSD_ERR_NULL;
  if (n_layers < 1 || n_layers > 4096) return SSD_ERR_BAD_CONFIG;
  const ssd_model_config& c = source->cfg;
  for (int i = 0; i < n_layers; ++i)
    if (host_layer_map[i] < 0 || host_layer_map[i] >= c.n_layers) return SSD_ERR_BAD_CONFIG;
  if ((uintptr_t)dev_arena & 255) return SSD_ERR_MISALIGNED;
  if (arena_bytes < ssd_model_inherited_arena_bytes(source, n_layers)) return SSD_ERR_TOO_SMALL;
  ssd_model* m = new (std::nothrow) ssd_model(*source);  // same pointers: no weight is copied
  if (!m) return SSD_ERR_CUDA;
  m->cfg.n_layers = n_layers;
  m->arena = (char*)dev_arena;
  m->layers.resize(n_layers);
  if (source->tc.enabled) m->tc.layers.resize(n_layers);
  for (int i = 0; i < n_layers; ++i) {
    m->layers[i] = source->layers[host_layer_map[i]];
    if (source->tc.enabled) m->tc.layers[i] = source->tc.layers[host_layer_map[i]];
  }
  char* A = (char*)dev_arena;
  cudaError_t e = cudaMemcpy(A, host_layer_map, (size_t)n_layers * 4, cudaMemcpyHostToDevice);
  m->fast.layer_map = (const int32_t*)A;  // n_src_layers stays the source's
  if (source->fast.enabled) {
    // The persistent kernel indexes q/k/v biases and norm gains by the model's own layer number:
    // small arrays, gathered here in the new model's layer order (the weights themselves are walked
    // in place through the layer map).
    const size_t nq = (size_t)(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim, d = c.d_model;
    float* bias = (float*)(A + align_up((size_t)n_layers * 4));
    float* gains = (float*)((char*)bias + align_up((size_t)n_layers * nq * 4));
    for (int i = 0; i < n_layers && e == cudaSuccess; ++i) {
      const int src = host_layer_map[i];
      e = cudaMemcpy(bias + (size_t)i * nq, source->fast.bias_qkv + (size_t)src * nq, nq * 4, cudaMemcpyDeviceToDevice);
      if (e == cudaSuccess)
        e = cudaMemcpy(gains + (size_t)i * 2 * d, source->fast.gains + (size_t)src * 2 * d, 2 * d * 4,
                       cudaMemcpyDeviceToDevice);
    }
    if (e == cudaSuccess)  // the final norm follows the last source layer
      e = cudaMemcpy(gains + (size_t)n_layers * 2 * d, source->fast.gains + (size_t)source->fast.n_src_layers * 2 * d,
                     d * 4, cudaMemcpyDeviceToDevice);
    m->fast.bias_qkv = bias;
    m->fast.gains = gains;
  }
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    delete m;
    return cuda_fail(e, "ssd_model_create_inherited copy");
  }
  *out = m;
  return SSD_OK;
}

void ssd_model_destroy(ssd_model* m) { delete m; }

size_t ssd_kv_bytes(const ssd_model_config* cfg, int32_t batch, int32_t capacity_tokens) {
  if (!cfg_ok(cfg) || batch < 1 || capacity_tokens < 1) return 0;
  size_t el = cfg->weight_dtype == 0 ? 4 : 2;
  return (size_t)cfg->n_layers * batch * 2 * cfg->n_kv_heads * (size_t)capacity_tokens * cfg->head_dim * el;
}

size_t ssd_workspace_bytes(const ssd_model_config* cfg, int32_t batch, int32_t max_gamma,
                           int32_t capacity_tokens) {
  if (!streams_args_ok(cfg, batch, max_gamma, capacity_tokens)) return 0;
  return plan_ws(*cfg, batch, max_gamma, capacity_tokens).total;
}

}  // extern "C"

namespace {

// Shared by the contiguous (n_pages = 0) and the paged form.
int streams_create_impl(const ssd_model* m, int32_t batch, int32_t capacity_tokens, int32_t max_gamma,
                        int32_t n_pages, int32_t max_pages, void* dev_kv, size_t kv_bytes,
                        void* dev_workspace, size_t ws_bytes, ssd_streams** out);

}  // namespace

extern "C" {

int ssd_streams_create(const ssd_model* m, int32_t batch, int32_t capacity_tokens,
                       int32_t max_gamma, void* dev_kv, size_t kv_bytes, void* dev_workspace,
                       size_t ws_bytes, ssd_streams** out) {
  return streams_create_impl(m, batch, capacity_tokens, max_gamma, 0, 0, dev_kv, kv_bytes, dev_workspace,
                             ws_bytes, out);
}

size_t ssd_paged_kv_bytes(const ssd_model_config* cfg, int32_t n_pages) {
  if (!cfg_ok(cfg) || cfg->weight_dtype != 1 || n_pages < 1) return 0;
  return (size_t)cfg->n_layers * n_pages * 2 * cfg->n_kv_heads * TC_PAGE_TOKENS * cfg->head_dim * 2;
}

size_t ssd_paged_workspace_bytes(const ssd_model_config* cfg, int32_t batch, int32_t max_gamma,
                                 int32_t n_pages, int32_t max_pages_per_stream) {
  if (!cfg || cfg->weight_dtype != 1 || n_pages < 1 || max_pages_per_stream < 1 ||
      max_pages_per_stream > (1 << 14) ||
      !streams_args_ok(cfg, batch, max_gamma, max_pages_per_stream * TC_PAGE_TOKENS))
    return 0;
  const WsPlan p = plan_ws(*cfg, batch, max_gamma, max_pages_per_stream * TC_PAGE_TOKENS, n_pages,
                           max_pages_per_stream);
  return p.max_rows <= TC_MAX_ROWS ? p.total : 0;
}

int ssd_streams_create_paged(const ssd_model* m, int32_t batch, int32_t n_pages,
                             int32_t max_pages_per_stream, int32_t max_gamma, void* dev_kv,
                             size_t kv_bytes, void* dev_workspace, size_t ws_bytes, ssd_streams** out) {
  if (!m) return SSD_ERR_NULL;
  if (!m->tc.enabled || n_pages < 1 || max_pages_per_stream < 1 || max_pages_per_stream > (1 << 14))
    return SSD_ERR_BAD_CONFIG;
  return streams_create_impl(m, batch, max_pages_per_stream * TC_PAGE_TOKENS, max_gamma, n_pages,
                             max_pages_per_stream, dev_kv, kv_bytes, dev_workspace, ws_bytes, out);
}

int ssd_paged_state(ssd_streams* s, int32_t* host_pages_used, int32_t* host_free_pages,
                    int32_t* host_page_table, void* stream) {
  if (!s) return SSD_ERR_NULL;
  if (!s->paged) return SSD_ERR_BAD_CONFIG;
  cudaStream_t st = (cudaStream_t)stream;
  if (host_pages_used)
    SSD_CUDA(cudaMemcpyAsync(host_pages_used, s->pages_used, (size_t)s->B * 4, cudaMemcpyDeviceToHost, st));
  if (host_free_pages) SSD_CUDA(cudaMemcpyAsync(host_free_pages, s->free_top, 4, cudaMemcpyDeviceToHost, st));
  if (host_page_table)
    SSD_CUDA(cudaMemcpyAsync(host_page_table, s->page_table, (size_t)s->B * s->max_pages * 4,
                             cudaMemcpyDeviceToHost, st));
  SSD_CUDA(cudaStreamSynchronize(st));
  return SSD_OK;
}

}  // extern "C"

namespace {

int streams_create_impl(const ssd_model* m, int32_t batch, int32_t capacity_tokens, int32_t max_gamma,
                        int32_t n_pages, int32_t max_pages, void* dev_kv, size_t kv_bytes,
                        void* dev_workspace, size_t ws_bytes, ssd_streams** out) {
  if (!m || !dev_kv || !dev_workspace || !out) return SSD_ERR_NULL;
  if (!streams_args_ok(&m->cfg, batch, max_gamma, capacity_tokens)) return SSD_ERR_BAD_CONFIG;
  if (((uintptr_t)dev_kv & 255) || ((uintptr_t)dev_workspace & 255)) return SSD_ERR_MISALIGNED;
  const ssd_model_config& c = m->cfg;
  const bool paged = n_pages > 0;
  if (kv_bytes < (paged ? ssd_paged_kv_bytes(&c, n_pages) : ssd_kv_bytes(&c, batch, capacity_tokens)))
    return SSD_ERR_TOO_SMALL;
  WsPlan p = plan_ws(c, batch, max_gamma, capacity_tokens, n_pages, max_pages);
  if (paged && (p.max_rows > TC_MAX_ROWS || !p.tc_part)) return SSD_ERR_BAD_CONFIG;
  if (ws_bytes < p.total) return SSD_ERR_TOO_SMALL;
  SSD_CUDA(cudaMemset(dev_workspace, 0, p.total));
  if (paged) {  // all pages free (page 0 on top of the stack), block tables empty (-1)
    std::vector<int32_t> stack(n_pages);
    for (int i = 0; i < n_pages; ++i) stack[i] = n_pages - 1 - i;
    SSD_CUDA(cudaMemcpy((char*)dev_workspace + p.free_stack, stack.data(), (size_t)n_pages * 4,
                        cudaMemcpyHostToDevice));
    SSD_CUDA(cudaMemcpy((char*)dev_workspace + p.free_top, &n_pages, 4, cudaMemcpyHostToDevice));
    SSD_CUDA(cudaMemset((char*)dev_workspace + p.page_table, 0xFF, (size_t)batch * max_pages * 4));
  }
  SSD_CUDA(cudaDeviceSynchronize());
  ssd_streams* s = new (std::nothrow) ssd_streams();
  if (!s) return SSD_ERR_CUDA;
  s->cfg = c;
  s->el = c.weight_dtype == 0 ? 4 : 2;
  s->B = batch;
  s->cap = capacity_tokens;
  s->max_gamma = max_gamma;
  s->max_rows = p.max_rows;
  s->nsplit_max = p.nsplit_max;
  s->kv = (char*)dev_kv;
  s->kv_layer_elems = paged ? (size_t)n_pages * 2 * c.n_kv_heads * (size_t)TC_PAGE_TOKENS * c.head_dim
                            : (size_t)batch * 2 * c.n_kv_heads * (size_t)capacity_tokens * c.head_dim;
  s->paged = paged ? 1 : 0;
  s->n_pages = n_pages;
  s->max_pages = max_pages;
  char* W = (char*)dev_workspace;
  s->ws = W;
  s->ws_bytes = p.total;
  s->len = (int32_t*)(W + p.len);
  s->pending = (int32_t*)(W + p.pending);
  s->status = (int32_t*)(W + p.status);
  s->counters = (int32_t*)(W + p.counters);
  s->row_ids = (int32_t*)(W + p.row_ids);
  s->accept_flags = (int32_t*)(W + p.accept_flags);
  s->h = (float*)(W + p.h);
  s->qkv = (float*)(W + p.qkv);
  s->qrot = (float*)(W + p.qrot);
  s->rope_cs = (float*)(W + p.rope_cs);
  s->part = (float*)(W + p.part);
  s->logits = (float*)(W + p.logits);
  s->row_stats = (float*)(W + p.row_stats);
  s->xn = (float*)(W + p.xn);
  s->attn_out = (float*)(W + p.attn_out);
  s->act = (float*)(W + p.act);
  s->st_tokens = (int32_t*)(W + p.st_tokens);
  s->st_k = (int32_t*)(W + p.st_k);
  s->st_y = (int32_t*)(W + p.st_y);
  s->st_probs = (float*)(W + p.st_probs);
  s->st_uni = (float*)(W + p.st_uni);
  s->hfix = (long long*)(W + p.hfix);
  s->xa = (uint32_t*)(W + p.xa);
  s->xb = (uint32_t*)(W + p.xb);
  s->xq = (uint32_t*)(W + p.xq);
  s->xd = (uint32_t*)(W + p.xd);
  s->ssq_a = (long long*)(W + p.ssq_a);
  s->ssq_b = (long long*)(W + p.ssq_b);
  s->flags = (uint32_t*)(W + p.flags);
  s->epoch_base = (uint32_t*)(W + p.epoch_base);
  s->attn_part = p.attn_part ? (float*)(W + p.attn_part) : nullptr;
  s->attn_cnt = p.attn_part ? (uint32_t*)(W + p.attn_cnt) : nullptr;
  s->key_split = capacity_tokens >= KEYSPLIT_MIN_CAPACITY ? 1 : 0;
  s->tc_xa = p.tc_part ? (uint8_t*)(W + p.tc_xa) : nullptr;
  s->tc_xattn = p.tc_part ? (uint8_t*)(W + p.tc_xattn) : nullptr;
  s->tc_xact = p.tc_part ? (uint8_t*)(W + p.tc_xact) : nullptr;
  s->tc_part = p.tc_part ? (float*)(W + p.tc_part) : nullptr;
  s->page_table = paged ? (int32_t*)(W + p.page_table) : nullptr;
  s->pages_used = paged ? (int32_t*)(W + p.pages_used) : nullptr;
  s->free_stack = paged ? (int32_t*)(W + p.free_stack) : nullptr;
  s->free_top = paged ? (int32_t*)(W + p.free_top) : nullptr;
  if (paged) s->key_split = 0;
  s->path = 0;
  s->attn_kernel = 0;
  s->split_act = 1;
  s->trace = nullptr;
  s->trace_cap = 0;
  *out = s;
  return SSD_OK;
}

// Paged cache: after anything that may have lowered a length, the pages beyond it are returned.
void release_pages(ssd_streams* s, cudaStream_t st) {
  if (s->paged)
    launch_page_release(s->len, s->B, s->page_table, s->pages_used, s->free_stack, s->free_top, s->max_pages, st);
}

}  // namespace

extern "C" {

void ssd_streams_destroy(ssd_streams* s) {
  if (!s) return;
  if (s->copy_stream) {
    cudaStreamDestroy(s->copy_stream);
    cudaEventDestroy(s->ev_free);
    cudaEventDestroy(s->ev_probs);
    if (s->h_stage) cudaFreeHost(s->h_stage);
  }
  delete s;
}

int ssd_fast_plan_host(const ssd_model_config* cfg, int32_t n_cta, int64_t* out8) {
  if (!cfg || !out8) return SSD_ERR_NULL;
  if (!cfg_ok(cfg) || !fast_supported(*cfg) || n_cta < 1 || n_cta > FAST_MAX_CTAS) return SSD_ERR_BAD_CONFIG;
  const FastPlan p = fast_make_plan(*cfg, n_cta);
  int64_t mn = INT64_MAX, mx = 0;
  for (int cta = 0; cta < n_cta; ++cta) {
    const size_t lo = p.stream_off[(size_t)cta * FAST_WARPS];
    const size_t hi = cta + 1 < n_cta ? p.stream_off[(size_t)(cta + 1) * FAST_WARPS] : p.total_bytes;
    mn = (int64_t)(hi - lo) < mn ? (int64_t)(hi - lo) : mn;
    mx = (int64_t)(hi - lo) > mx ? (int64_t)(hi - lo) : mx;
  }
  int32_t mu = 0;
  for (int32_t v : p.unit_cnt) mu = v > mu ? v : mu;
  out8[0] = (int64_t)p.total_bytes;
  out8[1] = mn;
  out8[2] = mx;
  out8[3] = mu;
  out8[4] = p.max_chunks;
  out8[5] = p.ops[FOP_DOWN].ksplit;
  out8[6] = p.ops[FOP_O].ksplit;
  out8[7] = (int64_t)p.unit_tile.size();
  return SSD_OK;
}

int ssd_fast_pack_roundtrip_host(const ssd_model_config* cfg, int32_t n_cta, const void* host_weights,
                                 size_t nbytes, void* host_out, int64_t* bad_chunks) {
  if (!cfg || !host_weights || !host_out || !bad_chunks) return SSD_ERR_NULL;
  if (!cfg_ok(cfg) || !fast_supported(*cfg) || n_cta < 1 || n_cta > FAST_MAX_CTAS) return SSD_ERR_BAD_CONFIG;
  if (nbytes != blob_elems(*cfg) * 2) return SSD_ERR_BAD_CONFIG;
  const FastPlan p = fast_make_plan(*cfg, n_cta);
  std::vector<uint8_t> packed(p.total_bytes);
  fast_pack_streams(*cfg, p, (const uint16_t*)host_weights, packed.data());
  *bad_chunks = fast_unpack_streams(*cfg, p, packed.data(), (uint16_t*)host_out);
  return SSD_OK;
}

int ssd_forward(ssd_model* model, ssd_streams* s, const int32_t* dev_draft_tokens, int32_t gamma,
                float* dev_logits, void* stream) {
  if (!model || !s || !dev_draft_tokens || !dev_logits) return SSD_ERR_NULL;
  if (!same_shape(model->cfg, s->cfg)) return SSD_ERR_BAD_CONFIG;
  if (gamma < 1 || gamma > s->max_gamma) return SSD_ERR_BAD_GAMMA;
  cudaStream_t st = (cudaStream_t)stream;
  const RowMap rm{0, s->B, gamma + 1};
  if (use_fast(model, s, rm)) return forward_fast(model, s, rm, nullptr, dev_draft_tokens, dev_logits, st);
  launch_gather_verify_ids(s->pending, dev_draft_tokens, gamma, s->B, s->row_ids, st);
  return forward(model, s, rm, dev_logits, st);
}

int ssd_streams_set_attention_kernel(ssd_streams* s, int32_t which) {
  if (!s) return SSD_ERR_NULL;
  if (which < 0 || which > 2) return SSD_ERR_BAD_PARAM;
  s->attn_kernel = which;
  return SSD_OK;
}

int ssd_streams_set_activation_split(ssd_streams* s, int32_t on) {
  if (!s) return SSD_ERR_NULL;
  if (on != 0 && on != 1) return SSD_ERR_BAD_PARAM;
  s->split_act = on;
  return SSD_OK;
}

int ssd_streams_set_path(ssd_streams* s, int32_t path) {
  if (!s) return SSD_ERR_NULL;
  if (path != 0 && path != 1) return SSD_ERR_BAD_PARAM;
  s->path = path;
  return SSD_OK;
}

int ssd_streams_set_trace(ssd_streams* s, int64_t* dev_trace, int32_t ctas, int32_t events_per_cta) {
  if (!s) return SSD_ERR_NULL;
  if (dev_trace && (ctas < FAST_MAX_CTAS || events_per_cta < 1)) return SSD_ERR_TOO_SMALL;
  s->trace = (long long*)dev_trace;
  s->trace_cap = dev_trace ? events_per_cta : 0;
  return SSD_OK;
}

int ssd_kv_truncate(ssd_streams* s, const int32_t* host_len, const int32_t* host_pending,
                    void* stream) {
  if (!s || !host_len || !host_pending) return SSD_ERR_NULL;
  for (int b = 0; b < s->B; ++b)
    if (host_len[b] < 0 || host_len[b] > s->cap) return SSD_ERR_KV_OVERFLOW;
  cudaStream_t st = (cudaStream_t)stream;
  SSD_CUDA(cudaMemcpyAsync(s->len, host_len, s->B * 4, cudaMemcpyHostToDevice, st));
  SSD_CUDA(cudaMemcpyAsync(s->pending, host_pending, s->B * 4, cudaMemcpyHostToDevice, st));
  release_pages(s, st);
  SSD_CUDA(cudaStreamSynchronize(st));
  return SSD_OK;
}

int ssd_kv_restore(ssd_streams* s, const int32_t* dev_len, const int32_t* dev_pending, void* stream) {
  if (!s || !dev_len || !dev_pending) return SSD_ERR_NULL;
  launch_kv_restore(s->len, s->pending, dev_len, dev_pending, s->B, s->cap, (cudaStream_t)stream);
  release_pages(s, (cudaStream_t)stream);
  SSD_CUDA(cudaGetLastError());
  return SSD_OK;
}

int ssd_streams_get_state(ssd_streams* s, int32_t* host_len, int32_t* host_pending, void* stream) {
  if (!s) return SSD_ERR_NULL;
  cudaStream_t st = (cudaStream_t)stream;
  if (host_len) SSD_CUDA(cudaMemcpyAsync(host_len, s->len, s->B * 4, cudaMemcpyDeviceToHost, st));
  if (host_pending)
    SSD_CUDA(cudaMemcpyAsync(host_pending, s->pending, s->B * 4, cudaMemcpyDeviceToHost, st));
  SSD_CUDA(cudaStreamSynchronize(st));
  return SSD_OK;
}

int ssd_prefill(ssd_model* m, ssd_streams* s, const int32_t* dev_ids, const int32_t* host_offsets,
                void* stream) {
  if (!m || !s || !dev_ids || !host_offsets) return SSD_ERR_NULL;
  if (!same_shape(m->cfg, s->cfg)) return SSD_ERR_BAD_CONFIG;
  for (int b = 0; b < s->B; ++b) {
    int n = host_offsets[b + 1] - host_offsets[b];
    if (n < 0) return SSD_ERR_BAD_PARAM;  // 0: this stream takes no part (it keeps its state)
    if (n - 1 > s->cap) return SSD_ERR_KV_OVERFLOW;
  }
  cudaStream_t st = (cudaStream_t)stream;
  // rows per forward: as many as the workspace holds when the tensor-core forward can take them
  // (one stream at a time, the chunk's rows causal among themselves), else a verify step's worth
  int chunk = s->max_gamma + 1;
  if (m->tc.enabled && s->path == 0 && s->tc_part && s->max_rows > FAST_MAX_T)
    chunk = s->max_rows < TC_MAX_ROWS ? s->max_rows : TC_MAX_ROWS;
  for (int b = 0; b < s->B; ++b) {
    const int32_t* ids = dev_ids + host_offsets[b];
    int n = host_offsets[b + 1] - host_offsets[b];
    if (n == 0) continue;
    for (int done = 0; done < n - 1; done += chunk) {
      int rows = n - 1 - done < chunk ? n - 1 - done : chunk;
      SSD_CUDA(cudaMemcpyAsync(s->row_ids, ids + done, rows * 4, cudaMemcpyDeviceToDevice, st));
      int rc = forward(m, s, RowMap{b, 1, rows}, nullptr, st);
      if (rc != SSD_OK) return rc;
      launch_advance_len(s->len, s->pending, b, rows, ids, -1, st);
    }
    launch_advance_len(s->len, s->pending, b, 0, ids, n - 1, st);
  }
  SSD_CUDA(cudaGetLastError());
  return SSD_OK;
}

int ssd_draft_step(ssd_model* draft, ssd_streams* ds, const int32_t* dev_in_ids, int32_t n_in,
                   const float* dev_uniform, const ssd_verify_params* params,
                   int32_t* dev_out_token, float* dev_out_prob_row, void* stream) {
  if (!draft || !ds || !dev_in_ids || !dev_uniform || !dev_out_token || !dev_out_prob_row)
    return SSD_ERR_NULL;
  if (!same_shape(draft->cfg, ds->cfg)) return SSD_ERR_BAD_CONFIG;
  int rc = params_ok(ds, params, false);
  if (rc != SSD_OK) return rc;
  if (n_in < 1 || n_in > 2 || n_in > ds->max_gamma + 1) return SSD_ERR_BAD_PARAM;
  return draft_step_impl(draft, ds, dev_in_ids, n_in, dev_uniform, params, dev_out_token, 1, dev_out_prob_row,
                         (size_t)draft->cfg.vocab_out, (cudaStream_t)stream);
}

int ssd_iteration(ssd_model* target, ssd_streams* ts, ssd_model* draft, ssd_streams* ds,
                  const ssd_verify_params* params, const ssd_loop_io* io, void* stream) {
  if (!target || !ts || !draft || !ds || !io) return SSD_ERR_NULL;
  if (!io->dev_uniform_pool || !io->dev_iteration || !io->dev_in_ids || !io->dev_draft_tokens ||
      !io->dev_draft_probs || !io->dev_accepted_len || !io->dev_next_token || !io->dev_out_tokens ||
      !io->dev_out_count)
    return SSD_ERR_NULL;
  if (!same_shape(target->cfg, ts->cfg) || !same_shape(draft->cfg, ds->cfg)) return SSD_ERR_BAD_CONFIG;
  if (ts->B != ds->B || target->cfg.vocab_out != draft->cfg.vocab_out) return SSD_ERR_BAD_CONFIG;
  int rc = params_ok(ts, params, true);
  if (rc != SSD_OK) return rc;
  const int B = ts->B, gamma = params->gamma, V = target->cfg.vocab_out;
  if (ds->max_gamma < 1 || (size_t)gamma * B > (size_t)ds->max_rows * 2) return SSD_ERR_BAD_GAMMA;
  if (io->n_iterations < 1 || io->out_capacity < 1) return SSD_ERR_BAD_PARAM;
  cudaStream_t st = (cudaStream_t)stream;
  launch_loop_stage_uniforms(io->dev_uniform_pool, io->n_iterations, io->dev_iteration, B, gamma, ds->st_uni,
                             ts->st_uni, st);
  for (int i = 0; i < gamma; ++i) {  // Eq. 2-3: x_i ~ p_i = M_p(T_in, x_1..x_{i-1})
    rc = draft_step_impl(draft, ds, i == 0 ? io->dev_in_ids : nullptr, i == 0 ? 2 : 1, ds->st_uni + (size_t)i * B,
                         params, io->dev_draft_tokens + i, gamma, io->dev_draft_probs + (size_t)i * V,
                         (size_t)gamma * V, st);
    if (rc != SSD_OK) return rc;
  }
  rc = ssd_verify(target, ts, io->dev_draft_tokens, io->dev_draft_probs, ts->st_uni, params,
                  io->dev_accepted_len, io->dev_next_token, nullptr, stream);  // Eq. 4-6
  if (rc != SSD_OK) return rc;
  rc = ssd_kv_commit(ts, io->dev_accepted_len, io->dev_next_token, stream);
  if (rc != SSD_OK) return rc;
  launch_loop_finish(ds->len, ds->pending, ds->cap, io->dev_in_ids, io->dev_draft_tokens, gamma,
                     io->dev_accepted_len, io->dev_next_token, B, io->dev_out_tokens, io->out_capacity,
                     io->dev_out_count, io->dev_accept_log, io->n_iterations, io->dev_iteration,
                     params->ras_window > 0 ? const_cast<int32_t*>(params->dev_recent_tokens) : nullptr,
                     params->ras_window, ts->status, st);
  release_pages(ds, st);
  SSD_CUDA(cudaGetLastError());
  return SSD_OK;
}

}  // extern "C"

namespace {

// ssd_verify's body; `probs_ready` (may be null) is an event the acceptance kernel waits for: the
// host-buffer entry uploads the draft rows on a side stream while the forward, which does not
// read them, is already running.
// The draft rows of the host-buffer entry: an upload on a side stream that is enqueued only after
// the forward has been launched (the forward does not read them, and every call made before its
// launch delays its start), and that the acceptance kernel then waits for.
struct ProbsUpload {
  cudaStream_t side;
  const void* host_src;
  void* dev_dst;
  size_t bytes;
  cudaEvent_t dst_free;  // already recorded on the main stream: earlier readers of dev_dst are done
  cudaEvent_t ready;
};

int verify_impl(ssd_model* target, ssd_streams* s, const int32_t* dev_draft_tokens,
                const float* dev_draft_probs, const float* dev_uniforms, const ssd_verify_params* params,
                int32_t* dev_accepted_len, int32_t* dev_next_token, float* dev_logits_or_null,
                cudaStream_t st, const ProbsUpload* upload) {
  const int gamma = params->gamma;
  float* logits = dev_logits_or_null ? dev_logits_or_null : s->logits;
  const RowMap rm{0, s->B, gamma + 1};
  int rc;
  if (use_fast(target, s, rm)) {
    rc = forward_fast(target, s, rm, nullptr, dev_draft_tokens, logits, st);
  } else {
    launch_gather_verify_ids(s->pending, dev_draft_tokens, gamma, s->B, s->row_ids, st);
    rc = forward(target, s, rm, logits, st);
  }
  if (rc != SSD_OK) return rc;
  if (upload) {
    SSD_CUDA(cudaStreamWaitEvent(upload->side, upload->dst_free, 0));
    SSD_CUDA(cudaMemcpyAsync(upload->dev_dst, upload->host_src, upload->bytes, cudaMemcpyHostToDevice, upload->side));
    SSD_CUDA(cudaEventRecord(upload->ready, upload->side));
    SSD_CUDA(cudaStreamWaitEvent(st, upload->ready, 0));
  }
  SSD_CUDA(launch_verify_sampler(logits, target->cfg.vocab_out, dev_draft_tokens, dev_draft_probs,
                                 dev_uniforms, s->B, gamma, 1.0f / params->temperature,
                                 params->top_k, params->top_p, params->beta, params->ras_window, params->ras_tau,
                                 params->dev_recent_tokens, s->row_stats, s->accept_flags,
                                 s->counters, dev_accepted_len, dev_next_token, s->status, st));
  return SSD_OK;
}

}  // namespace

extern "C" {

int ssd_verify(ssd_model* target, ssd_streams* s, const int32_t* dev_draft_tokens,
               const float* dev_draft_probs, const float* dev_uniforms,
               const ssd_verify_params* params, int32_t* dev_accepted_len,
               int32_t* dev_next_token, float* dev_logits_or_null, void* stream) {
  if (!target || !s || !dev_draft_tokens || !dev_draft_probs || !dev_uniforms || !dev_accepted_len ||
      !dev_next_token)
    return SSD_ERR_NULL;
  if (!same_shape(target->cfg, s->cfg)) return SSD_ERR_BAD_CONFIG;
  int rc = params_ok(s, params, true);
  if (rc != SSD_OK) return rc;
  return verify_impl(target, s, dev_draft_tokens, dev_draft_probs, dev_uniforms, params, dev_accepted_len,
                     dev_next_token, dev_logits_or_null, (cudaStream_t)stream, nullptr);
}

int ssd_kv_commit(ssd_streams* s, const int32_t* dev_accepted_len, const int32_t* dev_next_token,
                  void* stream) {
  if (!s || !dev_accepted_len || !dev_next_token) return SSD_ERR_NULL;
  launch_kv_commit(s->len, s->pending, dev_accepted_len, dev_next_token, s->B, s->cap, s->max_gamma, s->status,
                   (cudaStream_t)stream);
  release_pages(s, (cudaStream_t)stream);  // the rejected positions' pages, if they filled any
  SSD_CUDA(cudaGetLastError());
  return SSD_OK;
}

int ssd_verify_host(ssd_model* target, ssd_streams* s, const int32_t* host_draft_tokens,
                    const float* host_draft_probs, const float* host_uniforms,
                    const ssd_verify_params* params, int32_t* host_accepted_len,
                    int32_t* host_next_token, void* stream) {
  if (!target || !s || !host_draft_tokens || !host_draft_probs || !host_uniforms ||
      !host_accepted_len || !host_next_token)
    return SSD_ERR_NULL;
  // every check ssd_verify makes comes first: nothing may be enqueued on an error, and the
  // staging buffers were sized from the streams' own shape
  if (!same_shape(target->cfg, s->cfg)) return SSD_ERR_BAD_CONFIG;
  int rc = params_ok(s, params, true);
  if (rc != SSD_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t B = s->B, g = params->gamma, V = s->cfg.vocab_out;
  if (!s->copy_stream) {  // side stream and events of the overlapped upload, made on first use
    SSD_CUDA(cudaStreamCreateWithFlags(&s->copy_stream, cudaStreamNonBlocking));
    SSD_CUDA(cudaEventCreateWithFlags(&s->ev_free, cudaEventDisableTiming));
    SSD_CUDA(cudaEventCreateWithFlags(&s->ev_probs, cudaEventDisableTiming));
    // pinned host staging for the small inputs and the two result arrays (host memory, not device)
    s->h_stage_in = (size_t)((char*)s->st_uni - (char*)s->st_tokens) + (size_t)s->max_rows * 2 * 4;
    SSD_CUDA(cudaHostAlloc((void**)&s->h_stage, s->h_stage_in + 2 * B * 4, cudaHostAllocDefault));
  }
  // The draft rows are by far the largest input and only the acceptance kernel reads them: they
  // travel on the side stream (after whatever still reads the staging buffer on `stream`), and
  // that copy is enqueued once the forward has been launched; the small inputs go ahead.
  SSD_CUDA(cudaEventRecord(s->ev_free, st));
  const ProbsUpload upload{s->copy_stream, host_draft_probs, s->st_probs, B * g * V * 4, s->ev_free, s->ev_probs};
  // tokens and uniforms: gathered in the pinned staging buffer (a few hundred bytes), one copy
  const size_t uni_off = (size_t)((char*)s->st_uni - (char*)s->st_tokens), uni_bytes = B * (g + 1) * 2 * 4;
  memcpy(s->h_stage, host_draft_tokens, B * g * 4);
  memcpy(s->h_stage + uni_off, host_uniforms, uni_bytes);
  SSD_CUDA(cudaMemcpyAsync(s->st_tokens, s->h_stage, uni_off + uni_bytes, cudaMemcpyHostToDevice, st));
  rc = verify_impl(target, s, s->st_tokens, s->st_probs, s->st_uni, params, s->st_k, s->st_y, nullptr, st, &upload);
  if (rc != SSD_OK) return rc;
  rc = ssd_kv_commit(s, s->st_k, s->st_y, stream);
  if (rc != SSD_OK) return rc;
  char* h_out = s->h_stage + s->h_stage_in;  // [k | y] come back with one copy
  SSD_CUDA(cudaMemcpyAsync(h_out, s->st_k, 2 * B * 4, cudaMemcpyDeviceToHost, st));
  SSD_CUDA(cudaStreamSynchronize(st));
  memcpy(host_accepted_len, h_out, B * 4);
  memcpy(host_next_token, h_out + B * 4, B * 4);
  return SSD_OK;
}

int ssd_last_status(ssd_streams* s, int32_t* status, void* stream) {
  if (!s || !status) return SSD_ERR_NULL;
  cudaStream_t st = (cudaStream_t)stream;
  SSD_CUDA(cudaMemcpyAsync(status, s->status, 4, cudaMemcpyDeviceToHost, st));
  SSD_CUDA(cudaMemsetAsync(s->status, 0, 4, st));
  SSD_CUDA(cudaStreamSynchronize(st));
  return SSD_OK;
}

size_t ssd_tc_gemm_scratch_bytes(int32_t M, int32_t n_rows, int32_t K) {
  if (M < 1 || M > TC_MAX_ROWS || n_rows < 1 || K < 8 || (K & 7)) return 0;
  return align_up(tc_weight_bytes(n_rows, K)) + align_up(tc_act_bytes(tc_round16(M), K));
}

int ssd_tc_gemm_check(const void* dev_w, const float* dev_x, int32_t M, int32_t n_rows, int32_t K,
                      int32_t ksplit, int32_t epilogue, void* dev_scratch, size_t scratch_bytes,
                      void* dev_out, int32_t* dev_status, void* stream) {
  if (!dev_w || !dev_x || !dev_scratch || !dev_out || !dev_status) return SSD_ERR_NULL;
  const size_t need = ssd_tc_gemm_scratch_bytes(M, n_rows, K);
  if (need == 0 || ksplit < 1 || ksplit > (K + 15) / 16 || epilogue < 0 || epilogue > 2 ||
      (epilogue != TC_EPI_PARTIAL && ksplit != 1) || (epilogue == TC_EPI_SWIGLU && (n_rows & 1)))
    return SSD_ERR_BAD_PARAM;
  if ((uintptr_t)dev_scratch & 255) return SSD_ERR_MISALIGNED;
  if (scratch_bytes < need) return SSD_ERR_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* wp = (uint8_t*)dev_scratch;
  uint8_t* ap = wp + align_up(tc_weight_bytes(n_rows, K));
  SSD_CUDA(tc_pack_weights((const bf16*)dev_w, n_rows, K, wp, st));
  launch_tc_pack_rows(dev_x, M, K, ap, st);
  TcGemm g{};
  g.w = wp;
  g.a = ap;
  g.n_rows = n_rows;
  g.K = K;
  g.M = M;
  g.ksplit = ksplit;
  g.epi = epilogue;
  g.part = (float*)dev_out;
  g.out = (float*)dev_out;
  g.ldo = n_rows;
  g.act_out = (uint8_t*)dev_out;
  g.status = dev_status;
  SSD_CUDA(launch_tc_gemm(g, st));
  return SSD_OK;
}

int ssd_streams_inject_failure(ssd_streams* s, void* stream) {
  if (!s) return SSD_ERR_NULL;
  cudaStream_t st = (cudaStream_t)stream;
  const uint32_t one = 1u;  // the sticky failure word next to the barrier's launch base
  SSD_CUDA(cudaMemcpyAsync(s->epoch_base + 1, &one, 4, cudaMemcpyHostToDevice, st));
  SSD_CUDA(cudaStreamSynchronize(st));
  return SSD_OK;
}

uint64_t ssd_kernel_launch_count(void) { return launch_count(); }

const char* ssd_last_cuda_error(void) { return g_cuda_err; }

const char* ssd_strerror(int code) {
  switch (code) {
    case SSD_OK: return "ok";
    case SSD_ERR_NULL: return "null pointer argument";
    case SSD_ERR_BAD_CONFIG: return "unsupported or inconsistent configuration";
    case SSD_ERR_BAD_GAMMA: return "gamma out of range";
    case SSD_ERR_KV_OVERFLOW: return "KV cache capacity exceeded";
    case SSD_ERR_MISALIGNED: return "buffer not 256-byte aligned";
    case SSD_ERR_TOO_SMALL: return "caller buffer too small";
    case SSD_ERR_CUDA: return "CUDA runtime error";
    case SSD_ERR_BAD_PARAM: return "parameter out of range";
  }
  return "unknown error";
}

}  // extern "C"
