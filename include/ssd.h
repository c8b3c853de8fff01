/*
 * ssd.h - C ABI of the B200 (sm_100a) verify step of Speech Speculative Decoding (SSD).
 *
 * One SSD iteration (Algorithm 1) drafts gamma speech tokens with a small model M_p, runs the
 * target model M_q once over them ("parallel verification", Eq. 4), accepts a prefix of the
 * draft with the tolerance test r_i < min(1, q_i(x_i)/p_i(x_i)) + beta (Eq. 5), and emits one
 * more token: a resample from normalize(max(0, q_i - p_i)) at the first rejection (Eq. 6) or a
 * bonus token from q_{gamma+1} when nothing was rejected.  This library is that hot path.
 * Letters follow the paper: p = DRAFT distribution, q = TARGET distribution.
 *
 * Conventions for every call
 *  - Pointers named dev_* are device pointers, host_* are host pointers.  `stream` is a
 *    cudaStream_t passed as void* (NULL = the legacy default stream).
 *  - All device memory (weights arena, KV cache, workspace, inputs, outputs) is allocated and
 *    owned by the caller; handles returned by *_create are small host objects freed by *_destroy.
 *    The library never frees or reallocates caller memory and keeps the pointers it was given
 *    until the handle is destroyed.
 *  - Calls that take a stream only enqueue work on it and return without synchronising, unless
 *    stated otherwise.  Inputs are read-only.
 *  - Return value: SSD_OK (0) or a negative SSD_ERR_* code; nothing is enqueued on error.
 *    Conditions only the device can see (cache overflow, bad token id, non-finite logits) set
 *    bits of a device status word read back by ssd_last_status; kernels always terminate and
 *    never touch memory outside the buffers they were given.
 *
 * Stream state: a stream (utterance) whose prefix T_in has n tokens keeps K/V for tokens
 * 0..n-2 (`len` = n-1) and token n-1 as `pending`.  ssd_verify feeds [pending, x_1..x_gamma] at
 * positions len..len+gamma and writes their K/V; ssd_kv_commit makes k+1 of them permanent.
 * Rolling back rejected positions is O(1): slots at or beyond `len` are dead and get
 * overwritten by the next step.
 *
 * KV cache layout (caller-owned buffer of ssd_kv_bytes bytes), storage type = weight_dtype:
 *     kv[layer][stream][2 (0 = K, 1 = V)][kv_head][capacity][head_dim]
 * K is stored after the rotary embedding.
 */
#ifndef SSD_H_
#define SSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ssd_model ssd_model;     /* packed weights of one decoder (target or draft) */
typedef struct ssd_streams ssd_streams; /* B streams' KV cache descriptors, len[], pending[] */

enum {
  SSD_OK = 0,
  SSD_ERR_NULL = -1,        /* a required pointer was NULL */
  SSD_ERR_BAD_CONFIG = -2,  /* unsupported or inconsistent model / stream configuration */
  SSD_ERR_BAD_GAMMA = -3,   /* gamma outside 1..max_gamma given at ssd_streams_create */
  SSD_ERR_KV_OVERFLOW = -4, /* a length would exceed the cache capacity */
  SSD_ERR_MISALIGNED = -5,  /* a buffer is not aligned as required (256 bytes for arenas) */
  SSD_ERR_TOO_SMALL = -6,   /* a caller buffer is smaller than the *_bytes call reports */
  SSD_ERR_CUDA = -7,        /* a CUDA runtime call failed; see ssd_last_cuda_error */
  SSD_ERR_BAD_PARAM = -8    /* temperature <= 0, beta < 0, n_in out of range, ... */
};

/* bits of the device status word (ssd_last_status) */
enum {
  SSD_STATUS_KV_OVERFLOW = 1, /* len + rows > capacity: rows beyond capacity were not written */
  SSD_STATUS_BAD_TOKEN = 2,   /* a token id outside the embedding table was clamped; a draft token
                                 outside the vocabulary was rejected; ssd_kv_commit was handed an
                                 accepted length outside 0..max_gamma and left that stream alone */
  SSD_STATUS_NONFINITE = 4,   /* a logit row held NaN/Inf */
  SSD_STATUS_BAD_PROB = 8,    /* a draft probability p_i(x_i) was negative or not finite: rejected */
  SSD_STATUS_TIMEOUT = 16     /* a bounded wait inside a kernel ran out; the streams object refuses
                                 further small-batch launches until it is created anew */
};

/* Decoder shape: the "Transformer adapted from Qwen2.5" of Sec. 3.1 (pre-norm RMSNorm, GQA with
 * biased q/k/v projections, rotate-half RoPE, SiLU-gated FFN, final RMSNorm, untied head). */
typedef struct {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn;
  int32_t vocab_out;    /* speech vocabulary = rows of the LM head */
  int32_t vocab_text;   /* extra embedding rows [vocab_out, vocab_out + vocab_text) for text ids */
  float rope_theta, rms_eps;
  int32_t weight_dtype; /* 0 = fp32, 1 = bf16; the KV cache uses the same type */
  int32_t qkv_bias;     /* must be 1 (the blob always carries q/k/v biases) */
} ssd_model_config;

/* Per-call parameters of the sampler and of the acceptance rule. */
typedef struct {
  int32_t gamma;     /* draft length L_d of Algorithm 1 */
  float temperature; /* > 0; logits are divided by it */
  int32_t top_k;     /* <= 0 or >= vocab_out: off; else keep the top_k largest (lower id wins ties) */
  float beta;        /* tolerance factor of Eq. 5, >= 0 */
  float top_p;       /* nucleus: 0 or >= 1: off; else, among the ids top_k kept, most probable first
                        (lower id first among equals), an id stays while the mass before it is
                        below top_p: the shortest such prefix whose mass reaches top_p */
  /* Repetition-aware sampling of the TARGET (the sampler of the CosyVoice family; the paper is
   * silent): a nucleus / top-k draw that occurs at least ras_window * ras_tau times among the last
   * ras_window tokens is thrown away and redrawn from the full softmax.  The acceptance step uses
   * the distribution this procedure samples from, q(x) = q_nuc(x) [x not repeated] + R q_full(x)
   * with R = the nucleus mass of the repeated ids, as q_i in Eq. 5-6.  ras_window 0: off (at
   * most 32).  dev_recent_tokens: int32 [B, ras_window], the last tokens of each stream's T_in,
   * oldest first, the pending token last, -1 where the history is shorter; row i of a verify step
   * uses the last ras_window tokens of that followed by x_1..x_{i-1}.  ssd_iteration keeps the
   * array up to date (it appends the emitted tokens); ssd_draft_step ignores these fields. */
  int32_t ras_window;
  float ras_tau;
  const int32_t* dev_recent_tokens;
} ssd_verify_params;

/* ---- model ------------------------------------------------------------------------------- */

/* Bytes of device memory the packed model needs (0 if cfg is invalid). */
size_t ssd_model_arena_bytes(const ssd_model_config* cfg);

/* Packs a model into dev_arena (256-byte aligned, >= ssd_model_arena_bytes) and returns a handle.
 * host_weights is a flat blob of nbytes in this order, every element in weight_dtype:
 *   embed[vocab_out+vocab_text, d];
 *   per layer: norm1[d], wq[Hq*hd, d], bq[Hq*hd], wk[Hkv*hd, d], bk, wv[Hkv*hd, d], bv,
 *              wo[d, Hq*hd], norm2[d], w_gate[F, d], w_up[F, d], w_down[d, F];
 *   norm_f[d]; head[vocab_out, d].            (all matrices row-major [out, in])
 * Synchronous: returns after the copies finished; the blob may be freed afterwards. */
int ssd_model_create(const ssd_model_config* cfg, const void* host_weights, size_t nbytes,
                     void* dev_arena, size_t arena_bytes, ssd_model** out);
void ssd_model_destroy(ssd_model* m);

/* A model made of layers of another one, WITHOUT copying them: layer i of the new model is layer
 * host_layer_map[i] of `source`; embedding, final norm and LM head are the source's.  This is the
 * shape of the paper's draft model (Sec. 2.3: a shallower copy of the target built from its own
 * layers - in the experiments the target's lower two and upper six of 24 - before fine-tuning):
 * the draft pass then re-reads weights the verify pass has just pulled through L2 and adds no
 * weight memory.  dev_arena (256-byte aligned, ssd_model_inherited_arena_bytes) receives the map and
 * the new model's own copies of the small per-layer vectors (q/k/v biases, norm gains); `source`
 * and its arena must outlive the new handle.  Streams for it are created as for any model. */
size_t ssd_model_inherited_arena_bytes(const ssd_model* source, int32_t n_layers);
int ssd_model_create_inherited(const ssd_model* source, const int32_t* host_layer_map, int32_t n_layers,
                               void* dev_arena, size_t arena_bytes, ssd_model** out);

/* ---- streams ----------------------------------------------------------------------------- */

size_t ssd_kv_bytes(const ssd_model_config* cfg, int32_t batch, int32_t capacity_tokens);
size_t ssd_workspace_bytes(const ssd_model_config* cfg, int32_t batch, int32_t max_gamma,
                           int32_t capacity_tokens);

/* Binds `batch` streams of `capacity_tokens` cache slots each to caller buffers dev_kv and
 * dev_workspace (both 256-byte aligned).  The workspace holds len[], pending[], the status word
 * and all scratch of the kernels; it is zeroed here (synchronously), the KV buffer is not. */
int ssd_streams_create(const ssd_model* m, int32_t batch, int32_t capacity_tokens,
                       int32_t max_gamma, void* dev_kv, size_t kv_bytes, void* dev_workspace,
                       size_t ws_bytes, ssd_streams** out);
void ssd_streams_destroy(ssd_streams* s);

/* Paged form of the cache (bf16 models): instead of one slice of `capacity` slots per stream, all
 * streams draw 64-token pages from one pool, so that short and long utterances share memory and a
 * stream that ends hands its pages to the next one.  Pool layout (caller-owned, ssd_paged_kv_bytes):
 *     kv[layer][page][2 (0 = K, 1 = V)][kv_head][64][head_dim]
 * Token t of stream b lives in page table[b][t / 64], slot t % 64; the tables and the free-page
 * stack are device arrays inside the workspace, maintained by the library's kernels: a forward
 * first takes pages for the rows it appends, and every call that can lower a length (ssd_kv_commit,
 * ssd_kv_truncate, ssd_kv_restore) returns the pages that lie wholly beyond the new length - the
 * O(1) rollback of rejected positions, without moving data.  A stream leaves by being truncated to
 * length 0 and joins by a prefill (ssd_prefill accepts streams with no ids: they keep their state).
 * A stream may hold at most max_pages_per_stream pages (its capacity is 64 times that); if the pool
 * or a table is exhausted the rows that found no page are dropped and SSD_STATUS_KV_OVERFLOW is set.
 * All forwards of paged streams run on the batched tensor-core path; batch * (max_gamma + 1) must
 * not exceed 512 rows.  Everything else (verify, draft step, commit, the loop) is called as usual. */
size_t ssd_paged_kv_bytes(const ssd_model_config* cfg, int32_t n_pages);
size_t ssd_paged_workspace_bytes(const ssd_model_config* cfg, int32_t batch, int32_t max_gamma,
                                 int32_t n_pages, int32_t max_pages_per_stream);
int ssd_streams_create_paged(const ssd_model* m, int32_t batch, int32_t n_pages,
                             int32_t max_pages_per_stream, int32_t max_gamma, void* dev_kv,
                             size_t kv_bytes, void* dev_workspace, size_t ws_bytes, ssd_streams** out);
/* Pages each stream holds (int32 [B]), pages on the free stack, and the block tables
 * (int32 [B, max_pages_per_stream], -1 = none); any output may be NULL.  Synchronises `stream`. */
int ssd_paged_state(ssd_streams* s, int32_t* host_pages_used, int32_t* host_free_pages,
                    int32_t* host_page_table, void* stream);

/* Which kernels run the decoder forward (Eq. 4) for these streams.  path 0 (default): forwards of
 * at most 16 rows over a bf16 model run in one persistent kernel (one CTA per SM, weights streamed
 * through shared-memory rings), larger ones in the generic per-operation kernels; path 1: generic
 * kernels only.  Both produce the same results up to fp32 summation order. */
int ssd_streams_set_path(ssd_streams* s, int32_t path);

/* Diagnostics of the batched forward (more than 16 rows, or a paged cache): which kernel computes
 * the attention of Eq. 4.  0 (default): the tcgen05 kernel where a CTA's key range is long
 * enough to pay for its set-up (1024 keys or more; head sizes 64 and 128), else the warp-level
 * tensor-core kernel; 1: the warp-level kernel always; 2: the tcgen05 kernel wherever the head
 * size allows.  Both produce the same results up to fp32 summation order. */
int ssd_streams_set_attention_kernel(ssd_streams* s, int32_t which);

/* Precision of the activations that enter the tensor cores in the persistent kernel (weights and
 * K/V are bf16 as stored, accumulation is fp32, the residual stream is kept in fixed point, in
 * both modes).  on = 1 (default): each activation enters as its bf16 leading part plus the bf16
 * remainder, which agrees with a float64 evaluation of the 24-layer model to about 5e-4 in the
 * logits.  on = 0: each activation is rounded to bf16, the arithmetic of ordinary bf16 inference;
 * the logits then differ from a float64 evaluation by up to a few 1e-2. */
int ssd_streams_set_activation_split(ssd_streams* s, int32_t on);

/* Phase trace of the persistent kernel (a profiling aid, not part of the method).  With a device
 * buffer of ctas x events_per_cta int64 (ctas >= 256), thread 0 of every CTA stores its SM clock
 * (clock64) at each phase boundary of every later small-batch forward: after set-up, after the
 * embedding, after its grid barrier, then after each phase (per layer QKV, attention, O, gate/up,
 * down; finally the LM head) and after the barrier that follows it.  Event i of CTA c lands at
 * dev_trace[c * events_per_cta + i]; later launches overwrite earlier ones.  Clocks of different
 * SMs are not synchronised: compare within a CTA.  dev_trace = NULL turns the trace off. */
int ssd_streams_set_trace(ssd_streams* s, int64_t* dev_trace, int32_t ctas, int32_t events_per_cta);

/* Explicit rollback / state load: len[b] = host_len[b], pending[b] = host_pending[b].
 * O(1) per stream, no cache data moves.  Synchronous with respect to `stream`. */
int ssd_kv_truncate(ssd_streams* s, const int32_t* host_len, const int32_t* host_pending,
                    void* stream);
/* Same rollback with DEVICE arrays (int32 [B] each), enqueued on `stream` without synchronising:
 * the form a serving loop uses to discard a step or to re-run one from a saved state. */
int ssd_kv_restore(ssd_streams* s, const int32_t* dev_len, const int32_t* dev_pending, void* stream);
/* Reads len[] and pending[] back (either output may be NULL).  Synchronises `stream`. */
int ssd_streams_get_state(ssd_streams* s, int32_t* host_len, int32_t* host_pending, void* stream);

/* Loads prefixes T_in through the model: stream b receives ids dev_ids[host_offsets[b] ..
 * host_offsets[b+1]), appended after its current len.  K/V are written for all but the last id,
 * which becomes `pending`; a stream with no ids is left as it is.  Enqueues work only. */
int ssd_prefill(ssd_model* m, ssd_streams* s, const int32_t* dev_ids, const int32_t* host_offsets,
                void* stream);

/* ---- the SSD iteration ------------------------------------------------------------------- */

/* Draft generation (Algorithm 1, the lines that produce p_i and x_i ~ p_i; Eq. 2-3), one
 * autoregressive step of the draft model for every stream: feeds n_in (1 or 2) tokens
 * dev_in_ids[b, 0..n_in) at positions len[b].., commits them (len += n_in), applies the
 * sampling transform to the last row's logits and draws x ~ p with dev_uniform[b].
 * n_in = 2 serves the step after a fully accepted iteration, when the draft has no K/V yet for
 * x_gamma.  Outputs: dev_out_token[b], and the full row p (float [B, vocab_out]) the token was
 * drawn from, as Eq. 5-6 need it.  `pending` of the draft streams is set to the drawn token. */
int ssd_draft_step(ssd_model* draft, ssd_streams* draft_streams, const int32_t* dev_in_ids,
                   int32_t n_in, const float* dev_uniform, const ssd_verify_params* params,
                   int32_t* dev_out_token, float* dev_out_prob_row, void* stream);

/* Parallel verification and acceptance (Algorithm 1 from the M_q line to the bonus token;
 * Eq. 4-6) for all B streams:
 *   in  dev_draft_tokens int32 [B, gamma]       x_1..x_gamma
 *       dev_draft_probs  float [B, gamma, V]    rows p_i the tokens were drawn from
 *       dev_uniforms     float [B, gamma+1, 2]  [..,0] = r_i of Eq. 5 (row gamma unused),
 *                                               [..,1] = uniform of the categorical draw made
 *                                               at that row (resample at row i, bonus at gamma)
 *   out dev_accepted_len int32 [B]   k in [0, gamma]: draft tokens accepted
 *       dev_next_token   int32 [B]   the resampled (k < gamma) or bonus (k = gamma) token
 *       dev_logits_or_null float [B, gamma+1, V]  raw target logits, for parity checks
 * Writes provisional K/V at slots len..len+gamma; len/pending change only in ssd_kv_commit.
 * All uniforms must lie in [0, 1). */
int ssd_verify(ssd_model* target, ssd_streams* s, const int32_t* dev_draft_tokens,
               const float* dev_draft_probs, const float* dev_uniforms,
               const ssd_verify_params* params, int32_t* dev_accepted_len,
               int32_t* dev_next_token, float* dev_logits_or_null, void* stream);

/* The decoder forward of Eq. 4 alone: feeds [pending, x_1..x_gamma] of every stream at positions
 * len..len+gamma, writes their provisional K/V and the raw target logits float [B, gamma+1, V];
 * no acceptance step.  (ssd_verify = this followed by the acceptance kernel.) */
int ssd_forward(ssd_model* target, ssd_streams* s, const int32_t* dev_draft_tokens, int32_t gamma,
                float* dev_logits, void* stream);

/* Same step with HOST buffers: copies the three inputs to the device, runs ssd_verify and
 * ssd_kv_commit, copies accepted_len / next_token back and synchronises `stream`.  The draft rows
 * (by far the largest input, read only by the acceptance step) are uploaded on a side stream
 * while the forward runs, so host_draft_probs should be pinned; the small arrays travel through
 * a pinned staging buffer of a few hundred bytes.  The first call on a streams object creates
 * that side stream, two events and the staging buffer (host memory; no device allocation). */
int ssd_verify_host(ssd_model* target, ssd_streams* s, const int32_t* host_draft_tokens,
                    const float* host_draft_probs, const float* host_uniforms,
                    const ssd_verify_params* params, int32_t* host_accepted_len,
                    int32_t* host_next_token, void* stream);

/* "Append to T_in" (Algorithm 1): len[b] += 1 + accepted_len[b]; pending[b] = next_token[b].
 * Rejected positions need no work: they lie beyond the new len. */
int ssd_kv_commit(ssd_streams* s, const int32_t* dev_accepted_len, const int32_t* dev_next_token,
                  void* stream);

/* One whole SSD iteration (the body of Algorithm 1's while loop) for all B streams, enqueued on
 * `stream` without any host round trip: gamma draft steps (Eq. 2-3), the parallel verification and
 * acceptance (Eq. 4-6), "append to T_in" on the target's and on the draft's cache, and the
 * emitted tokens appended to a per-stream output.  Capture it in a CUDA graph and replay it to
 * run the loop from the device.
 *
 * Draft-cache rule: after an iteration the draft holds K/V for the old pending token and
 * x_1..x_{gamma-1}.  Every iteration therefore starts with a draft step over TWO ids, [the token
 * before the pending one, the pending one], at draft len = target len - 1: after a full acceptance
 * this computes the missing K/V of x_gamma, otherwise it recomputes one cached row from the same
 * inputs.  One rule for all streams, so no stream's acceptance count ever reaches the host.
 * Before the first iteration the caller prefills both models with the same prefix (>= 2 tokens),
 * rolls the DRAFT streams back by one (ssd_kv_truncate to len - 1) and stores the prefix's last
 * two ids in dev_in_ids.  The draft streams need max_gamma >= 1 and capacity for gamma + 1 more
 * tokens than the target's prefix.
 *
 * ssd_loop_io (all device pointers, caller-owned):
 *   dev_uniform_pool float [n_iterations][B][gamma + 2 (gamma + 1)]: per stream the gamma draws
 *                    for x_i ~ p_i, then (r_i, u_i) for the gamma + 1 verify rows, all in [0, 1);
 *   dev_iteration    int32 [1]: row of the pool the next iteration uses (modulo n_iterations);
 *                    advanced by one at the end of the iteration;
 *   dev_in_ids       int32 [B, 2]: the next iteration's first two draft inputs (see above); updated;
 *   dev_draft_tokens int32 [B, gamma], dev_draft_probs float [B, gamma, V]: x_i and p_i of the
 *                    iteration (outputs, also useful to inspect);
 *   dev_accepted_len, dev_next_token  int32 [B]: k and the new token of the iteration;
 *   dev_out_tokens   int32 [B, out_capacity], dev_out_count int32 [B]: x_1..x_k, y are appended at
 *                    out_count (tokens beyond the capacity are counted, not stored);
 *   dev_accept_log   int32 [n_iterations, B] or NULL: k of every iteration (row = pool row). */
typedef struct {
  const float* dev_uniform_pool;
  int32_t n_iterations;
  int32_t* dev_iteration;
  int32_t* dev_in_ids;
  int32_t* dev_draft_tokens;
  float* dev_draft_probs;
  int32_t* dev_accepted_len;
  int32_t* dev_next_token;
  int32_t* dev_out_tokens;
  int32_t out_capacity;
  int32_t* dev_out_count;
  int32_t* dev_accept_log;
} ssd_loop_io;
int ssd_iteration(ssd_model* target, ssd_streams* target_streams, ssd_model* draft,
                  ssd_streams* draft_streams, const ssd_verify_params* params, const ssd_loop_io* io,
                  void* stream);

/* Acceptance step without any device allocation (the paper has no counterpart: this is a
 * packaging variant of the acceptance kernel behind ssd_verify, not a step of the method).
 * For callers that may not allocate device memory at all - e.g. a serving loop whose memory pool
 * is fixed at start-up, or a plug-in that only receives device pointers from its host process -
 * and so cannot provide the workspace ssd_streams_create needs.  Given target logits the caller
 * already holds, it applies the sampling transform, the tolerance test of Eq. 5 and the resample /
 * bonus draw of Eq. 6 exactly as ssd_verify does, and writes the same two outputs.
 *   in  dev_logits float [batch, gamma+1, vocab]; dev_draft_tokens, dev_draft_probs, dev_uniforms
 *       as in ssd_verify;  out dev_accepted_len, dev_next_token int32 [batch].
 * The kernel's scratch lives in a fixed array inside the library (about 148 KB, held by every GPU
 * that loads the library until the process exits), sized for at most 256 streams and
 * gamma + 1 <= 16 rows: larger batches return SSD_ERR_TOO_SMALL, larger gamma SSD_ERR_BAD_GAMMA.
 * No cudaMalloc / cudaFree or allocating library routine is called.  The first call on a device
 * looks up the array's address (cudaGetSymbolAddress, with that device current); make that first
 * call before starting any stream capture.  All calls share the one array, which keeps the last
 * call's contents: the per-stream counters are cleared on `stream` at the start of each call, and
 * two calls that overlap on the GPU (different streams, or different threads) race on it.
 * This call reports no device status bits (there is no streams object to hold them): a draft token
 * outside [0, vocab) or a draft probability that is negative or not finite is treated as rejected
 * at its position, so accepted_len stops in front of it and next_token is the resample there. */
int ssd_accept_noalloc(const float* dev_logits, const int32_t* dev_draft_tokens,
                       const float* dev_draft_probs, const float* dev_uniforms,
                       const ssd_verify_params* params, int32_t batch, int32_t vocab,
                       int32_t* dev_accepted_len, int32_t* dev_next_token, void* stream);

/* ---- host-side checks of the persistent kernel's weight packing (no device needed) ------- */

/* Plan of the persistent small-batch kernel for a bf16 model on n_cta CTAs.  out8 receives:
 * packed bytes in total, fewest / most bytes any CTA streams, most output tiles a CTA owns for one
 * projection, most chunks in a warp's table, K slices of the down projection, K slices (groups
 * of query heads) of the O projection, output tiles over all CTAs and projections.  SSD_ERR_BAD_CONFIG if the model has no such path. */
int ssd_fast_plan_host(const ssd_model_config* cfg, int32_t n_cta, int64_t* out8);
/* Packs the projection weights of host_weights (blob of ssd_model_create) into the per-warp streams
 * and walks the streams back into host_out (same layout and size; only the projection matrices and
 * the LM head are written).  *bad_chunks = chunk-table entries that disagree with the walk. */
int ssd_fast_pack_roundtrip_host(const ssd_model_config* cfg, int32_t n_cta, const void* host_weights,
                                 size_t nbytes, void* host_out, int64_t* bad_chunks);

/* ---- the tensor-core projection kernel alone (tests of the batched forward's building block) -- */

/* One projection of the decoder (Sec. 3.1; Eq. 4) as the batched forward runs it on the tcgen05
 * tensor cores: acc[t, r] = sum_k x[t, k] * w[r, k] for M token rows (17..512 are what the forward
 * uses; 1..512 accepted) and n_rows weight rows, K a multiple of 8.
 *   dev_w   bf16 [n_rows, K] row-major;  dev_x  float [M, K];  both device pointers, read-only.
 *   dev_scratch  device buffer of at least ssd_tc_gemm_scratch_bytes(M, n_rows, K) bytes (256-byte
 *                aligned), zero-filled by the caller: receives the packed operands.
 *   epilogue 0: K split `ksplit` ways; dev_out float [ksplit, Mpad, ld] receives one slab of
 *               partial sums per K slice (Mpad = M rounded up to 16, ld = n_rows rounded up to
 *               128): element [s, t, r].  Their sum over s is acc.
 *   epilogue 1: ksplit must be 1; dev_out float [M, n_rows] = acc (the LM-head form).
 *   epilogue 2: ksplit must be 1; weight rows are (gate_j, up_j) pairs; dev_out receives
 *               SiLU(gate_j) * up_j as a packed operand of n_rows / 2 columns:
 *               byte(part, t, j) = ((t / Mc) * KS + j / 16) * Mc * 64 + ((j / 8) % 2) * Mc * 32
 *                                  + part * Mc * 16 + (t % Mc) * 16 + (j % 8) * 2,
 *               part 0 = bf16 leading part of the value, part 1 = bf16 of the remainder; KS =
 *               n_rows / 2 columns rounded up to 16, over 16; the rows are stored in C chunks of
 *               Mc rows: C = 1, Mc = Mpad up to 256 rows, else C = ceil(Mpad / 256) and Mc = Mpad / C
 *               rounded up to 16 (KS * C * Mc * 64 bytes in all).
 * Enqueues on `stream`; SSD_ERR_BAD_PARAM for sizes outside the ranges above. */
size_t ssd_tc_gemm_scratch_bytes(int32_t M, int32_t n_rows, int32_t K);
int ssd_tc_gemm_check(const void* dev_w, const float* dev_x, int32_t M, int32_t n_rows, int32_t K,
                      int32_t ksplit, int32_t epilogue, void* dev_scratch, size_t scratch_bytes,
                      void* dev_out, int32_t* dev_status, void* stream);

/* ---- diagnostics ------------------------------------------------------------------------- */

/* Reads and clears the device status word (SSD_STATUS_* bits).  Synchronises `stream`. */
int ssd_last_status(ssd_streams* s, int32_t* status, void* stream);
/* Host-made failure for tests of the error path: marks the streams object exactly as a bounded
 * wait that ran out inside the persistent kernel marks it.  Every later small-batch forward on
 * these streams returns at once without touching its outputs and raises SSD_STATUS_TIMEOUT; the
 * object must be created anew to be used again.  No kernel is made to wait or fail for this.
 * Synchronises `stream`. */
int ssd_streams_inject_failure(ssd_streams* s, void* stream);
/* Number of kernels this library has enqueued in this process so far (all handles). */
uint64_t ssd_kernel_launch_count(void);
/* Text of the last CUDA error seen by this library on this thread ("" if none). */
const char* ssd_last_cuda_error(void);
const char* ssd_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* SSD_H_ */
