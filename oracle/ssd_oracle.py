"""CPU oracle for the Speech Speculative Decoding (SSD) verify step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 restatement of what one SSD verification step computes, written from the
paper and used solely to check the CUDA path (tests, the smoke check, and the CPU-baseline leg of
the benchmark).  It shares no code with the CUDA path and must never be imported by the product.

What is computed, and from which passage:

* `forward`      - the target model M_q run once over the pending token and the gamma draft
                   tokens against the cached prefix, giving gamma+1 next-token distributions
                   (Algorithm 1, the parallel-verification line; Eq. 4).  The decoder is the
                   "Transformer adapted from Qwen2.5" of Sec. 3.1: pre-norm RMSNorm, grouped-query
                   attention with biased q/k/v projections and rotate-half RoPE, SiLU-gated
                   feed-forward, final RMSNorm, untied LM head.
* `transform`    - temperature, top-k and nucleus (top-p) applied to a logit row before softmax.
                   The paper does not describe a sampler; this is the workload's (stated reading:
                   z/T, keep the top_k largest with the lower id winning ties, then the shortest
                   prefix of those, most probable first, whose mass reaches top_p; softmax over
                   what is kept).
* `transform_ras`- repetition-aware sampling (a nucleus draw that is redrawn from the full softmax
                   when it repeats a recent token) written as the one distribution it samples from.
* `accept_step`  - the sequential tolerance test r_i < min(1, q_i(x_i)/p_i(x_i)) + beta (Eq. 5),
                   the residual resample from normalize(max(0, q_i - p_i)) at the first rejection
                   (Eq. 6), and the bonus token from q_{gamma+1} when nothing is rejected
                   (Algorithm 1, last branch).  p is the DRAFT distribution and q the TARGET
                   distribution, as in the paper (the reverse of the usual letters).
* `commit`       - "append to T_in": the prefix grows by the accepted draft tokens plus the one
                   corrected / bonus token (Algorithm 1).
* `PagedCache`   - a page pool with per-stream block tables: a layout, not arithmetic; pinned to
                   give exactly the contiguous cache's results while streams grow, roll back,
                   leave and join.

State convention: a stream holding n tokens keeps K/V for tokens 0..n-2 (`length` = n-1) and the
last token as `pending`.  A verify step feeds [pending, x_1..x_gamma] at positions
length..length+gamma, so row r predicts the token that follows x_r (row 0: the slot of x_1).

Arithmetic is float64 throughout.  Storage formats are part of the problem, not of the
arithmetic: weights arrive already rounded to the model's storage type, and K/V rows are rounded
to the cache's storage type (bf16 or fp32) when they are appended.

Pins (tests/test_oracle_*.py): forward vs gamma+1 sequential decodes; forward vs the
`transformers` Qwen2 implementation and torch's scaled_dot_product_attention as black-box library
routines; exact rational enumeration of the acceptance rule's output law (equal to q at beta = 0,
and to the closed form for beta > 0); brute-force inverse CDF; monotonicity in beta; commit /
rollback invariants.  No function here is "parity unpinned".
"""
from __future__ import annotations

from typing import Dict, List, Optional, Tuple

import numpy as np

F64 = np.float64


def _round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of float64 values to bf16-representable values (via float32)."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(F64)


class Model:
    """Decoder weights (float32 arrays holding exact storage values) plus shape fields."""

    def __init__(self, *, n_layers: int, d_model: int, n_q_heads: int, n_kv_heads: int,
                 head_dim: int, d_ffn: int, vocab_out: int, vocab_text: int, rope_theta: float,
                 rms_eps: float, kv_bf16: bool, weights: Dict[str, np.ndarray]):
        self.L, self.d = n_layers, d_model
        self.Hq, self.Hkv, self.hd = n_q_heads, n_kv_heads, head_dim
        self.F, self.V, self.Vtext = d_ffn, vocab_out, vocab_text
        self.theta, self.eps = float(rope_theta), float(rms_eps)
        self.kv_bf16 = bool(kv_bf16)
        self.w = weights


class Stream:
    """One utterance's state: cached K/V per layer, committed length, pending token."""

    def __init__(self, model: Model, capacity: int):
        self.K = [np.zeros((capacity, model.Hkv, model.hd), F64) for _ in range(model.L)]
        self.V = [np.zeros((capacity, model.Hkv, model.hd), F64) for _ in range(model.L)]
        self.capacity = capacity
        self.length = 0          # tokens whose K/V are committed
        self.pending = -1        # last token of T_in, not yet run through the model


# ------------------------------------------------------------------ decoder pieces (Sec. 3.1)

def rms_norm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * gain, row-wise."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain.astype(F64)


def rope(x: np.ndarray, positions: np.ndarray, theta: float) -> np.ndarray:
    """Rotate-half rotary embedding.  x: [rows, heads, hd]; positions: [rows] absolute."""
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = theta ** (-np.arange(half, dtype=F64) * 2.0 / hd)
    ang = positions.astype(F64)[:, None] * inv_freq[None, :]          # [rows, half]
    cos, sin = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def attention_rows(q: np.ndarray, K: np.ndarray, V: np.ndarray, first_pos: int) -> np.ndarray:
    """Causal grouped-query attention of new rows against a cache that already contains them.

    q: [R, Hq, hd] (row r sits at absolute position first_pos + r);
    K, V: [>= first_pos + R, Hkv, hd].  Row r attends to keys 0..first_pos + r.
    """
    R, Hq, hd = q.shape
    group = Hq // K.shape[1]
    out = np.zeros((R, Hq, hd), F64)
    for r in range(R):
        n_keys = first_pos + r + 1
        for h in range(Hq):
            g = h // group
            s = K[:n_keys, g, :] @ q[r, h, :] / np.sqrt(hd)
            s = np.exp(s - s.max())
            out[r, h, :] = (s / s.sum()) @ V[:n_keys, g, :]
    return out


def forward(model: Model, stream: Stream, ids: np.ndarray) -> np.ndarray:
    """Run `ids` through M_q at positions stream.length.., appending their K/V (Eq. 4).

    Returns logits [len(ids), V] in float64.  stream.length is NOT advanced: the appended rows
    stay provisional until `commit` (or a prefill) moves the length.
    """
    w, m = model.w, model
    ids = np.asarray(ids, dtype=np.int64)
    R, p0 = len(ids), stream.length
    assert p0 + R <= stream.capacity, "KV cache overflow"
    pos = p0 + np.arange(R)
    h = w["embed"][ids].astype(F64)
    for l in range(m.L):
        pre = f"l{l}."
        xn = rms_norm(h, w[pre + "norm1"], m.eps)
        q = (xn @ w[pre + "wq"].T.astype(F64) + w[pre + "bq"]).reshape(R, m.Hq, m.hd)
        k = (xn @ w[pre + "wk"].T.astype(F64) + w[pre + "bk"]).reshape(R, m.Hkv, m.hd)
        v = (xn @ w[pre + "wv"].T.astype(F64) + w[pre + "bv"]).reshape(R, m.Hkv, m.hd)
        q, k = rope(q, pos, m.theta), rope(k, pos, m.theta)
        if m.kv_bf16:
            k, v = _round_to_bf16(k), _round_to_bf16(v)
        else:
            k, v = k.astype(np.float32).astype(F64), v.astype(np.float32).astype(F64)
        stream.K[l][p0:p0 + R] = k
        stream.V[l][p0:p0 + R] = v
        att = attention_rows(q, stream.K[l], stream.V[l], p0).reshape(R, m.Hq * m.hd)
        h = h + att @ w[pre + "wo"].T.astype(F64)
        xn = rms_norm(h, w[pre + "norm2"], m.eps)
        gate = xn @ w[pre + "wg"].T.astype(F64)
        up = xn @ w[pre + "wu"].T.astype(F64)
        h = h + (silu(gate) * up) @ w[pre + "wd"].T.astype(F64)
    xn = rms_norm(h, w["norm_f"], m.eps)
    return xn @ w["head"].T.astype(F64)


def prefill(model: Model, stream: Stream, ids: np.ndarray, chunk: int = 64) -> None:
    """Load a prefix T_in: K/V for all but the last id, which becomes the pending token."""
    ids = np.asarray(ids, dtype=np.int64)
    assert stream.length == 0 and len(ids) >= 1
    for s in range(0, len(ids) - 1, chunk):
        part = ids[s:min(s + chunk, len(ids) - 1)]
        forward(model, stream, part)
        stream.length += len(part)
    stream.pending = int(ids[-1])


# ------------------------------------------------------------------ sampling transform

def transform(logits_row: np.ndarray, temperature: float, top_k: int, top_p: float = 0.0) -> np.ndarray:
    """Logit row -> the distribution the target's sampler draws from (q_i in Eq. 5-6).

    z = logits / T; keep the top_k largest (lower id wins ties; top_k <= 0 or >= V: all); then,
    with 0 < top_p < 1, the nucleus: walking the kept ids from the most to the least probable
    (lower id first among equals), an id stays while the mass of the ids before it is below
    top_p, i.e. the shortest such prefix whose mass reaches top_p; softmax over what is left.
    """
    z = np.asarray(logits_row, F64) / float(temperature)
    V = z.shape[0]
    order = np.argsort(-z, kind="stable")            # equal values: lower id first
    keep = np.ones(V, dtype=bool)
    if 0 < top_k < V:
        keep[:] = False
        keep[order[:top_k]] = True
    if 0.0 < top_p < 1.0:
        e = np.where(keep, np.exp(z - z[keep].max()), 0.0)
        prob = e / e.sum()
        before = 0.0
        for t in order:                              # kept ids come first in this order
            if not keep[t]:
                break
            if before >= top_p:
                keep[t] = False
            before += prob[t]
    e = np.where(keep, np.exp(z - z[keep].max()), 0.0)
    return e / e.sum()


def transform_ras(logits_row: np.ndarray, temperature: float, top_k: int, top_p: float,
                  window: np.ndarray, win_size: int, tau_r: float) -> np.ndarray:
    """Repetition-aware sampling as ONE distribution (the paper is silent on samplers; this is the
    sampler of the CosyVoice family the paper builds on, restated).

    The procedure: draw a token from the nucleus / top-k distribution q_nuc; if it occurs at least
    win_size * tau_r times among the last win_size tokens (`window`, any -1 entries ignored), throw
    it away and draw from the full softmax q_full instead.  Its output law is
        q(x) = q_nuc(x) * [x not repeated] + R * q_full(x),   R = sum of q_nuc over repeated ids,
    which is the target distribution q_i that Eq. 5-6 then use.
    """
    q_nuc = transform(logits_row, temperature, top_k, top_p)
    if win_size <= 0:
        return q_nuc
    q_full = transform(logits_row, temperature, 0, 0.0)
    w = np.asarray(window, dtype=np.int64)[-win_size:]
    w = w[w >= 0]
    ids, counts = np.unique(w, return_counts=True)
    repeated = ids[counts >= win_size * tau_r]
    mask = np.zeros(len(q_nuc), dtype=bool)
    mask[repeated[repeated < len(q_nuc)]] = True
    R = float(q_nuc[mask].sum())
    return np.where(mask, 0.0, q_nuc) + R * q_full


# ------------------------------------------------------------------ acceptance (Eq. 5, 6)

def categorical_draw(weights: np.ndarray, u: float) -> Tuple[int, float]:
    """Inverse-CDF draw in ascending id: smallest t with sum_{s<=t} w_s > u * sum(w).

    Also returns the draw's margin: the distance from u to the nearer CDF edge of the chosen
    id, in units of total mass (used by parity tests to skip knife-edge draws).
    """
    cdf = np.cumsum(weights.astype(F64))
    total = cdf[-1]
    target = float(u) * total
    t = int(np.searchsorted(cdf, target, side="right"))
    t = min(t, len(cdf) - 1)
    while t > 0 and weights[t] <= 0.0:       # never land on a zero-mass id
        t -= 1
    lo = cdf[t - 1] if t > 0 else 0.0
    margin = min(target - lo, cdf[t] - target) / total
    return t, float(margin)


def accept_step(q_rows: np.ndarray, p_rows: np.ndarray, draft_tokens: np.ndarray,
                uniforms: np.ndarray, beta: float) -> Dict[str, object]:
    """Algorithm 1's inner loop for one stream.

    q_rows [gamma+1, V] target distributions, p_rows [gamma, V] draft distributions,
    draft_tokens [gamma], uniforms [gamma+1, 2] with [:, 0] = r_i and [:, 1] = the draw's u.
    Returns accepted length k, the one new token y, and diagnostics (thresholds a_i, margins).
    """
    gamma = len(draft_tokens)
    thresholds: List[float] = []
    k = gamma
    for i in range(gamma):
        x = int(draft_tokens[i])
        qi, pi = float(q_rows[i][x]), float(p_rows[i][x])
        ratio = 1.0 if pi <= qi else qi / pi           # min(1, q/p) without dividing by zero
        a = ratio + float(beta)
        thresholds.append(a)
        if float(uniforms[i][0]) < a:
            continue                                    # accept x_i
        k = i
        break
    if k < gamma:                                       # first rejection at position k+1
        resid = np.maximum(0.0, q_rows[k].astype(F64) - p_rows[k].astype(F64))
        if resid.sum() <= 0.0:                          # numerical corner: fall back to q
            resid = q_rows[k].astype(F64)
        y, margin = categorical_draw(resid, float(uniforms[k][1]))
    else:                                               # all accepted: bonus from q_{gamma+1}
        y, margin = categorical_draw(q_rows[gamma].astype(F64), float(uniforms[gamma][1]))
    return {"k": k, "y": y, "thresholds": thresholds, "draw_margin": margin}


def verify(model: Model, stream: Stream, draft_tokens: np.ndarray, p_rows: np.ndarray,
           uniforms: np.ndarray, *, temperature: float, top_k: int, beta: float, top_p: float = 0.0,
           recent: Optional[np.ndarray] = None, win_size: int = 0, tau_r: float = 0.0
           ) -> Dict[str, object]:
    """One full verification step for one stream (forward, transform, accept); no commit.

    With win_size > 0 the target samples repetition-aware: `recent` holds the last tokens of T_in
    (the pending token last); row i's window is the last win_size tokens of recent + x_1..x_{i-1}.
    """
    ids = np.concatenate([[stream.pending], np.asarray(draft_tokens, np.int64)])
    logits = forward(model, stream, ids)
    if win_size > 0:
        hist = np.concatenate([np.asarray(recent, np.int64), np.asarray(draft_tokens, np.int64)])
        n0 = len(recent)
        q_rows = np.stack([transform_ras(row, temperature, top_k, top_p, hist[:n0 + i], win_size, tau_r)
                           for i, row in enumerate(logits)])
    else:
        q_rows = np.stack([transform(row, temperature, top_k, top_p) for row in logits])
    res = accept_step(q_rows, p_rows, draft_tokens, uniforms, beta)
    res["logits"] = logits
    res["q_rows"] = q_rows
    return res


def commit(stream: Stream, k: int, y: int) -> None:
    """T_in grows by the k accepted draft tokens and the new token y (Algorithm 1)."""
    stream.length += 1 + int(k)
    stream.pending = int(y)


def truncate(stream: Stream, new_length: int, pending: int) -> None:
    """Roll the stream back to an earlier prefix; later cache rows become dead."""
    assert 0 <= new_length <= stream.length
    stream.length, stream.pending = int(new_length), int(pending)


# ------------------------------------------------------------------ paged cache (layout only)

PAGE_TOKENS = 64


class PagedCache:
    """A pool of fixed-size K/V pages shared by several streams, with a block table per stream.

    The paper says nothing about memory layout: a paged cache must be indistinguishable from the
    contiguous one (same logits, same decisions) while letting streams of very different lengths
    share memory, join and leave.  Token t of stream b lives in page table[b][t // PAGE_TOKENS],
    slot t % PAGE_TOKENS.  Rolling a stream back to `length` tokens returns the pages that lie
    wholly beyond it to the free list: O(1) per page, no data moves.
    """

    def __init__(self, model: Model, n_streams: int, n_pages: int, max_pages_per_stream: int):
        self.m = model
        self.K = np.zeros((model.L, n_pages, PAGE_TOKENS, model.Hkv, model.hd), F64)
        self.V = np.zeros((model.L, n_pages, PAGE_TOKENS, model.Hkv, model.hd), F64)
        self.free = list(range(n_pages - 1, -1, -1))          # stack: pop() takes page 0 first
        self.table = [[] for _ in range(n_streams)]
        self.max_pages = max_pages_per_stream
        self.length = [0] * n_streams
        self.pending = [-1] * n_streams

    def ensure(self, b: int, n_tokens: int) -> None:
        """Make sure stream b owns pages for its first n_tokens slots."""
        need = -(-n_tokens // PAGE_TOKENS)
        assert need <= self.max_pages, "stream exceeds its block table"
        while len(self.table[b]) < need:
            assert self.free, "out of pages"
            self.table[b].append(self.free.pop())

    def release(self, b: int) -> None:
        """Return the pages wholly beyond the committed length of stream b."""
        keep = -(-self.length[b] // PAGE_TOKENS)
        while len(self.table[b]) > keep:
            self.free.append(self.table[b].pop())


def forward_paged(model: Model, cache: PagedCache, b: int, ids: np.ndarray) -> np.ndarray:
    """`forward` for stream b of a paged cache: gather its pages into a contiguous view, run the
    same forward, scatter the appended rows back into the pages."""
    ids = np.asarray(ids, dtype=np.int64)
    n0, R = cache.length[b], len(ids)
    cache.ensure(b, n0 + R)
    view = Stream(model, len(cache.table[b]) * PAGE_TOKENS)
    for l in range(model.L):
        for i, pg in enumerate(cache.table[b]):
            view.K[l][i * PAGE_TOKENS:(i + 1) * PAGE_TOKENS] = cache.K[l, pg]
            view.V[l][i * PAGE_TOKENS:(i + 1) * PAGE_TOKENS] = cache.V[l, pg]
    view.length, view.pending = n0, cache.pending[b]
    logits = forward(model, view, ids)
    for l in range(model.L):
        for t in range(n0, n0 + R):
            pg, slot = cache.table[b][t // PAGE_TOKENS], t % PAGE_TOKENS
            cache.K[l, pg, slot] = view.K[l][t]
            cache.V[l, pg, slot] = view.V[l][t]
    return logits


def commit_paged(cache: PagedCache, b: int, k: int, y: int) -> None:
    cache.length[b] += 1 + int(k)
    cache.pending[b] = int(y)
    cache.release(b)


def truncate_paged(cache: PagedCache, b: int, new_length: int, pending: int) -> None:
    assert 0 <= new_length <= cache.length[b]
    cache.length[b], cache.pending[b] = int(new_length), int(pending)
    cache.release(b)
