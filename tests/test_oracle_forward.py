"""Pins for the oracle's decoder forward (CPU only).

The verify forward (Eq. 4) has a plain definition: row r equals the logits of an ordinary
single-token decode after feeding T_in, x_1..x_r.  The architecture reading ("Transformer adapted
from Qwen2.5", Sec. 3.1) is pinned against the `transformers` Qwen2 implementation and torch's
attention used as black-box library routines.
"""
import numpy as np
import pytest
import torch

from oracle import ssd_oracle as orc
from paper_2505_15380_b200 import synth
from tests.helpers import oracle_model, small_shape


def _prefilled(shape, seed=5, n=12, capacity=64):
    w = synth.make_weights(shape, seed)
    m = oracle_model(shape, w)
    rng = np.random.default_rng(seed)
    ids = rng.integers(0, shape.vocab_in, size=n)
    st = orc.Stream(m, capacity)
    orc.prefill(m, st, ids)
    return m, st, ids


@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
def test_parallel_verify_equals_sequential_decodes(dtype):
    shape = small_shape(weight_dtype=dtype)
    m, st, _ = _prefilled(shape)
    draft = np.array([3, 17, 5, 29])
    par = orc.forward(m, st, np.concatenate([[st.pending], draft]))
    # sequential: one token at a time, each a full single-token decode
    m2, st2, _ = _prefilled(shape)
    seq = []
    for t in np.concatenate([[st2.pending], draft]):
        seq.append(orc.forward(m2, st2, np.array([t]))[0])
        st2.length += 1
    assert np.allclose(par, np.stack(seq), rtol=0, atol=1e-12)


def test_causality_inside_the_draft_block():
    shape = small_shape()
    m, st, _ = _prefilled(shape)
    a = orc.forward(m, st, np.array([st.pending, 3, 17, 5, 29]))
    b = orc.forward(m, st, np.array([st.pending, 3, 17, 6, 29]))      # change x_3 only
    assert np.array_equal(a[:3], b[:3])
    assert not np.allclose(a[3], b[3]) and not np.allclose(a[4], b[4])


def test_chunked_prefill_is_chunk_size_independent():
    shape = small_shape()
    w = synth.make_weights(shape, 2)
    m = oracle_model(shape, w)
    ids = np.random.default_rng(0).integers(0, shape.vocab_in, size=21)
    s1, s2 = orc.Stream(m, 32), orc.Stream(m, 32)
    orc.prefill(m, s1, ids, chunk=64)
    orc.prefill(m, s2, ids, chunk=3)
    assert s1.length == s2.length == 20 and s1.pending == s2.pending == ids[-1]
    for l in range(m.L):
        assert np.allclose(s1.K[l][:20], s2.K[l][:20], atol=1e-6)
        assert np.allclose(s1.V[l][:20], s2.V[l][:20], atol=1e-6)


@pytest.mark.parametrize("hq,hkv,hd", [(4, 2, 16), (6, 1, 8), (4, 4, 32)])
def test_forward_matches_transformers_qwen2(hq, hkv, hd):
    """Same weights into HF's Qwen2ForCausalLM (float64): logits must agree."""
    from transformers import Qwen2Config, Qwen2ForCausalLM
    shape = small_shape(n_q_heads=hq, n_kv_heads=hkv, head_dim=hd, d_model=48, rope_theta=1e6)
    w = synth.make_weights(shape, 11)
    # make the check sensitive to gains and biases
    rng = np.random.default_rng(1)
    for name in w:
        if "norm" in name:
            w[name] = (1.0 + 0.3 * rng.standard_normal(w[name].shape)).astype(np.float32)
        if name.split(".")[-1] in ("bq", "bk", "bv"):
            w[name] = (0.5 * rng.standard_normal(w[name].shape)).astype(np.float32)
        if name.split(".")[-1] in ("wq", "wk", "wo", "wg", "wu", "wd"):
            w[name] = w[name] * np.float32(6.0)
    m = oracle_model(shape, w)
    cfg = Qwen2Config(vocab_size=shape.vocab_in, hidden_size=shape.d_model,
                      intermediate_size=shape.d_ffn, num_hidden_layers=shape.n_layers,
                      num_attention_heads=hq, num_key_value_heads=hkv, head_dim=hd,
                      max_position_embeddings=128, rms_norm_eps=shape.rms_eps,
                      rope_theta=shape.rope_theta, tie_word_embeddings=False,
                      use_sliding_window=False, attention_dropout=0.0,
                      rope_parameters={"rope_type": "default", "rope_theta": shape.rope_theta})
    hf = Qwen2ForCausalLM(cfg).double().eval()
    sd = {"model.embed_tokens.weight": w["embed"], "model.norm.weight": w["norm_f"]}
    head = np.zeros((shape.vocab_in, shape.d_model), np.float32)
    head[:shape.vocab_out] = w["head"]
    sd["lm_head.weight"] = head
    names = {"norm1": "input_layernorm.weight", "wq": "self_attn.q_proj.weight",
             "bq": "self_attn.q_proj.bias", "wk": "self_attn.k_proj.weight",
             "bk": "self_attn.k_proj.bias", "wv": "self_attn.v_proj.weight",
             "bv": "self_attn.v_proj.bias", "wo": "self_attn.o_proj.weight",
             "norm2": "post_attention_layernorm.weight", "wg": "mlp.gate_proj.weight",
             "wu": "mlp.up_proj.weight", "wd": "mlp.down_proj.weight"}
    for l in range(shape.n_layers):
        for k, v in names.items():
            sd[f"model.layers.{l}.{v}"] = w[f"l{l}.{k}"]
    missing = hf.load_state_dict({k: torch.from_numpy(np.asarray(v)).double() for k, v in sd.items()},
                                 strict=True)
    ids = np.random.default_rng(3).integers(0, shape.vocab_in, size=19)
    with torch.no_grad():
        ref = hf(torch.from_numpy(ids)[None]).logits[0, :, :shape.vocab_out].numpy()
    # oracle: prefill 14 tokens, then a 5-row verify forward
    st = orc.Stream(m, 32)
    orc.prefill(m, st, ids[:15])
    got = orc.forward(m, st, ids[14:19])
    assert np.abs(ref[14:19]).max() > 0.1
    # the oracle's fp32 cache rounds K/V to float32 (storage format) and HF builds its rotary
    # tables in float32, so agreement is to float32 resolution; a wrong convention (RoPE layout,
    # GQA grouping, bias or norm placement) moves logits by >= 1e-2 here.
    assert np.allclose(got, ref[14:19], rtol=0, atol=2e-6)


def test_attention_rows_match_torch_sdpa():
    rng = np.random.default_rng(0)
    R, Hq, Hkv, hd, p0 = 5, 6, 2, 16, 9
    q = rng.standard_normal((R, Hq, hd))
    K = rng.standard_normal((p0 + R, Hkv, hd))
    V = rng.standard_normal((p0 + R, Hkv, hd))
    got = orc.attention_rows(q, K, V, p0)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(K).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)[None]
    tv = torch.from_numpy(V).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)[None]
    mask = torch.zeros(R, p0 + R, dtype=torch.bool)
    for r in range(R):
        mask[r, :p0 + r + 1] = True
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask)
    assert np.allclose(got, ref[0].permute(1, 0, 2).numpy(), atol=1e-12)


def test_rope_is_relative():
    rng = np.random.default_rng(0)
    q, k = rng.standard_normal((1, 1, 32)), rng.standard_normal((1, 1, 32))
    def score(pq, pk):
        return float(np.sum(orc.rope(q, np.array([pq]), 1e4) * orc.rope(k, np.array([pk]), 1e4)))
    assert abs(score(7, 3) - score(107, 103)) < 1e-9
    assert abs(score(7, 3) - score(8, 3)) > 1e-6
    # position 0 is the identity; norms are preserved
    assert np.allclose(orc.rope(q, np.array([0]), 1e4), q)
    assert np.isclose(np.linalg.norm(orc.rope(q, np.array([13]), 1e4)), np.linalg.norm(q))


def test_rms_norm_and_silu_closed_forms():
    x = np.array([[3.0, -4.0]])
    out = orc.rms_norm(x, np.array([2.0, 0.5], np.float32), 0.0)
    assert np.allclose(out, [[2.0 * 3 / np.sqrt(12.5), 0.5 * -4 / np.sqrt(12.5)]])
    assert np.isclose(orc.silu(np.array([0.0]))[0], 0.0)
    assert np.isclose(orc.silu(np.array([2.0]))[0], 2.0 / (1 + np.exp(-2.0)))
    t = torch.tensor([-1.5, 0.3, 4.0], dtype=torch.float64)
    assert np.allclose(orc.silu(t.numpy()), torch.nn.functional.silu(t).numpy())


def test_kv_storage_rounding():
    shape = small_shape(weight_dtype=synth.BF16)
    m, st, _ = _prefilled(shape)
    k = st.K[0][:st.length]
    assert np.array_equal(synth.bf16_round(k.astype(np.float32)).astype(np.float64), k)


def test_bf16_rounding_is_round_to_nearest_even():
    """The cache's storage rounding against torch's own float32 -> bfloat16 conversion (a library
    routine) and against ties worked out by hand: bf16 keeps 8 significand bits, so around 1 the
    spacing is 2^-7 and a value exactly half way goes to the even neighbour."""
    rng = np.random.Generator(np.random.Philox(key=5))
    x = np.concatenate([rng.standard_normal(4000) * 3.0, rng.standard_normal(2000) * 1e-3,
                        rng.standard_normal(1000) * 1e4, [0.0, -0.0, 1.0, -1.0]]).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(orc._round_to_bf16(x.astype(np.float64)), ref)
    e = 2.0 ** -8                                      # half a bf16 step at 1
    cases = {1 + e: 1.0,                               # tie -> even (down)
             1 + 3 * e: 1 + 4 * e,                     # tie -> even (up)
             1 + e + 2.0 ** -20: 1 + 2 * e,            # just above the tie
             1 + e - 2.0 ** -20: 1.0,                  # just below
             -(1 + e): -1.0, -(1 + 3 * e): -(1 + 4 * e),
             0.3: 0.30078125, -2.7: -2.703125}
    for v, want in cases.items():
        assert orc._round_to_bf16(np.array([v]))[0] == want, v
    # truncation or round-half-up would each fail one of the ties above
    assert orc._round_to_bf16(np.array([1 + 3 * e]))[0] != 1 + 2 * e
    assert orc._round_to_bf16(np.array([1 + e]))[0] != 1 + 2 * e


def test_commit_then_verify_equals_fresh_prefill():
    shape = small_shape()
    m, st, ids = _prefilled(shape)
    draft = np.array([3, 17, 5, 29])
    orc.forward(m, st, np.concatenate([[st.pending], draft]))
    orc.commit(st, 2, 33)                              # keep x_1, x_2, new token 33
    again = orc.forward(m, st, np.array([st.pending, 1, 2]))
    m2 = m
    st2 = orc.Stream(m2, 64)
    orc.prefill(m2, st2, np.concatenate([ids, draft[:2], [33]]))
    fresh = orc.forward(m2, st2, np.array([33, 1, 2]))
    assert st.length == st2.length == len(ids) + 2
    assert np.allclose(again, fresh, atol=1e-10)


def test_truncate_makes_verify_idempotent():
    shape = small_shape()
    m, st, _ = _prefilled(shape)
    ids = np.array([st.pending, 3, 17, 5, 29])
    a = orc.forward(m, st, ids)
    length, pending = st.length, st.pending
    orc.commit(st, 4, 7)
    orc.truncate(st, length, pending)
    b = orc.forward(m, st, ids)
    assert np.array_equal(a, b)


def test_paged_cache_equals_contiguous_cache_under_churn():
    """Three streams share a small page pool: prefill, verify-style forwards with commits and
    rollbacks, one stream leaves and another prefix joins in its place.  Every forward must give
    bit-identical logits to the same history on a private contiguous cache; pages are conserved,
    never owned twice, and a rollback returns exactly the pages beyond the committed length."""
    shape = small_shape()
    w = synth.make_weights(shape, 21)
    m = oracle_model(shape, w)
    P = orc.PAGE_TOKENS
    n_pages = 9
    cache = orc.PagedCache(m, 3, n_pages, 4)
    rng = np.random.default_rng(4)

    def check_pages():
        owned = [pg for t in cache.table for pg in t]
        assert len(owned) == len(set(owned))
        assert sorted(owned + cache.free) == list(range(n_pages))
        for b in range(3):
            assert len(cache.table[b]) == -(-cache.length[b] // P)

    plain = [orc.Stream(m, 4 * P) for _ in range(3)]
    lens = [70, 5, 130]
    for b, n in enumerate(lens):
        ids = rng.integers(0, shape.vocab_out, size=n)
        for s0 in range(0, n - 1, 50):                     # chunked prefill on both
            part = ids[s0:min(s0 + 50, n - 1)]
            a = orc.forward_paged(m, cache, b, part)
            cache.length[b] += len(part)
            r = orc.forward(m, plain[b], part)
            plain[b].length += len(part)
            assert np.array_equal(a, r)
        cache.pending[b] = plain[b].pending = int(ids[-1])
    check_pages()
    for step in range(6):
        for b in range(3):
            draft = rng.integers(0, shape.vocab_out, size=4)
            ids = np.concatenate([[plain[b].pending], draft])
            a = orc.forward_paged(m, cache, b, ids)
            r = orc.forward(m, plain[b], ids)
            assert np.array_equal(a, r)
            k = int(rng.integers(0, 5))
            y = int(rng.integers(0, shape.vocab_out))
            orc.commit_paged(cache, b, k, y)               # releases the provisional pages
            orc.commit(plain[b], k, y)
        check_pages()
    # rollback across a page boundary frees that page at once
    before = len(cache.free)
    b = 2
    assert cache.length[b] > 2 * P
    held = len(cache.table[b])
    orc.truncate_paged(cache, b, P - 3, 7)
    orc.truncate(plain[b], P - 3, 7)
    assert len(cache.table[b]) == 1 and len(cache.free) == before + held - 1
    check_pages()
    ids = np.array([7, 1, 2])
    assert np.array_equal(orc.forward_paged(m, cache, b, ids), orc.forward(m, plain[b], ids))
    cache.release(b)
    # stream 0 leaves; a new, longer prefix joins in its place and reuses the freed pages
    orc.truncate_paged(cache, 0, 0, -1)
    assert cache.table[0] == []
    plain[0] = orc.Stream(m, 4 * P)
    ids = rng.integers(0, shape.vocab_out, size=150)
    a = orc.forward_paged(m, cache, 0, ids[:-1])
    cache.length[0] += 149
    r = orc.forward(m, plain[0], ids[:-1])
    plain[0].length += 149
    assert np.array_equal(a, r)
    check_pages()
    # the other streams' data survived the churn
    for b in (1, 2):
        ids = np.array([plain[b].pending, 3, 4])
        assert np.array_equal(orc.forward_paged(m, cache, b, ids), orc.forward(m, plain[b], ids))
        cache.release(b)
    check_pages()
    # the pool is finite: asking for more than it holds fails loudly
    with pytest.raises(AssertionError):
        cache.ensure(1, 4 * P)
        cache.ensure(2, 4 * P)
        cache.ensure(0, 4 * P)
