"""Glue used by tests only: build oracle objects from the synthetic generators."""
from __future__ import annotations

import numpy as np

from oracle import ssd_oracle as orc
from paper_2505_15380_b200 import synth


def oracle_model(shape: synth.ModelShape, weights) -> orc.Model:
    return orc.Model(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                     n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ffn=shape.d_ffn,
                     vocab_out=shape.vocab_out, vocab_text=shape.vocab_text,
                     rope_theta=shape.rope_theta, rms_eps=shape.rms_eps,
                     kv_bf16=(shape.weight_dtype == synth.BF16), weights=weights)


def small_shape(**kw) -> synth.ModelShape:
    base = dict(n_layers=2, d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16, d_ffn=96,
                vocab_out=40, vocab_text=8, rope_theta=1e4, weight_dtype=synth.F32)
    base.update(kw)
    return synth.ModelShape(**base)


def crafted_draft_rows(q_logits: np.ndarray, sigma: float, temperature: float, top_k: int,
                       seed: int) -> np.ndarray:
    """Draft rows that resemble the target's: transform(target logits + sigma * noise).

    q_logits [gamma, V] are ORACLE logits; used so that every accepted length 0..gamma and both
    the residual and the bonus branch get exercised (independent random models almost always
    reject at the first position).
    """
    rng = np.random.Generator(np.random.Philox(key=[seed, 21]))
    noisy = q_logits + sigma * rng.standard_normal(q_logits.shape)
    return np.stack([orc.transform(r, temperature, top_k) for r in noisy]).astype(np.float32)
