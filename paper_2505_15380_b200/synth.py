"""Seeded synthetic inputs for the SSD verify path: model shapes, weights, ids, uniforms.

This module only *generates data*.  It holds none of the method's arithmetic (no decoder
forward, no acceptance rule, no sampling transform) and is the one module that both the CPU
oracle's tests and the CUDA path's tests / bench draw their inputs from.  Nothing here imports
the oracle or the CUDA binding.

The paper evaluates on LibriTTS prompts with trained CosyVoice 2 weights (Sec. 3.1-3.2); neither
is available, so these generators stand in: same shapes, sequence-length mix and id ranges, with
random-init weights.

Conventions
-----------
* Weights are i.i.d. N(0, 0.02); norm gains are 1.  For a bf16 model every value is rounded to
  bf16 (round-to-nearest-even) and handed out as float32 arrays holding exactly those values.
* Uniform draws come from Philox4x32-10 with key (seed, 0) and counter
  (row r, stream b, step, purpose) where purpose 0 is the acceptance draw r_i of Eq. 5 and
  purpose 1 is the categorical draw used by the resample of Eq. 6 / the bonus token;
  u = (x >> 8) * 2**-24 lies in [0, 1).
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Tuple

import numpy as np

F32 = 0
BF16 = 1


@dataclasses.dataclass(frozen=True)
class ModelShape:
    """Decoder shape (the paper's target is a 24-layer Qwen2.5-0.5B-style LM, Sec. 3.1)."""
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab_out: int           # speech-token vocabulary (rows of the LM head)
    vocab_text: int          # extra embedding rows for text ids (prefill only)
    rope_theta: float
    rms_eps: float = 1e-6
    weight_dtype: int = BF16  # F32 or BF16; the KV cache uses the same storage type
    qkv_bias: int = 1

    @property
    def vocab_in(self) -> int:
        return self.vocab_out + self.vocab_text

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    def tensor_list(self) -> List[Tuple[str, Tuple[int, ...]]]:
        """Names and shapes in the order of the flat weight blob handed to ssd_model_create."""
        d, qd, kvd, f = self.d_model, self.q_dim, self.kv_dim, self.d_ffn
        out: List[Tuple[str, Tuple[int, ...]]] = [("embed", (self.vocab_in, d))]
        for l in range(self.n_layers):
            p = f"l{l}."
            out += [(p + "norm1", (d,)),
                    (p + "wq", (qd, d)), (p + "bq", (qd,)),
                    (p + "wk", (kvd, d)), (p + "bk", (kvd,)),
                    (p + "wv", (kvd, d)), (p + "bv", (kvd,)),
                    (p + "wo", (d, qd)),
                    (p + "norm2", (d,)),
                    (p + "wg", (f, d)), (p + "wu", (f, d)), (p + "wd", (d, f))]
        out += [("norm_f", (d,)), ("head", (self.vocab_out, d))]
        return out

    def n_params(self) -> int:
        return sum(int(np.prod(s)) for _, s in self.tensor_list())

    def streamed_weight_bytes(self) -> int:
        """Bytes of weights one verify step must read: everything but the embedding table."""
        el = 4 if self.weight_dtype == F32 else 2
        return el * sum(int(np.prod(s)) for n, s in self.tensor_list() if n != "embed")

    def kv_bytes_per_token(self) -> int:
        el = 4 if self.weight_dtype == F32 else 2
        return self.n_layers * 2 * self.kv_dim * el


@dataclasses.dataclass(frozen=True)
class Workload:
    """One verify-step workload: which model, how many streams, gamma, sampling parameters."""
    name: str
    target: ModelShape
    draft: ModelShape
    batch: int
    gamma: int
    temperature: float
    top_k: int               # 0 = off
    prefix_lens: Tuple[int, ...]   # tokens per stream, including the pending (last) token
    n_text: int              # leading ids of each prefix drawn from the text-id range
    model_seed: int
    data_seed: int


_TINY_T = ModelShape(2, 128, 4, 2, 32, 512, 512, 0, 1e4, weight_dtype=F32)
_TINY_D = ModelShape(1, 64, 2, 1, 32, 256, 512, 0, 1e4, weight_dtype=F32)
_QWEN_T = ModelShape(24, 896, 14, 2, 64, 4864, 6564, 32768, 1e6)
_QWEN_D = ModelShape(4, 512, 8, 2, 64, 2048, 6564, 32768, 1e6)
_LARGE_T = ModelShape(28, 1536, 12, 2, 128, 8960, 6564, 32768, 1e6)


def ragged_lengths(batch: int, lo: int, hi: int, seed: int) -> Tuple[int, ...]:
    rng = np.random.Generator(np.random.Philox(key=seed + 77))
    return tuple(int(v) for v in rng.integers(lo, hi + 1, size=batch))


def workload(cfg: int, gamma: int | None = None, prefix: int | None = None) -> Workload:
    """The five benchmark configurations (0 tiny fp32 ... 4 large batched)."""
    if cfg == 0:
        return Workload("cfg0_tiny_fp32", _TINY_T, _TINY_D, 1, gamma or 4, 1.0, 0,
                        (prefix or 64,), 0, 1000, 0)
    if cfg == 1:
        return Workload("cfg1_qwen2style_b1", _QWEN_T, _QWEN_D, 1, gamma or 4, 1.0, 0,
                        (prefix or 300,), 60, 1001, 1)
    if cfg == 2:
        g, n = gamma or 4, prefix or 1024
        return Workload(f"cfg2_sweep_g{g}_n{n}", _QWEN_T, _QWEN_D, 1, g, 1.0, 0, (n,), 0, 1001, 2)
    if cfg == 3:
        return Workload("cfg3_b16_ragged", _QWEN_T, _QWEN_D, 16, gamma or 5, 0.8, 25,
                        ragged_lengths(16, 200, 1500, 3), 0, 1001, 3)
    if cfg == 4:
        return Workload("cfg4_large_b64", _LARGE_T, _QWEN_D, 64, gamma or 6, 0.8, 25,
                        tuple([prefix or 4096] * 64), 0, 1004, 4)
    raise ValueError(f"unknown config {cfg}")


# --------------------------------------------------------------------------- storage formats

def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result is float32."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of bf16-representable float32 values."""
    return (bf16_round(x).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------- weights

def make_weights(shape: ModelShape, seed: int) -> Dict[str, np.ndarray]:
    """All tensors of `shape` as float32 arrays (bf16-valued when the model stores bf16)."""
    rng = np.random.Generator(np.random.Philox(key=seed))
    w: Dict[str, np.ndarray] = {}
    for name, shp in shape.tensor_list():
        if "norm" in name:
            t = np.ones(shp, dtype=np.float32)
        else:
            t = rng.standard_normal(shp, dtype=np.float32) * np.float32(0.02)
            if shape.weight_dtype == BF16:
                t = bf16_round(t)
        w[name] = t
    return w


def weights_blob(shape: ModelShape, w: Dict[str, np.ndarray]) -> np.ndarray:
    """Flat host blob in tensor_list() order, elements in the model's storage dtype."""
    parts = []
    for name, shp in shape.tensor_list():
        t = w[name].reshape(-1)
        parts.append(t.astype(np.float32) if shape.weight_dtype == F32 else to_bf16_bits(t))
    return np.concatenate(parts)


# --------------------------------------------------------------------------- token ids

def make_prefix(wl: Workload, stream: int) -> np.ndarray:
    """Prefix ids of one stream: n_text ids from the text range, the rest speech ids."""
    n = wl.prefix_lens[stream]
    rng = np.random.Generator(np.random.Philox(key=[wl.data_seed, 1 + stream]))
    ids = rng.integers(0, wl.target.vocab_out, size=n).astype(np.int32)
    nt = min(wl.n_text, n - 1) if wl.target.vocab_text > 0 else 0
    if nt > 0:
        ids[:nt] = wl.target.vocab_out + rng.integers(0, wl.target.vocab_text, size=nt)
    return ids


# --------------------------------------------------------------------------- Philox uniforms

_M0, _M1 = 0xD2511F53, 0xCD9E8D57
_W0, _W1 = 0x9E3779B9, 0xBB67AE85


def philox4x32_10(counter: np.ndarray, key: Tuple[int, int]) -> np.ndarray:
    """Philox4x32 with 10 rounds.  counter: uint32 [..., 4]; returns uint32 [..., 4]."""
    c = np.array(counter, dtype=np.uint64, copy=True)
    c0, c1, c2, c3 = (c[..., i].copy() for i in range(4))
    k0, k1 = np.uint64(key[0] & 0xFFFFFFFF), np.uint64(key[1] & 0xFFFFFFFF)
    mask = np.uint64(0xFFFFFFFF)
    for _ in range(10):
        p0 = np.uint64(_M0) * c0
        p1 = np.uint64(_M1) * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & mask
        hi1, lo1 = p1 >> np.uint64(32), p1 & mask
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & mask, lo1, (hi0 ^ c3 ^ k1) & mask, lo0
        k0 = (k0 + np.uint64(_W0)) & mask
        k1 = (k1 + np.uint64(_W1)) & mask
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def verify_uniforms(seed: int, batch: int, rows: int, step: int = 0) -> np.ndarray:
    """float32 [batch, rows, 2]: [..., 0] acceptance draws r_i, [..., 1] categorical draws."""
    ctr = np.zeros((batch, rows, 2, 4), dtype=np.uint32)
    ctr[..., 0] = np.arange(rows, dtype=np.uint32)[None, :, None]
    ctr[..., 1] = np.arange(batch, dtype=np.uint32)[:, None, None]
    ctr[..., 2] = np.uint32(step)
    ctr[..., 3] = np.arange(2, dtype=np.uint32)[None, None, :]
    x = philox4x32_10(ctr, (seed, 0))[..., 0]
    return ((x >> np.uint32(8)).astype(np.float32) * np.float32(2.0 ** -24)).astype(np.float32)


# --------------------------------------------------------------------------- draft rows

def random_prob_rows(n_rows: int, vocab: int, seed: int, sharpness: float = 2.0,
                     support: int = 0) -> np.ndarray:
    """Random categorical distributions, float32 [n_rows, vocab], each summing to ~1.

    Stand-in for draft-model rows p_i when no draft model is run: Gaussian scores scaled by
    `sharpness`, exponentiated and normalised; with `support` > 0 only that many randomly
    chosen ids per row are non-zero (like a top-k sampled draft).
    """
    rng = np.random.Generator(np.random.Philox(key=[seed, 9]))
    s = rng.standard_normal((n_rows, vocab)) * sharpness
    if 0 < support < vocab:
        keep = np.argsort(rng.random((n_rows, vocab)), axis=1)[:, :support]
        m = np.full((n_rows, vocab), -np.inf)
        np.put_along_axis(m, keep, 0.0, axis=1)
        s = s + m
    e = np.exp(s - s.max(axis=1, keepdims=True))
    return (e / e.sum(axis=1, keepdims=True)).astype(np.float32)


def sample_from_rows(p: np.ndarray, seed: int) -> np.ndarray:
    """One id per row drawn from p by inverse CDF (int32 [n_rows]); ids always have p > 0."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 10]))
    u = rng.random(p.shape[0])
    cdf = np.cumsum(p.astype(np.float64), axis=1)
    idx = (cdf > (u * cdf[:, -1])[:, None]).argmax(axis=1)
    return idx.astype(np.int32)


def fill_synthetic_kv(kv, lens, seed: int, std: float = 0.6) -> None:
    """Seeded random prefix K/V written into a device cache tensor
    kv[layer, stream, 2, kv_head, capacity, head_dim] for slots < lens[stream].

    Stand-in for a real prefill where that would take too long: entries ~ N(0, std^2) in the
    cache's storage type (std 0.6 is what random-init projections of unit-RMS inputs produce).
    """
    import torch
    g = torch.Generator(device=kv.device)
    g.manual_seed(seed)
    for b, n in enumerate(lens):
        blk = torch.randn((kv.shape[0], 2, kv.shape[3], int(n), kv.shape[5]), generator=g,
                          device=kv.device, dtype=torch.float32) * std
        kv[:, b, :, :, :int(n), :] = blk.to(kv.dtype)
