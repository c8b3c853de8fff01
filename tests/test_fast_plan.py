"""Host-side logic of the persistent small-batch kernel: the split of the projections over the
CTAs and the packing of the weights into per-warp streams (no GPU needed)."""
import ctypes

import numpy as np
import pytest

from paper_2505_15380_b200 import binding, synth


@pytest.fixture(scope="module")
def L():
    return binding.lib()


def _plan(L, shape, n_cta):
    cfg = binding.make_config(shape)
    out = (ctypes.c_int64 * 8)()
    rc = L.ssd_fast_plan_host(ctypes.byref(cfg), n_cta, out)
    return rc, list(out)


def test_plan_streams_every_projection_byte_once_and_evenly(L):
    shape = synth.workload(1).target                      # 24 layers, d 896, FFN 4864, vocab 6564
    rc, (total, mn, mx, max_units, max_chunks, down_split, o_split, n_tiles) = _plan(L, shape, 148)
    assert rc == 0
    d, F, V, Lyr = shape.d_model, shape.d_ffn, shape.vocab_out, shape.n_layers
    qd, kvd = shape.n_q_heads * shape.head_dim, shape.n_kv_heads * shape.head_dim
    per_layer = (qd + 2 * kvd) * d + d * qd + 3 * F * d
    head_rows = (V + 7) // 8 * 8                          # the last tile of the LM head is padded
    assert total == 2 * (Lyr * per_layer + head_rows * d)
    # the algorithmic bytes of the step (norm gains, biases and head padding aside)
    assert abs(total - shape.streamed_weight_bytes()) < 256 * 1024
    assert mx <= 1.08 * total / 148 and mn >= 0.92 * total / 148      # balanced streams
    assert down_split == 8 and o_split == 14 and max_units <= 16 and max_chunks <= 128
    # tiles: every projection's tiles once; the O projection's once per query head and the down
    # projection's once per K slice (both are split over K)
    tiles = (qd + 2 * kvd) // 8 + shape.n_q_heads * d // 8 + 2 * F // 8 + down_split * d // 8 + (V + 7) // 8
    assert n_tiles == tiles


@pytest.mark.parametrize("n_cta", [1, 7, 132, 148, 160])
def test_plan_holds_for_other_sm_counts(L, n_cta):
    shape = synth.ModelShape(3, 256, 8, 2, 64, 1408, 1000, 16, 1e6, weight_dtype=synth.BF16)
    rc, out = _plan(L, shape, n_cta)
    assert rc == 0
    qd, kvd, d, F = 512, 128, 256, 1408
    assert out[0] == 2 * (3 * ((qd + 2 * kvd) * d + d * qd + 3 * F * d) + 1000 * d)
    if n_cta >= 7:
        assert out[2] <= 1.35 * out[0] / n_cta


def test_k_slices_stay_within_the_arrival_count(L):
    """Projections split over K add into residual words that count arrivals in 4 bits: never more
    than 16 slices, whole heads per slice of the O projection, and a CTA for every slice."""
    for hq, hkv, n_cta, want in [(14, 2, 148, 14), (32, 2, 148, 16), (28, 4, 148, 14), (17, 17, 148, 1),
                                 (12, 2, 148, 12), (8, 1, 7, 4), (8, 1, 1, 1), (64, 8, 148, 16)]:
        shape = synth.ModelShape(2, 256, hq, hkv, 32, 8960, 500, 0, 1e4, weight_dtype=synth.BF16)
        rc, out = _plan(L, shape, n_cta)
        assert rc == 0 and out[6] == want and out[5] <= 16
        assert hq % out[6] == 0


def test_plan_rejects_models_without_the_path(L):
    assert _plan(L, synth.workload(0).target, 148)[0] == -2            # fp32 weights
    odd = synth.ModelShape(2, 128, 6, 2, 64, 200, 300, 8, 1e4, weight_dtype=synth.BF16)
    assert _plan(L, odd, 148)[0] == -2                                  # FFN width not a multiple of 16


@pytest.mark.parametrize("shape,n_cta", [
    (synth.ModelShape(2, 64, 4, 2, 64, 96, 300, 8, 1e4, weight_dtype=synth.BF16), 148),
    (synth.ModelShape(2, 128, 14, 2, 64, 256, 301, 8, 1e4, weight_dtype=synth.BF16), 148),
    (synth.ModelShape(1, 256, 4, 2, 128, 2816, 700, 8, 1e4, weight_dtype=synth.BF16), 37),
    (synth.ModelShape(2, 128, 4, 2, 32, 512, 513, 0, 1e4, weight_dtype=synth.BF16), 5),
    (synth.ModelShape(1, 64, 32, 4, 32, 64, 100, 0, 1e4, weight_dtype=synth.BF16), 148),   # two heads per O slice
    (synth.ModelShape(1, 64, 5, 5, 64, 64, 100, 0, 1e4, weight_dtype=synth.BF16), 3),      # all heads in one slice
])
def test_pack_then_walk_the_streams_reproduces_every_weight(L, shape, n_cta):
    """Packing permutes rows (rotary partners and gate/up made adjacent), tiles and splits K;
    walking the streams the way a consumer does must put every weight back where it was."""
    w = synth.make_weights(shape, 5)
    blob = np.ascontiguousarray(synth.weights_blob(shape, w))
    cfg = binding.make_config(shape)
    out = np.zeros_like(blob)
    bad = ctypes.c_int64(-1)
    rc = L.ssd_fast_pack_roundtrip_host(ctypes.byref(cfg), n_cta, blob.ctypes.data, blob.nbytes,
                                        out.ctypes.data, ctypes.byref(bad))
    assert rc == 0 and bad.value == 0
    a = blob.view(np.uint16).ravel()
    b = out.view(np.uint16).ravel()
    d, F, V = shape.d_model, shape.d_ffn, shape.vocab_out
    qd, kvd = shape.n_q_heads * shape.head_dim, shape.n_kv_heads * shape.head_dim
    off = (V + shape.vocab_text) * d                       # embedding: not packed
    assert not b[:off].any()
    for _ in range(shape.n_layers):
        for n, packed in ((d, False), (qd * d, True), (qd, False), (kvd * d, True), (kvd, False),
                          (kvd * d, True), (kvd, False), (d * qd, True), (d, False), (F * d, True),
                          (F * d, True), (d * F, True)):
            if packed:
                assert np.array_equal(a[off:off + n], b[off:off + n])
            else:
                assert not b[off:off + n].any()            # gains and biases travel separately
            off += n
    off += d
    assert np.array_equal(a[off:off + V * d], b[off:off + V * d])
    assert off + V * d == a.size
