"""Host-side checks of the seeded input generators (no GPU, no oracle)."""
import numpy as np

from paper_2505_15380_b200 import synth


def _kat(path):
    rows = []
    with open(path) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                rows.append([int(t, 16) for t in line.split()])
    return rows


def test_philox_known_answers():
    import os
    here = os.path.dirname(__file__)
    for row in _kat(os.path.join(here, "golden", "philox4x32_10_kat.txt")):
        ctr, key, want = row[0:4], row[4:6], row[6:10]
        got = synth.philox4x32_10(np.array(ctr, dtype=np.uint32), (key[0], key[1]))
        assert [int(v) for v in got] == want


def test_uniforms_range_and_determinism():
    u = synth.verify_uniforms(0, 3, 9)
    assert u.shape == (3, 9, 2) and u.dtype == np.float32
    assert (u >= 0).all() and (u < 1).all()
    assert np.array_equal(u, synth.verify_uniforms(0, 3, 9))
    assert not np.array_equal(u, synth.verify_uniforms(1, 3, 9))
    assert not np.array_equal(u[..., 0], u[..., 1])
    big = synth.verify_uniforms(5, 64, 9, step=3).ravel()
    assert abs(big.mean() - 0.5) < 0.05


def test_bf16_round_ties_to_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -9, -0.3], np.float32)
    r = synth.bf16_round(x)
    # 1 + 2^-8 lies half-way between 1 and 1 + 2^-7: ties go to the even mantissa (1.0)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == np.float32(1.0 + 2 ** -6) and r[3] == 1.0
    assert np.array_equal(synth.from_bf16_bits(synth.to_bf16_bits(x)), r)
    assert abs(r[4] + 0.3) < 0.3 * 2 ** -8


def test_byte_counts_match_shape_arithmetic():
    qwen = synth.workload(1).target
    per_layer = 2 * 896 * 896 + 2 * 896 * 128 + 3 * 896 * 4864 + 1152 + 2 * 896
    assert qwen.streamed_weight_bytes() == 2 * (24 * per_layer + 6564 * 896 + 896) == 727_558_912
    assert qwen.kv_bytes_per_token() == 12_288
    large = synth.workload(4).target
    assert large.streamed_weight_bytes() == 2_640_845_824
    assert large.kv_bytes_per_token() == 28_672


def test_weights_blob_layout():
    shape = synth.workload(0).target
    w = synth.make_weights(shape, 1000)
    blob = synth.weights_blob(shape, w)
    assert blob.dtype == np.float32 and blob.size == shape.n_params()
    off = 0
    for name, shp in shape.tensor_list():
        n = int(np.prod(shp))
        assert np.array_equal(blob[off:off + n], w[name].ravel())
        off += n
    assert abs(float(w["l0.wq"].std()) - 0.02) < 0.002
    assert np.all(w["l1.norm2"] == 1.0)


def test_bf16_weights_are_bf16_valued():
    shape = synth.ModelShape(1, 64, 2, 1, 32, 128, 50, 10, 1e6)
    w = synth.make_weights(shape, 3)
    assert np.array_equal(synth.bf16_round(w["l0.wg"]), w["l0.wg"])
    blob = synth.weights_blob(shape, w)
    assert blob.dtype == np.uint16 and blob.size == shape.n_params()


def test_prefix_ids_ranges():
    wl = synth.workload(1)
    ids = synth.make_prefix(wl, 0)
    assert len(ids) == 300
    assert (ids[:60] >= 6564).all() and (ids[:60] < 6564 + 32768).all()
    assert (ids[60:] >= 0).all() and (ids[60:] < 6564).all()
    wl3 = synth.workload(3)
    assert len(wl3.prefix_lens) == 16 and min(wl3.prefix_lens) >= 200 and max(wl3.prefix_lens) <= 1500


def test_random_prob_rows():
    p = synth.random_prob_rows(5, 100, 1, support=10)
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-5)
    assert ((p > 0).sum(axis=1) == 10).all()
    x = synth.sample_from_rows(p, 2)
    assert (p[np.arange(5), x] > 0).all()
